"""ctypes loader for the fp64 CPU oracle (test infrastructure only).

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may import this package.
It shares nothing with the CUDA library: the C file is compiled on its own with gcc.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "iq_oracle.c")
_LIB = os.path.join(_HERE, "libiq_oracle.so")

_c_int = ctypes.c_int
_c_i64 = ctypes.c_int64
_c_dbl = ctypes.c_double
_vp = ctypes.c_void_p


def build(force: bool = False) -> str:
    """Compile oracle/iq_oracle.c into oracle/libiq_oracle.so (gcc -O2 -fopenmp)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.iqo_half_to_double.restype = _c_dbl
        _lib.iqo_half_to_double.argtypes = [ctypes.c_uint16]
        _lib.iqo_quantize_row.restype = ctypes.c_float
        _lib.iqo_quantize_append.restype = _c_i64
        _lib.iqo_num_threads.restype = _c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(_vp)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _u16(a):
    a = np.ascontiguousarray(a)
    if a.dtype == np.float16:
        a = a.view(np.uint16)
    assert a.dtype == np.uint16
    return a


def num_threads() -> int:
    return int(lib().iqo_num_threads())


def set_num_threads(n: int) -> None:
    lib().iqo_set_num_threads(_c_int(int(n)))


def row_bytes(d: int, bits: int = 3) -> int:
    return bits * d // 8


def so4_block(q8) -> np.ndarray:
    q8 = _f32(q8).reshape(8)
    M = np.zeros((4, 4), dtype=np.float64)
    lib().iqo_so4_block(_p(q8), _p(M))
    return M


def hadamard(d: int) -> np.ndarray:
    H = np.zeros((d, d), dtype=np.float64)
    lib().iqo_hadamard(_c_int(d), _p(H))
    return H


def rotation_matrix(d: int, quats) -> np.ndarray:
    """quats: [d/4][8] fp32 of one KV head -> dense R [d][d] (fp64)."""
    quats = _f32(quats).reshape(d // 4, 8)
    R = np.zeros((d, d), dtype=np.float64)
    lib().iqo_rotation_matrix(_c_int(d), _p(quats), _p(R))
    return R


def quantize_row(d: int, R, thresholds, x_half):
    """One row (fp16) -> (codes uint8 [d], fp32 scale, u fp64 [d]). The number of thresholds (3, 7 or 15) gives the bit width."""
    R = np.ascontiguousarray(R, dtype=np.float64)
    th = _f32(thresholds).reshape(-1)
    bits = {3: 2, 7: 3, 15: 4}[th.size]
    x = _u16(x_half).reshape(d)
    codes = np.zeros(d, dtype=np.uint8)
    u = np.zeros(d, dtype=np.float64)
    s = lib().iqo_quantize_row(_c_int(d), _c_int(bits), _p(R), _p(th), _p(x), _p(codes), _p(u))
    return codes, np.float32(s), u


def pack_row(d: int, codes, bits: int = 3) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8).reshape(d)
    row = np.zeros(row_bytes(d, bits), dtype=np.uint8)
    lib().iqo_pack_row(_c_int(d), _c_int(bits), _p(codes), _p(row))
    return row


def unpack_row(d: int, row, bits: int = 3) -> np.ndarray:
    row = np.ascontiguousarray(row, dtype=np.uint8).reshape(row_bytes(d, bits))
    codes = np.zeros(d, dtype=np.uint8)
    lib().iqo_unpack_row(_c_int(d), _c_int(bits), _p(row), _p(codes))
    return codes


def v_row_codes(d: int, v_area, t: int, bits: int = 3) -> np.ndarray:
    """Codes of V row t from the token-transposed V bytes of one (sequence, KV head): v_area is the uint8 array
    [t_cap][3d/8] slice of that head (viewed flat)."""
    area = np.ascontiguousarray(v_area, dtype=np.uint8).reshape(-1)
    codes = np.zeros(d, dtype=np.uint8)
    lib().iqo_v_row_codes(_c_int(d), _c_int(bits), _p(area), _c_i64(int(t)), _p(codes))
    return codes


def new_cache(B: int, H_kv: int, d: int, t_cap: int, bits: int = 3):
    assert t_cap % 128 == 0, "t_cap must be a multiple of 128 (token-transposed V blocks)"
    P = row_bytes(d, bits)
    return dict(
        k_codes=np.zeros((B, H_kv, t_cap, P), dtype=np.uint8),
        k_scales=np.zeros((B, H_kv, t_cap), dtype=np.float32),
        v_codes=np.zeros((B, H_kv, t_cap, P), dtype=np.uint8),
        v_scales=np.zeros((B, H_kv, t_cap), dtype=np.float32),
    )


def round_scales_fp16(cache) -> None:
    """The binary16-scales variant of the cache (50 instead of 52 bytes per row and side): every stored norm rounded to
    the nearest binary16 value (saturating at 65504), kept in the fp32 arrays. Rows are normalised by their exact norm
    either way; only the stored scale, which decode multiplies back, is rounded. Idempotent."""
    for name in ("k_scales", "v_scales"):
        a = cache[name]
        a[...] = np.minimum(a, np.float32(65504.0)).astype(np.float16).astype(np.float32)


def _bits_of_cache(cache, d: int) -> int:
    return cache["k_codes"].shape[3] * 8 // d


def quantize_append(quats, thresholds, k_new, v_new, append_pos, n_new, cache, thresholds_v=None) -> int:
    """k_new, v_new: fp16 [B][n_new_max][H_kv][d] (any strides, last dim contiguous). Appends in place. thresholds:
    the 2^b - 1 thresholds of the K side (b from the cache's row size); thresholds_v: those of the V side (default: the same)."""
    k = k_new.view(np.uint16) if k_new.dtype == np.float16 else k_new
    v = v_new.view(np.uint16) if v_new.dtype == np.float16 else v_new
    B, n_max, H_kv, d = k.shape
    assert v.shape == k.shape and k.strides == v.strides and k.strides[3] == 2
    sb, st, sh = (s // 2 for s in k.strides[:3])
    t_cap = cache["k_scales"].shape[2]
    quats = _f32(quats).reshape(H_kv, d // 4, 8)
    bits = _bits_of_cache(cache, d)
    th = _f32(thresholds).reshape((1 << bits) - 1)
    thv = th if thresholds_v is None else _f32(thresholds_v).reshape((1 << bits) - 1)
    pos = np.ascontiguousarray(append_pos, dtype=np.int32).reshape(B)
    nn = None if n_new is None else np.ascontiguousarray(n_new, dtype=np.int32).reshape(B)
    for a in cache.values():
        assert a.flags["C_CONTIGUOUS"]
    return int(lib().iqo_quantize_append(
        _c_int(B), _c_int(H_kv), _c_int(d), _c_int(bits), _c_int(t_cap), _p(quats), _p(th), _p(thv), _p(k), _p(v),
        _c_i64(sb), _c_i64(st), _c_i64(sh), _p(pos), _p(nn), _c_int(n_max),
        _p(cache["k_codes"]), _p(cache["k_scales"]), _p(cache["v_codes"]), _p(cache["v_scales"])))


def decode_attention(quats, levels, q, cache, seq_lens, H_kv: int, sm_scale: float = 0.0, want_rot: bool = False, levels_v=None):
    """q: fp16 [B][H_q][d]. Returns dict(out [B][H_q][d] fp64, lse, argmax, (o_rot)). levels: the 2^b levels of the K side
    (b from the cache's row size); levels_v: those of the V side (default: the same)."""
    qq = _u16(q)
    B, H_q, d = qq.shape
    t_cap = cache["k_scales"].shape[2]
    quats = _f32(quats).reshape(H_kv, d // 4, 8)
    bits = _bits_of_cache(cache, d)
    lv = _f32(levels).reshape(1 << bits)
    lvv = lv if levels_v is None else _f32(levels_v).reshape(1 << bits)
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32).reshape(B)
    out = np.zeros((B, H_q, d), dtype=np.float64)
    lse = np.zeros((B, H_q), dtype=np.float64)
    am = np.zeros((B, H_q), dtype=np.int32)
    orot = np.zeros((B, H_q, d), dtype=np.float64) if want_rot else None
    for a in cache.values():
        assert a.flags["C_CONTIGUOUS"]
    lib().iqo_decode_attention(
        _c_int(B), _c_int(H_q), _c_int(H_kv), _c_int(d), _c_int(bits), _c_int(t_cap), _c_dbl(sm_scale), _p(quats), _p(lv), _p(lvv),
        _p(qq), _p(cache["k_codes"]), _p(cache["k_scales"]), _p(cache["v_codes"]), _p(cache["v_scales"]),
        _p(lens), _p(out), _p(lse), _p(am), _p(orot))
    r = dict(out=out, lse=lse, argmax=am)
    if want_rot:
        r["o_rot"] = orot
    return r


def reconstruct_rows(quats, levels, cache, seq_lens, H_kv: int, levels_v=None, d: int = 0):
    """Figure 1 (top), the reconstruct-then-compute model: every cached row of every (sequence, KV head) dequantised
    and rotated back, x_hat = R^T (scale * level[code] / sqrt(d)). Returns (K, V), fp64 [B][t_cap][H_kv][d]; rows
    beyond a sequence's length are zero."""
    B, _, t_cap = cache["k_scales"].shape
    nlev = _f32(levels).size
    bits = {4: 2, 8: 3, 16: 4}[nlev]
    d = d or cache["k_codes"].shape[3] * 8 // bits
    quats = _f32(quats).reshape(H_kv, d // 4, 8)
    lv = _f32(levels).reshape(nlev)
    lvv = lv if levels_v is None else _f32(levels_v).reshape(nlev)
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32).reshape(B)
    k = np.zeros((B, t_cap, H_kv, d), dtype=np.float64)
    v = np.zeros((B, t_cap, H_kv, d), dtype=np.float64)
    for a in cache.values():
        assert a.flags["C_CONTIGUOUS"]
    lib().iqo_reconstruct_rows(_c_int(B), _c_int(H_kv), _c_int(d), _c_int(bits), _c_int(t_cap), _p(quats), _p(lv), _p(lvv), _p(cache["k_codes"]),
                               _p(cache["k_scales"]), _p(cache["v_codes"]), _p(cache["v_scales"]), _p(lens), _p(k), _p(v))
    return k, v


def scores(quats, levels, q, cache, b: int, h: int, length: int, H_kv: int, sm_scale: float = 0.0) -> np.ndarray:
    qq = _u16(q)
    B, H_q, d = qq.shape
    t_cap = cache["k_scales"].shape[2]
    quats = _f32(quats).reshape(H_kv, d // 4, 8)
    bits = _bits_of_cache(cache, d)
    lv = _f32(levels).reshape(1 << bits)
    z = np.zeros(max(length, 1), dtype=np.float64)
    qbh = np.ascontiguousarray(qq[b, h])
    lib().iqo_scores(_c_int(H_q), _c_int(H_kv), _c_int(d), _c_int(bits), _c_int(t_cap), _c_dbl(sm_scale), _p(quats), _p(lv),
                     _p(qbh), _c_int(b), _c_int(h), _p(cache["k_codes"]), _p(cache["k_scales"]), _c_int(length), _p(z))
    return z[:length]


def combine_splits(quats, part_acc, part_ml, part_argmax, H_kv: int):
    """part_acc fp32 [B][H_q][S][d], part_ml fp32 [B][H_q][S][2], part_argmax int32 [B][H_q][S] or None."""
    pa = _f32(part_acc)
    B, H_q, S, d = pa.shape
    pm = _f32(part_ml).reshape(B, H_q, S, 2)
    pg = None if part_argmax is None else np.ascontiguousarray(part_argmax, dtype=np.int32).reshape(B, H_q, S)
    quats = _f32(quats).reshape(H_kv, d // 4, 8)
    out = np.zeros((B, H_q, d), dtype=np.float64)
    lse = np.zeros((B, H_q), dtype=np.float64)
    am = np.zeros((B, H_q), dtype=np.int32)
    lib().iqo_combine_splits(_c_int(B), _c_int(H_q), _c_int(H_kv), _c_int(d), _c_int(S), _p(quats), _p(pa), _p(pm),
                             _p(pg), _p(out), _p(lse), _p(am))
    return dict(out=out, lse=lse, argmax=am)
