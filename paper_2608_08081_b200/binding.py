"""ctypes binding of libisoquant.so: same names as the C ABI, argument marshalling only."""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

from . import build as _build

_vp = ctypes.c_void_p
_i32 = ctypes.c_int32
_i64 = ctypes.c_int64


class _IqShape(ctypes.Structure):
    _fields_ = [("batch", _i32), ("n_q_heads", _i32), ("n_kv_heads", _i32), ("head_dim", _i32),
                ("t_cap", _i32), ("bits", _i32), ("sm_scale", ctypes.c_float)]


class _IqCodebook(ctypes.Structure):
    _fields_ = [("bits", _i32), ("separate_v", _i32), ("levels", ctypes.c_float * 16), ("thresholds", ctypes.c_float * 15),
                ("v_levels", ctypes.c_float * 16), ("v_thresholds", ctypes.c_float * 15)]


class _IqCache(ctypes.Structure):
    _fields_ = [("k_codes", _vp), ("k_scales", _vp), ("v_codes", _vp), ("v_scales", _vp),
                ("block_table_dev", _vp), ("page_rows", _i32), ("num_pages", _i32), ("scales_fp16", _i32)]


class IQError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {iq_strerror(code)} ({code})")


def lib_path() -> str:
    return _build.LIB


def _load():
    path = lib_path()
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python paper_2608_08081_b200/build.py` (needs nvcc). "
            "There is no fallback implementation.")
    lib = ctypes.CDLL(path)
    lib.iq_version.restype = ctypes.c_int
    lib.iq_format_version.restype = ctypes.c_int
    lib.iq_strerror.restype = ctypes.c_char_p
    lib.iq_strerror.argtypes = [ctypes.c_int]
    lib.iq_row_bytes.restype = ctypes.c_size_t
    lib.iq_row_bytes.argtypes = [_i32]
    lib.iq_row_bytes_bits.restype = ctypes.c_size_t
    lib.iq_row_bytes_bits.argtypes = [_i32, _i32]
    lib.iq_lloyd_max_codebook.argtypes = [_i32, _i32, _i32, ctypes.POINTER(_IqCodebook)]
    lib.iq_codebook_set_v.argtypes = [ctypes.POINTER(_IqCodebook), ctypes.POINTER(_IqCodebook)]
    lib.iq_rotation_floats.restype = ctypes.c_size_t
    lib.iq_rotation_floats.argtypes = [_i32, _i32]
    lib.iq_default_codebook.argtypes = [_i32, ctypes.POINTER(_IqCodebook)]
    lib.iq_int8_codebook.argtypes = [_i32, ctypes.POINTER(_IqCodebook)]
    lib.iq_make_rotation.argtypes = [_i32, _i32, ctypes.c_uint64, _vp, _vp, _vp]
    lib.iq_quantize_append.argtypes = [ctypes.POINTER(_IqShape), _vp, ctypes.POINTER(_IqCodebook), _vp, _vp, _i64, _i64,
                                       _i64, _vp, _vp, _i32, ctypes.POINTER(_IqCache), _vp, _vp]
    lib.iq_decode_attention.argtypes = [ctypes.POINTER(_IqShape), _vp, ctypes.POINTER(_IqCodebook), _vp,
                                        ctypes.POINTER(_IqCache), _vp, _i32, _vp, _vp, _vp, _vp, _vp]
    lib.iq_combine_splits.argtypes = [ctypes.POINTER(_IqShape), _vp, _i32, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp]
    lib.iq_combine_splits_sharded.argtypes = [ctypes.POINTER(_IqShape), _vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp]
    lib.iq_static_scratch_bytes.restype = ctypes.c_size_t
    lib.iq_decode_attention_static.argtypes = [ctypes.POINTER(_IqShape), _vp, ctypes.POINTER(_IqCodebook), _vp,
                                               ctypes.POINTER(_IqCache), _vp, _i32, _vp, _i32, _vp, _vp, _vp]
    lib.iq_reconstruct_rows.argtypes = [ctypes.POINTER(_IqShape), _vp, ctypes.POINTER(_IqCodebook), ctypes.POINTER(_IqCache), _vp,
                                        _vp, _vp, _i32, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, _vp]
    lib.iq_decode_step_host.argtypes = [ctypes.POINTER(_IqShape), _vp, ctypes.POINTER(_IqCodebook), _vp, _vp, _vp, _vp,
                                        ctypes.POINTER(_IqCache), _i32, _vp, _vp, _vp, _vp, _i32, _vp, _vp]
    lib.iq_rotated_histogram.argtypes = [ctypes.POINTER(_IqShape), _vp, _vp, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, _vp,
                                         _i32, _vp, _i32, ctypes.c_float, _vp]
    lib.iq_fit_codebook.argtypes = [_vp, _i32, ctypes.c_float, _i32, _i32, _i32, ctypes.POINTER(_IqCodebook)]
    lib.iq_suggest_splits.restype = _i32
    lib.iq_suggest_splits.argtypes = [ctypes.POINTER(_IqShape), _i32]
    lib.iq_wht_coordinates.argtypes = [ctypes.POINTER(_IqShape), _vp, _i64, _i64, _i64, _vp, _i32, _vp, _vp]
    lib.iq_fit_rotation.argtypes = [_vp, _i32, _i64, _i32, ctypes.POINTER(_IqCodebook), _vp, _vp]
    lib.iq_selftest_bounded_wait.argtypes = [_vp, ctypes.c_uint32, _vp]
    lib.iq_decode_step_workspace_bytes.argtypes = [ctypes.POINTER(_IqShape), _i32]
    lib.iq_decode_step_workspace_bytes.restype = ctypes.c_size_t
    lib.iq_decode_step_fused.argtypes = [ctypes.POINTER(_IqShape), _vp, ctypes.POINTER(_IqCodebook), _vp, _vp, _vp,
                                         ctypes.POINTER(_IqCache), _vp, _i32, _vp, _vp, _i32, _vp, _vp, _vp, _vp]
    return lib


_lib = _load()


# Shape and Codebook are immutable, so each builds its C struct once: a decode step of a short batch is bound by the
# host's time per call, not by the kernels.
@dataclass(frozen=True)
class Shape:
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    t_cap: int
    bits: int = 3
    sm_scale: float = 0.0

    def c(self) -> _IqShape:
        cs = self.__dict__.get("_c")
        if cs is None:
            cs = _IqShape(self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim, self.t_cap, self.bits, self.sm_scale)
            object.__setattr__(self, "_c", cs)
        return cs


@dataclass(frozen=True)
class Codebook:
    """2^b ascending levels and 2^b - 1 thresholds (b = 2, 3 or 4, read off the number of levels); v_levels / v_thresholds:
    a codebook of their own for the V rows (None: the V rows use the same one)."""
    levels: tuple
    thresholds: tuple
    v_levels: tuple = None
    v_thresholds: tuple = None

    @property
    def bits(self) -> int:
        return {4: 2, 8: 3, 16: 4}[len(self.levels)]

    def c(self) -> _IqCodebook:
        cb = self.__dict__.get("_c")
        if cb is None:
            n = len(self.levels)
            assert len(self.thresholds) == n - 1
            cb = _IqCodebook()
            cb.bits = self.bits
            for i in range(n):
                cb.levels[i] = float(self.levels[i])
            for i in range(n - 1):
                cb.thresholds[i] = float(self.thresholds[i])
            if self.v_levels is not None:
                assert len(self.v_levels) == n and len(self.v_thresholds) == n - 1
                cb.separate_v = 1
                for i in range(n):
                    cb.v_levels[i] = float(self.v_levels[i])
                for i in range(n - 1):
                    cb.v_thresholds[i] = float(self.v_thresholds[i])
            object.__setattr__(self, "_c", cb)
        return cb

    def with_v(self, v_side: "Codebook") -> "Codebook":
        """This codebook for the K rows, v_side's (K side) for the V rows."""
        assert v_side.bits == self.bits
        return Codebook(self.levels, self.thresholds, tuple(v_side.levels), tuple(v_side.thresholds))


def _from_c(cb: _IqCodebook) -> Codebook:
    n = 1 << cb.bits
    if cb.separate_v:
        return Codebook(tuple(cb.levels[:n]), tuple(cb.thresholds[:n - 1]), tuple(cb.v_levels[:n]), tuple(cb.v_thresholds[:n - 1]))
    return Codebook(tuple(cb.levels[:n]), tuple(cb.thresholds[:n - 1]))


def iq_codebook_set_v(codebook: Codebook, v_side: Codebook) -> Codebook:
    """A two-sided codebook: `codebook` for the K rows, the K side of `v_side` for the V rows (through the C ABI)."""
    a, b = _IqCodebook.from_buffer_copy(codebook.c()), v_side.c()
    _check(_lib.iq_codebook_set_v(ctypes.byref(a), ctypes.byref(b)), "iq_codebook_set_v")
    return _from_c(a)


def iq_row_bytes_bits(head_dim: int, bits: int) -> int:
    return int(_lib.iq_row_bytes_bits(head_dim, bits))


@dataclass
class Cache:
    """Contiguous: k_codes uint8 [B][H_kv][t_cap][bits * d / 8], k_scales fp32 [B][H_kv][t_cap] (V alike). Paged: the same
    arrays with a pool of pages in place of the batch, [num_pages][H_kv][page_rows]..., and block_table int32
    [B][t_cap / page_rows] on the device."""
    k_codes: torch.Tensor
    k_scales: torch.Tensor
    v_codes: torch.Tensor
    v_scales: torch.Tensor
    block_table: Optional[torch.Tensor] = None
    page_rows: int = 0

    def c(self) -> _IqCache:
        assert self.k_scales.dtype == self.v_scales.dtype and self.k_scales.dtype in (torch.float32, torch.float16)
        f16 = 1 if self.k_scales.dtype == torch.float16 else 0   # binary16 scale arrays: 50 instead of 52 bytes per row
        if self.block_table is None:
            return _IqCache(self.k_codes.data_ptr(), self.k_scales.data_ptr(), self.v_codes.data_ptr(), self.v_scales.data_ptr(), None, 0, 0, f16)
        assert self.block_table.dtype == torch.int32 and self.block_table.is_contiguous()
        return _IqCache(self.k_codes.data_ptr(), self.k_scales.data_ptr(), self.v_codes.data_ptr(), self.v_scales.data_ptr(),
                        self.block_table.data_ptr(), self.page_rows, self.k_scales.shape[0], f16)


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def _check(rc: int, where: str):
    if rc != 0:
        raise IQError(rc, where)


def iq_version() -> int:
    return int(_lib.iq_version())


def iq_format_version() -> int:
    return int(_lib.iq_format_version())


def iq_strerror(code: int) -> str:
    return _lib.iq_strerror(int(code)).decode()


def iq_row_bytes(head_dim: int, bits: int = 3) -> int:
    return int(_lib.iq_row_bytes_bits(head_dim, bits))


def iq_lloyd_max_codebook(head_dim: int, bits: int, grid: str = "int8") -> Codebook:
    """2^bits Lloyd-Max levels for the post-rotation marginal; grid "int8" (integer decode path) or "fp16"."""
    cb = _IqCodebook()
    _check(_lib.iq_lloyd_max_codebook(head_dim, bits, {"fp16": 0, "int8": 1}[grid], ctypes.byref(cb)), "iq_lloyd_max_codebook")
    return _from_c(cb)


def iq_rotation_floats(head_dim: int, n_kv_heads: int) -> int:
    return int(_lib.iq_rotation_floats(head_dim, n_kv_heads))


def iq_default_codebook(head_dim: int) -> Codebook:
    cb = _IqCodebook()
    _check(_lib.iq_default_codebook(head_dim, ctypes.byref(cb)), "iq_default_codebook")
    return _from_c(cb)


def iq_int8_codebook(head_dim: int) -> Codebook:
    cb = _IqCodebook()
    _check(_lib.iq_int8_codebook(head_dim, ctypes.byref(cb)), "iq_int8_codebook")
    return _from_c(cb)


def iq_make_rotation(head_dim: int, n_kv_heads: int, seed: int, quats_host, rot_dev: torch.Tensor, stream=None) -> None:
    """quats_host: None or a contiguous fp32 numpy array [n_kv_heads][head_dim/4][8]."""
    qp = None
    if quats_host is not None:
        assert quats_host.dtype.name == "float32" and quats_host.flags["C_CONTIGUOUS"]
        assert quats_host.size == iq_rotation_floats(head_dim, n_kv_heads)
        qp = quats_host.ctypes.data
    _check(_lib.iq_make_rotation(head_dim, n_kv_heads, ctypes.c_uint64(seed), qp, _ptr(rot_dev), _stream(stream)),
           "iq_make_rotation")


def iq_quantize_append(shape: Shape, rot_dev, codebook: Codebook, k_new, v_new, append_pos_dev, n_new_dev,
                       n_new_max: int, cache: Cache, status_dev=None, stream=None) -> None:
    """k_new, v_new: fp16 device tensors [B][n_new_max][H_kv][d] (any strides with a contiguous last dim)."""
    assert k_new.dtype == torch.float16 and v_new.dtype == torch.float16
    assert k_new.stride() == v_new.stride() and k_new.stride(3) == 1
    sb, st, sh = k_new.stride(0), k_new.stride(1), k_new.stride(2)
    cs, cb, cc = shape.c(), codebook.c(), cache.c()
    _check(_lib.iq_quantize_append(ctypes.byref(cs), _ptr(rot_dev), ctypes.byref(cb), _ptr(k_new), _ptr(v_new), sb, st, sh,
                                   _ptr(append_pos_dev), _ptr(n_new_dev), n_new_max, ctypes.byref(cc), _ptr(status_dev),
                                   _stream(stream)), "iq_quantize_append")


def iq_decode_attention(shape: Shape, rot_dev, codebook: Codebook, q, cache: Cache, seq_lens_dev, num_splits: int,
                        part_acc, part_ml, part_argmax=None, status_dev=None, stream=None) -> None:
    cs, cb, cc = shape.c(), codebook.c(), cache.c()
    _check(_lib.iq_decode_attention(ctypes.byref(cs), _ptr(rot_dev), ctypes.byref(cb), _ptr(q), ctypes.byref(cc),
                                    _ptr(seq_lens_dev), num_splits, _ptr(part_acc), _ptr(part_ml), _ptr(part_argmax),
                                    _ptr(status_dev), _stream(stream)), "iq_decode_attention")


def iq_combine_splits(shape: Shape, rot_dev, num_splits: int, part_acc, part_ml, part_argmax, out, lse_out=None,
                      argmax_out=None, stream=None) -> None:
    cs = shape.c()
    _check(_lib.iq_combine_splits(ctypes.byref(cs), _ptr(rot_dev), num_splits, _ptr(part_acc), _ptr(part_ml),
                                  _ptr(part_argmax), _ptr(out), 1 if out.dtype == torch.float16 else 0, _ptr(lse_out),
                                  _ptr(argmax_out), _stream(stream)), "iq_combine_splits")


def iq_combine_splits_sharded(shape: Shape, rot_dev, num_splits: int, n_shards: int, part_acc, part_ml, part_argmax, row_offsets,
                              out, lse_out=None, argmax_out=None, stream=None) -> None:
    """Merge over the partials of n_shards ranks laid out rank after rank ([n_shards][B][H][S][..]), in place."""
    cs = shape.c()
    _check(_lib.iq_combine_splits_sharded(ctypes.byref(cs), _ptr(rot_dev), num_splits, n_shards, _ptr(part_acc), _ptr(part_ml),
                                          _ptr(part_argmax), _ptr(row_offsets), _ptr(out), 1 if out.dtype == torch.float16 else 0,
                                          _ptr(lse_out), _ptr(argmax_out), _stream(stream)), "iq_combine_splits_sharded")


def iq_decode_step_workspace_bytes(shape: Shape, num_splits: int) -> int:
    cs = shape.c()
    return int(_lib.iq_decode_step_workspace_bytes(ctypes.byref(cs), num_splits))


def iq_decode_step_fused(shape: Shape, rot_dev, codebook: Codebook, q, k_new, v_new, cache: Cache, seq_lens_dev, num_splits: int,
                         workspace, out, lse_out=None, argmax_out=None, status_dev=None, stream=None) -> None:
    """The decode step in two launches: the decode kernel also appends k_new / v_new [B][H_kv][d] at row seq_lens[b]
    (the lengths before the step), the merge takes the new row's partial as one more slot and rotates back into `out`.
    `workspace`: a device uint8 tensor of iq_decode_step_workspace_bytes(shape, num_splits) bytes."""
    cs, cb, cc = shape.c(), codebook.c(), cache.c()
    _check(_lib.iq_decode_step_fused(ctypes.byref(cs), _ptr(rot_dev), ctypes.byref(cb), _ptr(q), _ptr(k_new), _ptr(v_new),
                                     ctypes.byref(cc), _ptr(seq_lens_dev), num_splits, _ptr(workspace), _ptr(out),
                                     1 if out.dtype == torch.float16 else 0, _ptr(lse_out), _ptr(argmax_out), _ptr(status_dev),
                                     _stream(stream)), "iq_decode_step_fused")


def iq_static_scratch_bytes() -> int:
    return int(_lib.iq_static_scratch_bytes())


def iq_decode_attention_static(shape: Shape, rot_dev, codebook: Codebook, q, cache: Cache, seq_lens_dev, num_splits: int,
                               out, lse_out=None, status_dev=None, stream=None) -> None:
    """Decode + combine with the split partials in the library's fixed scratch array: for callers that cannot
    allocate device memory. Allocates nothing; calls that overlap on the GPU race on the shared array."""
    cs, cb, cc = shape.c(), codebook.c(), cache.c()
    _check(_lib.iq_decode_attention_static(ctypes.byref(cs), _ptr(rot_dev), ctypes.byref(cb), _ptr(q), ctypes.byref(cc),
                                           _ptr(seq_lens_dev), num_splits, _ptr(out), 1 if out.dtype == torch.float16 else 0,
                                           _ptr(lse_out), _ptr(status_dev), _stream(stream)), "iq_decode_attention_static")


def iq_reconstruct_rows(shape: Shape, rot_dev, codebook: Codebook, cache: Cache, seq_lens_dev, k_out, v_out, stream=None) -> None:
    """k_out, v_out: fp16 device tensors [B][T][H_kv][d] (any strides with a contiguous last dim): rows
    [0, min(seq_lens[b], T)) receive the reconstructed K and V rows, the others are left as they are."""
    assert k_out.dtype == torch.float16 and v_out.dtype == torch.float16 and k_out.shape == v_out.shape
    assert k_out.stride() == v_out.stride() and k_out.stride(3) == 1
    cs, cb, cc = shape.c(), codebook.c(), cache.c()
    _check(_lib.iq_reconstruct_rows(ctypes.byref(cs), _ptr(rot_dev), ctypes.byref(cb), ctypes.byref(cc), _ptr(seq_lens_dev),
                                    _ptr(k_out), _ptr(v_out), k_out.shape[1], k_out.stride(0), k_out.stride(1), k_out.stride(2),
                                    _stream(stream)),
           "iq_reconstruct_rows")


def iq_decode_step_host(shape: Shape, rot_dev, codebook: Codebook, inputs_host, inputs_dev, append_pos_dev, seq_lens_dev,
                        cache: Cache, ws: "DecodeWorkspace", out_dev, out_host, stream=None) -> None:
    """One decode step from host buffers (blocking): inputs_host = fp16 host tensor holding q, k_new, v_new back to
    back; inputs_dev a device tensor of the same size; out_dev / out_host fp32 or fp16 [B][H_q][d]."""
    assert inputs_host.dtype == torch.float16 and inputs_dev.dtype == torch.float16 and inputs_host.is_contiguous()
    n = shape.batch * (shape.n_q_heads + 2 * shape.n_kv_heads) * shape.head_dim
    assert inputs_host.numel() == n and inputs_dev.numel() == n and out_dev.dtype == out_host.dtype
    cs, cb, cc = shape.c(), codebook.c(), cache.c()
    _check(_lib.iq_decode_step_host(ctypes.byref(cs), _ptr(rot_dev), ctypes.byref(cb), _ptr(inputs_host), _ptr(inputs_dev),
                                    _ptr(append_pos_dev), _ptr(seq_lens_dev), ctypes.byref(cc), ws.num_splits, _ptr(ws.part_acc),
                                    _ptr(ws.part_ml), _ptr(out_dev), _ptr(out_host), 1 if out_dev.dtype == torch.float16 else 0,
                                    _ptr(ws.status), _stream(stream)), "iq_decode_step_host")


class HostStepper:
    """iq_decode_step_host for a loop of steps with every argument marshalled once: the step's host inputs are rows of one
    pinned tensor [n_steps][B * (H_q + 2 H_kv) * d], the lengths rows of one device table [n_steps + 1][B] (row i: before
    step i), and a step only adds offsets to base pointers. Same call, same kernels; what it saves is the host's time
    per step (tensor views, pointer queries, argument conversion), which sits inside an end-to-end step."""

    def __init__(self, shape: Shape, rot_dev, codebook: Codebook, inputs_host_all, inputs_dev, lens_table_dev, cache: Cache,
                 ws: "DecodeWorkspace", out_dev, out_host, stream=None):
        n = shape.batch * (shape.n_q_heads + 2 * shape.n_kv_heads) * shape.head_dim
        assert inputs_host_all.dtype == torch.float16 and inputs_host_all.dim() == 2 and inputs_host_all.shape[1] == n
        assert inputs_host_all.is_contiguous() and inputs_dev.dtype == torch.float16 and inputs_dev.numel() == n
        assert lens_table_dev.dtype == torch.int32 and lens_table_dev.is_contiguous() and lens_table_dev.shape[1] == shape.batch
        assert out_dev.dtype == out_host.dtype
        self._keep = (shape, codebook, cache, rot_dev, inputs_host_all, inputs_dev, lens_table_dev, ws, out_dev, out_host)
        self._cs, self._cb, self._cc = shape.c(), codebook.c(), cache.c()
        self._hin, self._hin_stride = inputs_host_all.data_ptr(), n * 2
        self._lens, self._lens_stride = lens_table_dev.data_ptr(), shape.batch * 4
        self.n_steps = min(inputs_host_all.shape[0], lens_table_dev.shape[0] - 1)
        self._fixed = (ctypes.byref(self._cs), _ptr(rot_dev), ctypes.byref(self._cb))
        self._tail = (ctypes.byref(self._cc), ws.num_splits, _ptr(ws.part_acc), _ptr(ws.part_ml), _ptr(out_dev), _ptr(out_host),
                      1 if out_dev.dtype == torch.float16 else 0, _ptr(ws.status), _stream(stream))
        self._din = _ptr(inputs_dev)

    def step(self, i: int) -> None:
        """Step i (blocking): inputs row i, lengths row i before and row i + 1 after the append."""
        rc = _lib.iq_decode_step_host(*self._fixed, self._hin + i * self._hin_stride, self._din, self._lens + i * self._lens_stride,
                                      self._lens + (i + 1) * self._lens_stride, *self._tail)
        if rc != 0:
            raise IQError(rc, "iq_decode_step_host")


def iq_rotated_histogram(shape: Shape, rot_dev, x, n_rows_dev, hist_dev, rng_half: float, stream=None) -> None:
    """Adds the histogram of the rotated, normalised coordinates of the rows x (fp16 device tensor [B][T][H_kv][d]) to
    hist_dev (uint32/int32 device tensor [bins]); n_rows_dev: int32 [B] or None (all T rows)."""
    assert x.dtype == torch.float16 and x.stride(3) == 1 and hist_dev.dtype in (torch.int32, torch.uint32)
    cs = shape.c()
    _check(_lib.iq_rotated_histogram(ctypes.byref(cs), _ptr(rot_dev), _ptr(x), x.stride(0), x.stride(1), x.stride(2),
                                     _ptr(n_rows_dev), x.shape[1], _ptr(hist_dev), hist_dev.numel(), float(rng_half),
                                     _stream(stream)), "iq_rotated_histogram")


def iq_fit_codebook(hist_host, rng_half: float, symmetric: bool = True, grid: str = "int8", bits: int = 3) -> Codebook:
    """Lloyd-Max codebook fitted to a histogram from iq_rotated_histogram (a contiguous int32/uint32 numpy array or CPU
    tensor). grid: "int8" (integer tensor-core decode path) or "fp16" (exact binary16 levels)."""
    h = hist_host.numpy() if isinstance(hist_host, torch.Tensor) else hist_host
    assert h.dtype.itemsize == 4 and h.dtype.kind in "iu" and h.flags["C_CONTIGUOUS"]
    cb = _IqCodebook()
    _check(_lib.iq_fit_codebook(h.ctypes.data, h.size, float(rng_half), bits, 1 if symmetric else 0, {"fp16": 0, "int8": 1}[grid],
                                ctypes.byref(cb)), "iq_fit_codebook")
    return _from_c(cb)


def iq_suggest_splits(shape: Shape, max_seq_len: int) -> int:
    cs = shape.c()
    return int(_lib.iq_suggest_splits(ctypes.byref(cs), max_seq_len))


def iq_wht_coordinates(shape: Shape, x, n_rows_dev, n_rows_max: int, z_out, stream=None) -> None:
    """z = sqrt(d) H x^ of the rows x [B][T][H_kv][d] (fp16) into z_out [B][n_rows_max][H_kv][d] (fp32)."""
    cs = shape.c()
    _check(_lib.iq_wht_coordinates(ctypes.byref(cs), _ptr(x), x.stride(0), x.stride(1), x.stride(2), _ptr(n_rows_dev), n_rows_max,
                                   _ptr(z_out), _stream(stream)), "iq_wht_coordinates")


def iq_fit_rotation(z_rows, head_dim: int, codebook: Codebook, quats):
    """Host fit of one KV head's SO(4) blocks: z_rows numpy fp32 [n][d] (that head's rows of iq_wht_coordinates), quats
    numpy fp32 [d/4][8] the starting rotation. Returns (fitted quats fp32 [d/4][8], distortion before, after)."""
    import numpy as np

    z = np.ascontiguousarray(z_rows, dtype=np.float32)
    q = np.ascontiguousarray(quats, dtype=np.float32).copy()
    dist = (ctypes.c_double * 2)()
    cb = codebook.c()
    _check(_lib.iq_fit_rotation(z.ctypes.data, z.shape[0], z.shape[1], head_dim, ctypes.byref(cb), q.ctypes.data,
                                ctypes.cast(dist, ctypes.c_void_p)), "iq_fit_rotation")
    return q, float(dist[0]), float(dist[1])


def iq_selftest_bounded_wait(status, polls: int, stream=None) -> None:
    _check(_lib.iq_selftest_bounded_wait(_ptr(status), int(polls), _stream(stream)), "iq_selftest_bounded_wait")


# ------------------------------------------------------------------ small conveniences (allocation only)
def new_cache(shape: Shape, device="cuda", scales_dtype=torch.float32) -> Cache:
    """scales_dtype: torch.float32, or torch.float16 for binary16 scale arrays."""
    P = iq_row_bytes(shape.head_dim, shape.bits)
    n = (shape.batch, shape.n_kv_heads, shape.t_cap)
    return Cache(torch.zeros(n + (P,), dtype=torch.uint8, device=device), torch.zeros(n, dtype=scales_dtype, device=device),
                 torch.zeros(n + (P,), dtype=torch.uint8, device=device), torch.zeros(n, dtype=scales_dtype, device=device))


def new_paged_cache(shape: Shape, num_pages: int, page_rows: int, block_table: torch.Tensor, device="cuda",
                    scales_dtype=torch.float32) -> Cache:
    """A pool of num_pages pages of page_rows rows (a multiple of 128 that divides shape.t_cap) and the block table
    (int32 device tensor [batch][t_cap / page_rows]) that maps the sequences' rows onto it."""
    assert page_rows % 128 == 0 and shape.t_cap % page_rows == 0
    assert tuple(block_table.shape) == (shape.batch, shape.t_cap // page_rows)
    P = iq_row_bytes(shape.head_dim, shape.bits)
    n = (num_pages, shape.n_kv_heads, page_rows)
    return Cache(torch.zeros(n + (P,), dtype=torch.uint8, device=device), torch.zeros(n, dtype=scales_dtype, device=device),
                 torch.zeros(n + (P,), dtype=torch.uint8, device=device), torch.zeros(n, dtype=scales_dtype, device=device),
                 block_table, page_rows)


class DecodeWorkspace:
    """Caller-owned partial buffers for a fixed shape and split count."""

    def __init__(self, shape: Shape, num_splits: int, want_argmax: bool = False, device="cuda"):
        B, H, d, S = shape.batch, shape.n_q_heads, shape.head_dim, num_splits
        self.num_splits = S
        self.part_acc = torch.empty((B, H, S, d), dtype=torch.float32, device=device)
        self.part_ml = torch.empty((B, H, S, 2), dtype=torch.float32, device=device)
        self.part_argmax = torch.empty((B, H, S), dtype=torch.int32, device=device) if want_argmax else None
        self.out = torch.empty((B, H, d), dtype=torch.float32, device=device)
        self.lse = torch.empty((B, H), dtype=torch.float32, device=device)
        self.argmax = torch.empty((B, H), dtype=torch.int32, device=device) if want_argmax else None
        self.status = torch.zeros(4, dtype=torch.int32, device=device)


def decode_step(shape: Shape, rot_dev, codebook: Codebook, q, cache: Cache, seq_lens_dev, ws: DecodeWorkspace, stream=None):
    """iq_decode_attention followed by iq_combine_splits into the workspace's output buffers."""
    iq_decode_attention(shape, rot_dev, codebook, q, cache, seq_lens_dev, ws.num_splits, ws.part_acc, ws.part_ml,
                        ws.part_argmax, ws.status, stream)
    iq_combine_splits(shape, rot_dev, ws.num_splits, ws.part_acc, ws.part_ml, ws.part_argmax, ws.out, ws.lse, ws.argmax, stream)
    return ws.out
