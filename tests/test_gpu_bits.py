"""Parity at 2 and 4 bits and with separate K and V codebooks (Algorithm 1 is written for a general bit width and
codebook; Section 3.2, Step 3): codes bit-exact against the oracle's (ties excused), attention and reconstruction within
the tolerances of the 3-bit tests."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
import workloads
from helpers import OUT_ATOL, OUT_RTOL, cache_to_numpy, check_decode, gpu_decode
from oracle import lloyd_max

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch():
    import torch as t

    if not t.cuda.is_available():
        pytest.skip("no CUDA device")
    return t


@pytest.fixture(scope="module")
def iq(torch):
    import paper_2608_08081_b200 as m

    return m


def two_codebooks(d, bits, kind, separate=True):
    """(levels_k, thresholds_k, levels_v, thresholds_v): the Lloyd-Max codebook for the K rows and, for the V rows, the
    same one stretched by 7 % (on a grid of its own for the integer path, rounded to binary16 for the fp16 path)."""
    n = 1 << bits
    lv, th = (lloyd_max.int8_codebook if kind == "int8" else lloyd_max.fp16_codebook)(d, n)
    if not separate:
        return lv, th, lv, th
    if kind == "int8":
        lvv = (lv.astype(np.float64) * 1.0703125).astype(np.float32)       # n * (delta * 1.0703125): exact in fp32
    else:
        lvv = (lv.astype(np.float64) * 1.07).astype(np.float16).astype(np.float32)
    thv = (0.5 * (lvv[1:].astype(np.float64) + lvv[:-1].astype(np.float64))).astype(np.float32)
    return lv, th, lvv, thv


def compare_codes(w, bits, th_k, th_v, g, ref, lens):
    """Every code of every valid row against the oracle's; a differing code must be a tie: the coordinate within 1e-5 of
    the threshold between the two codes. Scales equal to 1 ulp."""
    d = w.d
    total = bad = ties = 0
    for b in range(w.B):
        n = int(lens[b])
        if n == 0:
            continue
        for h in range(w.H_kv):
            R = None
            assert np.all(np.abs(g["k_scales"][b, h, :n].view(np.int32).astype(np.int64) - ref["k_scales"][b, h, :n].view(np.int32)) <= 1)
            assert np.all(np.abs(g["v_scales"][b, h, :n].view(np.int32).astype(np.int64) - ref["v_scales"][b, h, :n].view(np.int32)) <= 1)
            same_k = np.all(g["k_codes"][b, h, :n] == ref["k_codes"][b, h, :n], axis=-1)
            for t in range(n):
                total += 2 * d
                ck = None
                if not same_k[t]:
                    ck = (oracle.unpack_row(d, g["k_codes"][b, h, t], bits), oracle.unpack_row(d, ref["k_codes"][b, h, t], bits), w.k[b, t, h], th_k)
                cv_g = oracle.v_row_codes(d, g["v_codes"][b, h], t, bits)
                cv_r = oracle.v_row_codes(d, ref["v_codes"][b, h], t, bits)
                cands = [ck] if ck is not None else []
                if not np.array_equal(cv_g, cv_r):
                    cands.append((cv_g, cv_r, w.v[b, t, h], th_v))
                for cg, cr, x, th in cands:
                    if R is None:
                        R = oracle.rotation_matrix(d, w.quats[h])
                    _, _, u = oracle.quantize_row(d, R, th, x)
                    for i in np.nonzero(cg != cr)[0]:
                        lo, hi = sorted((int(cg[i]), int(cr[i])))
                        if hi - lo == 1 and abs(u[i] - float(th[lo])) < 1e-5:
                            ties += 1
                        else:
                            bad += 1
    assert bad == 0, f"{bad} code mismatches that are not ties"
    assert ties <= 1e-5 * total + 0.999, f"{ties} ties in {total} codes"
    return total, ties


def run_case(iq, torch, w, bits, kind, lens, splits, separate=True, append_in_pieces=False):
    lv_k, th_k, lv_v, th_v = two_codebooks(w.d, bits, kind, separate)
    cb = iq.Codebook(tuple(map(float, lv_k)), tuple(map(float, th_k)), tuple(map(float, lv_v)) if separate else None,
                     tuple(map(float, th_v)) if separate else None)
    assert cb.bits == bits
    lens = np.asarray(lens, np.int32)
    shape = iq.Shape(w.B, w.H_q, w.H_kv, w.d, w.t_cap, bits=bits)
    rot = torch.empty(iq.iq_rotation_floats(w.d, w.H_kv), dtype=torch.float32, device="cuda")
    iq.iq_make_rotation(w.d, w.H_kv, 0, np.ascontiguousarray(w.quats), rot)
    cache = iq.new_cache(shape)
    assert cache.k_codes.shape[-1] == bits * w.d // 8
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    k, v = torch.from_numpy(w.k).cuda(), torch.from_numpy(w.v).cuda()
    ref = oracle.new_cache(w.B, w.H_kv, w.d, w.t_cap, bits)
    if append_in_pieces:   # three calls that start and end inside 128-row blocks, the last ones a few rows each
        done = np.zeros(w.B, np.int32)
        for piece in (np.minimum(lens, 100), np.maximum(lens - 103, 0), np.full(w.B, 3, np.int32)):
            nn = np.minimum(piece, lens - done).astype(np.int32)
            T = int(nn.max()) if nn.size else 0
            if T == 0:
                continue
            idx = np.minimum(done[:, None] + np.arange(T)[None, :], w.k.shape[1] - 1)
            kk = np.ascontiguousarray(np.take_along_axis(w.k, idx[:, :, None, None], axis=1))
            vv = np.ascontiguousarray(np.take_along_axis(w.v, idx[:, :, None, None], axis=1))
            iq.iq_quantize_append(shape, rot, cb, torch.from_numpy(kk).cuda(), torch.from_numpy(vv).cuda(), torch.from_numpy(done).cuda(),
                                  torch.from_numpy(nn).cuda(), T, cache, status)
            oracle.quantize_append(w.quats, th_k, kk, vv, done.copy(), nn, ref, thresholds_v=th_v)
            done = done + nn
        assert np.array_equal(done, lens)
    else:
        iq.iq_quantize_append(shape, rot, cb, k, v, torch.zeros(w.B, dtype=torch.int32, device="cuda"), torch.from_numpy(lens).cuda(),
                              k.shape[1], cache, status)
        oracle.quantize_append(w.quats, th_k, w.k, w.v, np.zeros(w.B, np.int32), lens, ref, thresholds_v=th_v)
    torch.cuda.synchronize()
    st = status.cpu().numpy()
    assert st[0] == 0 and st[2] == 0, st
    g = cache_to_numpy(cache)
    stats = dict(codes=compare_codes(w, bits, th_k, th_v, g, ref, lens))
    for S in splits:
        res = gpu_decode(iq, torch, shape, rot, cb, w.q, cache, lens, S)
        c = check_decode(w, lv_k, w.q, res, g, lens, levels_v=lv_v)
        stats[f"S{S}"] = (c["max_err"], c["margin"], c["argmax_exact"], c["argmax_ties"])
    # reconstruct-then-compute reads the same cache
    T = int(lens.max())
    if T > 0:
        ko = torch.zeros((w.B, T, w.H_kv, w.d), dtype=torch.float16, device="cuda")
        vo = torch.zeros_like(ko)
        iq.iq_reconstruct_rows(shape, rot, cb, cache, torch.from_numpy(lens).cuda(), ko, vo)
        torch.cuda.synchronize()
        K, V = oracle.reconstruct_rows(w.quats, lv_k, g, lens, w.H_kv, levels_v=lv_v, d=w.d)
        for b in range(w.B):
            n = int(lens[b])
            if n == 0:
                continue
            for got, want in ((ko, K), (vo, V)):
                a = got[b, :n].cpu().numpy().astype(np.float64)
                r = want[b, :n]
                assert np.all(np.abs(a - r) <= 1e-3 * np.abs(r) + 1e-3 * np.max(np.abs(r)) + 1e-6)
    return stats


@pytest.mark.parametrize("kind", ["int8", "fp16"])
@pytest.mark.parametrize("d", [128, 256])
@pytest.mark.parametrize("bits", [2, 4])
def test_other_bit_widths_with_two_codebooks(iq, torch, bits, d, kind):
    lens = [0, 1, 127, 128, 129, 300, 517, 64]
    w = workloads.tiny(800 + bits, 8, 8 if d == 128 else 4, 2, d, 517, lens=lens)
    print(run_case(iq, torch, w, bits, kind, lens, [1, 3, 8, 20]))


@pytest.mark.parametrize("kind", ["int8", "fp16"])
@pytest.mark.parametrize("bits", [2, 3, 4])
def test_appends_in_pieces_and_one_codebook(iq, torch, bits, kind):
    lens = [5, 130, 259, 400]
    w = workloads.tiny(810 + bits, 4, 4, 2, 128, 400, lens=lens)
    print(run_case(iq, torch, w, bits, kind, lens, [2, 16], separate=(bits == 3), append_in_pieces=True))


@pytest.mark.parametrize("bits", [2, 4])
def test_long_sequences_other_bit_widths(iq, torch, bits):
    lens = [4096, 3000]
    w = workloads.tiny(820 + bits, 2, 16, 2, 128, 4096, lens=lens)
    shape = iq.Shape(2, 16, 2, 128, w.t_cap, bits=bits)
    print(run_case(iq, torch, w, bits, "int8", lens, [iq.iq_suggest_splits(shape, 4096), 5]))


def test_three_bits_with_two_codebooks_bulk(iq, torch):
    lens = [1000, 777, 0]
    w = workloads.tiny(830, 3, 8, 2, 256, 1000, lens=lens)
    for kind in ("int8", "fp16"):
        print(run_case(iq, torch, w, 3, kind, lens, [1, 8]))


def test_library_codebooks_match_the_oracles(iq):
    for d in (128, 256):
        for bits in (2, 3, 4):
            for kind, make in (("int8", lloyd_max.int8_codebook), ("fp16", lloyd_max.fp16_codebook)):
                cb = iq.iq_lloyd_max_codebook(d, bits, kind)
                lv, th = make(d, 1 << bits)
                assert np.allclose(cb.levels, lv, rtol=0, atol=2e-3) and np.allclose(cb.thresholds, th, rtol=0, atol=2e-3)
                assert np.all(np.diff(cb.levels) > 0)
