"""Shared helpers for the parity tests: run the CUDA path through the C-ABI binding, run the oracle on
the same seeded inputs, compare."""
from __future__ import annotations

import math

import numpy as np

import oracle

OUT_ATOL = 2e-3   # |o - o_ref| <= OUT_ATOL + OUT_RTOL * |o_ref| element-wise
OUT_RTOL = 1e-3
TIE_FRACTION_MAX = 1e-5


def codebook_for(iq, codebooks, d):
    lv, th = codebooks[d]
    return iq.Codebook(tuple(float(x) for x in lv), tuple(float(x) for x in th))


def gpu_quantize(iq, torch, w, cb, t_cap=None, append_pos=None, n_new=None, cache=None, status=None):
    """Quantize-append workload rows on the GPU; returns (shape, rot_dev, cache, status tensor)."""
    dev = "cuda"
    t_cap = t_cap or w.t_cap
    shape = iq.Shape(w.B, w.H_q, w.H_kv, w.d, t_cap)
    rot = torch.empty(iq.iq_rotation_floats(w.d, w.H_kv), dtype=torch.float32, device=dev)
    iq.iq_make_rotation(w.d, w.H_kv, 0, np.ascontiguousarray(w.quats), rot)
    cache = cache or iq.new_cache(shape)
    status = status if status is not None else torch.zeros(4, dtype=torch.int32, device=dev)
    k = torch.from_numpy(w.k).to(dev)
    v = torch.from_numpy(w.v).to(dev)
    pos = torch.from_numpy(np.asarray(append_pos if append_pos is not None else np.zeros(w.B), np.int32)).to(dev)
    nn = None if n_new is None else torch.from_numpy(np.asarray(n_new, np.int32)).to(dev)
    iq.iq_quantize_append(shape, rot, cb, k, v, pos, nn, k.shape[1], cache, status)
    torch.cuda.synchronize()
    return shape, rot, cache, status


def cache_to_numpy(cache):
    return dict(k_codes=cache.k_codes.cpu().numpy(), k_scales=cache.k_scales.cpu().numpy(),
                v_codes=cache.v_codes.cpu().numpy(), v_scales=cache.v_scales.cpu().numpy())


def oracle_quantize(w, th, t_cap=None, append_pos=None, n_new=None):
    cache = oracle.new_cache(w.B, w.H_kv, w.d, t_cap or w.t_cap)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.asarray(append_pos if append_pos is not None else np.zeros(w.B), np.int32),
                           n_new, cache)
    return cache


def ulp_diff_f32(a, b):
    ai = a.view(np.int32).astype(np.int64)
    bi = b.view(np.int32).astype(np.int64)
    return np.abs(ai - bi)


def compare_caches(w, th, gpu, ref, lens, tie_fraction_max=TIE_FRACTION_MAX):
    """Codes bit-exact except excused ties; scales equal to within 1 ulp on a vanishing fraction. Returns stats."""
    d, P = w.d, oracle.row_bytes(w.d)
    total_codes = 0
    excused = 0
    unexcused = 0
    scale_off = 0
    rows = 0
    Rs = {}
    for which, src in (("k", w.k), ("v", w.v)):
        gc, rc = gpu[which + "_codes"], ref[which + "_codes"]
        gs, rs = gpu[which + "_scales"], ref[which + "_scales"]
        for b in range(w.B):
            n = int(lens[b])
            if n == 0:
                continue
            total_codes += n * w.H_kv * d
            rows += n * w.H_kv
            ud = ulp_diff_f32(np.ascontiguousarray(gs[b, :, :n]), np.ascontiguousarray(rs[b, :, :n]))
            assert ud.max() <= 1, f"{which} scale differs by {ud.max()} ulp"
            scale_off += int((ud > 0).sum())
            if which == "k":
                row_codes = lambda arr, g, t: oracle.unpack_row(d, arr[b, g, t])
                neq = np.any(gc[b, :, :n] != rc[b, :, :n], axis=-1)
                bad = list(zip(*np.nonzero(neq)))
            else:   # token-transposed: compare whole 128-row blocks, then the rows of the blocks that differ
                row_codes = lambda arr, g, t: oracle.v_row_codes(d, arr[b, g], t)
                nb = (n + 127) // 128
                gb = gc[b].reshape(w.H_kv, -1, 128 * P)[:, :nb]
                rb = rc[b].reshape(w.H_kv, -1, 128 * P)[:, :nb]
                bad = []
                for g, j in zip(*np.nonzero(np.any(gb != rb, axis=-1))):
                    differing = 0
                    for t in range(128 * j, min(128 * j + 128, n)):
                        if not np.array_equal(row_codes(gc, g, t), row_codes(rc, g, t)):
                            bad.append((g, t))
                            differing += 1
                    # the bits of the block's rows that were never appended must be untouched (as allocated) on both sides
                    assert differing > 0, f"V block {j} of (sequence {b}, head {g}) differs only in rows that were never appended"
            for g, t in bad:
                cg = row_codes(gc, g, t).astype(np.int64)
                cr = row_codes(rc, g, t).astype(np.int64)
                if g not in Rs:
                    Rs[g] = oracle.rotation_matrix(d, w.quats[g])
                _, _, u = oracle.quantize_row(d, Rs[g], th, src[b, t, g])
                for i in np.nonzero(cg != cr)[0]:
                    tj = float(th[min(cg[i], cr[i])])          # threshold separating the two adjacent codes
                    ok = abs(int(cg[i]) - int(cr[i])) == 1 and abs(u[i] - tj) <= 2.0 ** -23 * max(1.0, abs(tj))
                    excused += int(ok)
                    unexcused += int(not ok)
    assert unexcused == 0, f"{unexcused} code mismatches that are not ties"
    assert excused <= tie_fraction_max * max(total_codes, 1) + 0.999, f"{excused} tie mismatches in {total_codes} codes"
    assert scale_off <= 1e-5 * rows + 1, f"{scale_off} scales off by 1 ulp in {rows} rows"
    return dict(total_codes=total_codes, excused=excused, scale_off=scale_off)


def gpu_decode(iq, torch, shape, rot, cb, q_np, cache, lens, num_splits, want_argmax=True):
    dev = "cuda"
    ws = iq.DecodeWorkspace(shape, num_splits, want_argmax=want_argmax)
    q = torch.from_numpy(q_np).to(dev)
    sl = torch.from_numpy(np.asarray(lens, np.int32)).to(dev)
    iq.decode_step(shape, rot, cb, q, cache, sl, ws)
    torch.cuda.synchronize()
    assert int(ws.status[0].item()) == 0, "device status flags set"
    return dict(out=ws.out.cpu().numpy().astype(np.float64), lse=ws.lse.cpu().numpy().astype(np.float64),
                argmax=None if ws.argmax is None else ws.argmax.cpu().numpy(), ws=ws)


ARGMAX_TIE_RTOL = 4e-6   # a different argmax row is a tie iff its fp64 score is within this (relative) of the maximum
ARGMAX_TIE_ATOL = 2e-6   # ... plus this: the kernel's scores are fp32 values of 21-bit (integer path) or 22-bit (fp16 path) queries


def check_decode(w, lv, q_np, gpu_res, cache_np, lens, sm_scale=0.0, argmax_tol=None, levels_v=None):
    """Outputs within tolerance of the fp64 oracle run on the same packed cache; argmax identical, except that a row
    whose fp64 score ties with the maximum within the rounding of the kernel's fp32 scores is accepted (counted, and
    at most 2 % of the heads + 1)."""
    ref = oracle.decode_attention(w.quats, lv, q_np, cache_np, lens, w.H_kv, sm_scale, levels_v=levels_v)
    err = np.abs(gpu_res["out"] - ref["out"])
    bound = OUT_ATOL + OUT_RTOL * np.abs(ref["out"])
    assert np.all(err <= bound), f"max err {err.max():.3e} (worst excess {np.max(err - bound):.3e})"
    nz = np.asarray(lens) > 0
    if nz.any():
        num = np.linalg.norm((gpu_res["out"] - ref["out"])[nz], axis=-1)
        den = np.linalg.norm(ref["out"][nz], axis=-1)
        assert np.all(num <= OUT_RTOL * den + 1e-6), f"relative l2 error {np.max(num / np.maximum(den, 1e-30)):.3e}"
        assert np.allclose(gpu_res["lse"][nz], ref["lse"][nz], atol=2e-3, rtol=1e-5)   # fp32 scores: relative at large |z|
    assert np.all(np.isneginf(gpu_res["lse"][~nz])) and np.all(gpu_res["out"][~nz] == 0)
    exact = ties = 0
    if gpu_res["argmax"] is not None:
        B, H_q = ref["argmax"].shape
        for b in range(B):
            for h in range(H_q):
                ga, ra = int(gpu_res["argmax"][b, h]), int(ref["argmax"][b, h])
                if ga == ra:
                    exact += 1
                    continue
                assert lens[b] > 0 and 0 <= ga < lens[b], f"argmax {ga} outside the sequence"
                z = oracle.scores(w.quats, lv, q_np, cache_np, b, h, int(lens[b]), w.H_kv, sm_scale)
                tol = argmax_tol if argmax_tol is not None else ARGMAX_TIE_ATOL + ARGMAX_TIE_RTOL * abs(z[ra])
                assert z[ra] - z[ga] <= tol, f"argmax differs: gpu row {ga} scores {z[ga]}, oracle row {ra} scores {z[ra]}"
                ties += 1
        assert ties <= 0.02 * B * H_q + 1, f"{ties} argmax ties in {B * H_q} heads"
    return dict(max_err=float(err.max()), margin=float(np.max(err / bound)), argmax_exact=exact, argmax_ties=ties, ref=ref)
