"""GPU-vs-oracle parity through the C ABI: packed codes bit-exact (ties excused and counted), attention
outputs within 2e-3 + 1e-3 |ref| of the fp64 oracle run on the same packed cache, argmax identical."""
import math
import os

import numpy as np
import pytest

import oracle
import workloads
from helpers import (cache_to_numpy, check_decode, codebook_for, compare_caches, gpu_decode, gpu_quantize,
                     oracle_quantize)

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


def _roundtrip(iq, torch, codebooks, w, splits_list, n_new=None, t_cap=None, tie_fraction_max=1e-5):
    lv, th = codebooks[w.d]
    cb = codebook_for(iq, codebooks, w.d)
    lens = w.seq_lens if n_new is None else np.asarray(n_new, np.int32)
    shape, rot, cache, status = gpu_quantize(iq, torch, w, cb, t_cap=t_cap, n_new=n_new if n_new is not None else w.seq_lens)
    st = status.cpu().numpy()
    assert st[0] == 0 and st[2] == 0
    g = cache_to_numpy(cache)
    ref = oracle_quantize(w, th, t_cap=t_cap, n_new=lens)
    stats = compare_caches(w, th, g, ref, lens, tie_fraction_max)
    stats["rechecked_rows"] = int(st[1])
    for S in splits_list:
        res = gpu_decode(iq, torch, shape, rot, cb, w.q, cache, lens, S)
        c = check_decode(w, lv, w.q, res, g, lens)
        stats[f"S{S}"] = (c["max_err"], c["margin"])
    return stats


def test_config1_tiny_decode(iq, torch, codebooks):
    w = workloads.config1()
    stats = _roundtrip(iq, torch, codebooks, w, [1, 2, 3, 16])
    assert stats["total_codes"] == 2 * 1024 * 128
    print(stats)


@pytest.mark.parametrize("d", [128, 256])
@pytest.mark.parametrize("T", [1, 2, 31, 32, 33, 63, 64, 65, 127, 128, 129, 1000])
def test_shape_sweep_context_lengths(iq, torch, codebooks, d, T):
    w = workloads.tiny(100 + T, 1, 8 if d == 128 else 4, 2, d, T, lens=[T])
    print(_roundtrip(iq, torch, codebooks, w, [1, 3], n_new=[T]))


@pytest.mark.parametrize("G", [1, 2, 4, 8, 16])
def test_shape_sweep_group_sizes(iq, torch, codebooks, G):
    w = workloads.tiny(200 + G, 2, 2 * G, 2, 128, 300, lens=[300, 123])
    print(_roundtrip(iq, torch, codebooks, w, [1, 4], n_new=[300, 123]))


def test_ragged_batch_with_empty_and_full_sequences(iq, torch, codebooks):
    lens = [0, 1, 64, 257, 512, 100, 0, 511]
    w = workloads.tiny(300, 8, 8, 2, 128, 512, lens=lens)
    _roundtrip(iq, torch, codebooks, w, [1, 2, 5, 9], n_new=lens)


def test_more_sequences_than_sms_and_than_threads(iq, torch, codebooks):
    # the decode kernel gives every SM a range of the batch's 128-row blocks: here there are more sequences than CTAs
    # and than threads of a CTA (each thread then sums several sequences for the range boundaries), many of them empty
    B = 700
    g = np.random.Generator(np.random.Philox(77))
    lens = g.integers(0, 300, B).astype(np.int64)
    lens[g.integers(0, B, 60)] = 0
    lens[5] = 300
    w = workloads.tiny(302, B, 4, 2, 128, 300, lens=[int(x) for x in lens])
    _roundtrip(iq, torch, codebooks, w, [1, 2, 3], n_new=[int(x) for x in lens])


def test_few_slots_for_a_long_sequence_next_to_short_ones(iq, torch, codebooks):
    # with S = 2 an item may span at most two ranges, which forces ranges longer than an equal share of the blocks;
    # with S = 7 the long sequence is cut into many pieces and the short ones share ranges with it
    lens = [5000, 17, 0, 129, 2300]
    w = workloads.tiny(303, 5, 16, 2, 128, 5000, lens=lens)
    _roundtrip(iq, torch, codebooks, w, [2, 7, 40], n_new=lens)


def test_dominant_row_over_a_long_tail_of_equal_values(iq, torch, codebooks):
    """One key far above a long flat tail whose total probability mass still matters, and value rows that all point the
    same way: every small probability adds with the same sign, so a path that rounds them away (fixed-point or
    half-precision probabilities) shows a bias here; and the flat tail makes the lazily raised softmax reference and
    the in-TMEM accumulation run over many blocks without a raise."""
    T, d = 12000, 128
    w = workloads.tiny(320, 1, 8, 1, d, T)
    g = np.random.Generator(np.random.Philox(321))
    w.k[:] = workloads.to_fp16(0.02 * g.standard_normal(w.k.shape))                 # flat scores near 0
    base = g.standard_normal(d)
    w.v[:] = workloads.to_fp16(base[None, None, None, :] * (1 + 0.01 * g.standard_normal((1, T, 1, 1))))
    for h in range(8):                                                              # the needle of head h: z ~ 11 nats above the tail
        w.k[0, 1000 + 997 * h, 0] = workloads.to_fp16(11.0 * np.sqrt(d) * w.q[0, h].astype(np.float64) / np.dot(w.q[0, h].astype(np.float64), w.q[0, h].astype(np.float64)))
    stats = _roundtrip(iq, torch, codebooks, w, [1, 2, 9])
    print(stats)


def test_large_scale_rows_and_zero_rows(iq, torch, codebooks):
    w = workloads.tiny(301, 1, 4, 1, 128, 256, scale=300.0)
    w.k[0, 5] = 0
    w.v[0, 7] = 0
    w.k[0, 9] = np.float16(60000.0)   # a constant row rotates onto a multiple of e_0: 127 coordinates sit EXACTLY on the
    w.v[0, 11, 0, :3] = np.float16(-65504.0)  # threshold 0 -- genuine ties, so only "every mismatch is a tie" is asserted here
    print(_roundtrip(iq, torch, codebooks, w, [1, 2], tie_fraction_max=1e-2))


def test_append_positions_strides_and_out_of_range_rows(iq, torch, codebooks):
    """Append in two calls at non-zero positions (not multiples of 32), from a strided source; rows beyond t_cap
    are skipped and flagged."""
    d, T = 128, 160
    lv, th = codebooks[d]
    cb = codebook_for(iq, codebooks, d)
    w = workloads.tiny(302, 2, 4, 2, d, T)
    shape = iq.Shape(2, 4, 2, d, 128)
    rot = torch.empty(iq.iq_rotation_floats(d, 2), dtype=torch.float32, device="cuda")
    iq.iq_make_rotation(d, 2, 0, np.ascontiguousarray(w.quats), rot)
    cache = iq.new_cache(shape)
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    big_k = torch.zeros((2, T, 2, 2 * d), dtype=torch.float16, device="cuda")      # strided view: every other 128-slab
    big_v = torch.zeros_like(big_k)
    big_k[..., :d] = torch.from_numpy(w.k).cuda()
    big_v[..., :d] = torch.from_numpy(w.v).cuda()
    kview, vview = big_k[..., :d], big_v[..., :d]
    pos0 = torch.zeros(2, dtype=torch.int32, device="cuda")
    n0 = torch.tensor([40, 17], dtype=torch.int32, device="cuda")
    iq.iq_quantize_append(shape, rot, cb, kview[:, :40], vview[:, :40], pos0, n0, 40, cache, status)
    pos1 = n0.clone()
    n1 = torch.tensor([104, 30], dtype=torch.int32, device="cuda")                 # sequence 0: rows 128..143 fall outside t_cap = 128
    k2 = torch.stack([kview[0, 40:144], kview[1, 17:121]])
    v2 = torch.stack([vview[0, 40:144], vview[1, 17:121]])
    iq.iq_quantize_append(shape, rot, cb, k2, v2, pos1, n1, 104, cache, status)
    torch.cuda.synchronize()
    st = status.cpu().numpy()
    assert st[0] & 1 and st[2] == 16 * 2 * 2                                        # 16 rows x 2 KV heads x (K, V)
    g = cache_to_numpy(cache)
    lens = np.array([128, 47], np.int32)
    ref = oracle.new_cache(2, 2, d, 128)
    wk = np.zeros((2, 128, 2, d), np.float16); wv = np.zeros_like(wk)
    wk[0], wv[0] = w.k[0, :128], w.v[0, :128]
    wk[1, :47], wv[1, :47] = w.k[1, :47], w.v[1, :47]
    oracle.quantize_append(w.quats, th, wk, wv, np.zeros(2, np.int32), lens, ref)
    w2 = workloads.Workload("x", 2, 4, 2, d, 128, wk, wv, w.q, w.quats, lens)
    compare_caches(w2, th, g, ref, lens)
    assert np.array_equal(g["v_codes"], ref["v_codes"])                             # incl. rows never appended (stay zero)
    res = gpu_decode(iq, torch, shape, rot, cb, w.q, cache, lens, 2)
    check_decode(w2, lv, w.q, res, g, lens)


@pytest.mark.parametrize("d", [128, 256])
def test_small_appends_take_the_same_codes_as_one_bulk_append(iq, torch, codebooks, d):
    """Calls with a few new rows per sequence (the decode-step path: one warp per row, V written by read-modify-write
    into the transposed records) must leave exactly the cache a single bulk append leaves, at every row-in-unit
    position, with ragged per-sequence counts and rows beyond t_cap skipped and flagged."""
    T, t_cap = 140, 128
    lv, th = codebooks[d]
    cb = codebook_for(iq, codebooks, d)
    w = workloads.tiny(310 + d, 3, 4, 2, d, T)
    shape = iq.Shape(3, 4, 2, d, t_cap)
    rot = torch.empty(iq.iq_rotation_floats(d, 2), dtype=torch.float32, device="cuda")
    iq.iq_make_rotation(d, 2, 0, np.ascontiguousarray(w.quats), rot)
    cache = iq.new_cache(shape)
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    k, v = torch.from_numpy(w.k).cuda(), torch.from_numpy(w.v).cuda()
    pos = np.zeros(3, np.int64)
    total = np.array([T, 75, 0])                       # sequence 0 runs 12 rows past t_cap, sequence 2 never appends
    step = 0
    while (pos < total).any():
        nmax = 1 + step % 4                            # 1..4 rows per call
        n = np.minimum(nmax, total - pos).astype(np.int32)
        idx = (pos[:, None] + np.arange(nmax)[None, :]).clip(max=T - 1)
        kk = torch.stack([k[b, idx[b]] for b in range(3)])
        vv = torch.stack([v[b, idx[b]] for b in range(3)])
        iq.iq_quantize_append(shape, rot, cb, kk, vv, torch.from_numpy(pos.astype(np.int32)).cuda(),
                              torch.from_numpy(n).cuda(), nmax, cache, status)
        pos += n
        step += 1
    torch.cuda.synchronize()
    st = status.cpu().numpy()
    assert st[0] & 1 and st[2] == 12 * 2 * 2           # 12 rows x 2 KV heads x (K, V) beyond t_cap
    g = cache_to_numpy(cache)
    lens = np.array([t_cap, 75, 0], np.int32)
    ref = oracle.new_cache(3, 2, d, t_cap)
    oracle.quantize_append(w.quats, th, w.k[:, :t_cap], w.v[:, :t_cap], np.zeros(3, np.int32), lens, ref)
    w2 = workloads.Workload("x", 3, 4, 2, d, t_cap, w.k[:, :t_cap], w.v[:, :t_cap], w.q, w.quats, lens)
    compare_caches(w2, th, g, ref, lens)


@pytest.mark.parametrize("d", [128, 256])
def test_reconstructed_rows_match_the_oracle(iq, torch, codebooks, d):
    """iq_reconstruct_rows (the reconstruct-then-compute model's first half) against the oracle's dense R^T per row:
    fp32 arithmetic and one rounding to binary16. Ragged lengths with an empty sequence, a partial last block, an
    output shorter than the longest sequence, K and V interleaved in one strided buffer; rows that must not be
    written keep their sentinel."""
    B, H_q, H_kv, T, T_out = 3, 4, 2, 300, 256
    lens = np.array([300, 129, 0], np.int32)
    lv, th = codebooks[d]
    cb = codebook_for(iq, codebooks, d)
    w = workloads.tiny(500 + d, B, H_q, H_kv, d, T, lens)
    shape, rot, cache, status = gpu_quantize(iq, torch, w, cb, n_new=lens)
    kv = torch.full((B, T_out, H_kv, 2 * d), 7.0, dtype=torch.float16, device="cuda")
    k_out, v_out = kv[..., :d], kv[..., d:]
    iq.iq_reconstruct_rows(shape, rot, cb, cache, torch.from_numpy(lens).cuda(), k_out, v_out)
    torch.cuda.synchronize()
    K, V = oracle.reconstruct_rows(w.quats, lv, cache_to_numpy(cache), lens, H_kv)
    for got, ref in ((k_out.cpu().numpy().astype(np.float64), K), (v_out.cpu().numpy().astype(np.float64), V)):
        for b in range(B):
            n = min(int(lens[b]), T_out)
            assert np.all(got[b, n:] == 7.0)
            if n == 0:
                continue
            r = ref[b, :n]
            bound = 2.0 ** -11 * 1.001 * np.abs(r) + 1e-5 * np.abs(r).max(axis=-1, keepdims=True)   # fp16 rounding + fp32 sums
            assert np.all(np.abs(got[b, :n] - r) <= bound), float(np.max(np.abs(got[b, :n] - r) / bound))
            x = (w.k if ref is K else w.v)[b, :n].astype(np.float64)
            rel = np.sum((x - got[b, :n]) ** 2, axis=-1) / np.sum(x * x, axis=-1)
            assert 0.025 < float(rel.mean()) < 0.045                                  # the codebook's distortion, end to end


@pytest.mark.parametrize("d", [128, 256])
def test_codebook_that_is_not_symmetric_takes_the_same_codes(iq, torch, codebooks, d):
    """The bulk kernels decide with two compares on |u| when the thresholds are symmetric about zero and with a
    three-step search otherwise: shifted thresholds must still give the oracle's codes, in the bulk kernels (300
    rows at once, a partly filled last block) and in the few-rows kernel (3 more rows)."""
    lv, th = codebooks[d]
    th2 = (np.asarray(th, np.float64) + np.array([0.013, -0.02, 0.007, 0.011, 0.0, -0.017, 0.02])).astype(np.float32)
    assert np.all(np.diff(th2) > 0) and th2[3] != 0
    cb = iq.Codebook(tuple(float(x) for x in lv), tuple(float(x) for x in th2))
    T = 303
    w = workloads.tiny(900 + d, 2, 4, 2, d, T)
    lens = np.array([300, 170], np.int32)
    shape, rot, cache, status = gpu_quantize(iq, torch, w, cb, n_new=lens)
    k, v = torch.from_numpy(w.k).cuda(), torch.from_numpy(w.v).cuda()
    idx = (lens[:, None] + np.arange(3)[None, :]).clip(max=T - 1)
    kk = torch.stack([k[b, idx[b]] for b in range(2)])
    vv = torch.stack([v[b, idx[b]] for b in range(2)])
    iq.iq_quantize_append(shape, rot, cb, kk, vv, torch.from_numpy(lens).cuda(), None, 3, cache, status)
    torch.cuda.synchronize()
    lens2 = lens + 3
    ref = oracle.new_cache(2, 2, d, w.t_cap)
    oracle.quantize_append(w.quats, th2, w.k, w.v, np.zeros(2, np.int32), lens, ref)
    oracle.quantize_append(w.quats, th2, kk.cpu().numpy(), vv.cpu().numpy(), lens, None, ref)
    full_k = np.zeros_like(w.k); full_v = np.zeros_like(w.v)
    for b in range(2):
        full_k[b, :lens[b]] = w.k[b, :lens[b]]; full_v[b, :lens[b]] = w.v[b, :lens[b]]
        full_k[b, lens[b]:lens2[b]] = w.k[b, idx[b]]; full_v[b, lens[b]:lens2[b]] = w.v[b, idx[b]]
    w2 = workloads.Workload("asym", 2, 4, 2, d, w.t_cap, full_k, full_v, w.q, w.quats, lens2)
    print(compare_caches(w2, th2, cache_to_numpy(cache), ref, lens2))
    assert status.cpu().numpy()[0] == 0


@pytest.mark.parametrize("out_dtype", ["float32", "float16"])
def test_decode_step_from_host_buffers(iq, torch, codebooks, out_dtype):
    """iq_decode_step_host (copy in, append one row per sequence, decode, combine, copy out, wait) against the oracle:
    the appended rows and the attention output, over three steps with ragged lengths and an empty sequence."""
    d, B, H_q, H_kv, T0, steps = 128, 3, 8, 2, 200, 3
    lv, th = codebooks[d]
    cb = codebook_for(iq, codebooks, d)
    w = workloads.tiny(61, B, H_q, H_kv, d, T0 + steps)
    lens0 = np.array([T0, 127, 0], np.int32)
    t_cap = workloads.cap128(T0 + steps)
    shape = iq.Shape(B, H_q, H_kv, d, t_cap)
    rot = torch.empty(iq.iq_rotation_floats(d, H_kv), dtype=torch.float32, device="cuda")
    iq.iq_make_rotation(d, H_kv, 0, np.ascontiguousarray(w.quats), rot)
    cache, status = iq.new_cache(shape), torch.zeros(4, dtype=torch.int32, device="cuda")
    iq.iq_quantize_append(shape, rot, cb, torch.from_numpy(w.k[:, :T0]).cuda(), torch.from_numpy(w.v[:, :T0]).cuda(),
                          torch.zeros(B, dtype=torch.int32, device="cuda"), torch.from_numpy(lens0).cuda(), T0, cache, status)
    ref = oracle.new_cache(B, H_kv, d, t_cap)
    oracle.quantize_append(w.quats, th, w.k[:, :T0], w.v[:, :T0], np.zeros(B, np.int32), lens0, ref)
    ws = iq.DecodeWorkspace(shape, iq.iq_suggest_splits(shape, t_cap))
    dt = getattr(torch, out_dtype)
    n_in = B * (H_q + 2 * H_kv) * d
    h_in = torch.empty(n_in, dtype=torch.float16).pin_memory()
    d_in = torch.empty(n_in, dtype=torch.float16, device="cuda")
    out_dev = torch.empty((B, H_q, d), dtype=dt, device="cuda")
    out_host = torch.full((B, H_q, d), 99.0, dtype=dt).pin_memory()
    g = np.random.default_rng(9)
    rows = lens0.astype(np.int64).copy()
    for i in range(steps):
        kn = np.stack([w.k[b, rows[b]] for b in range(B)])[:, None]
        vn = np.stack([w.v[b, rows[b]] for b in range(B)])[:, None]
        qn = workloads.to_fp16(g.standard_normal((B, H_q, d)))
        h_in.copy_(torch.from_numpy(np.concatenate([qn.reshape(-1), kn.reshape(-1), vn.reshape(-1)])))
        pos = torch.from_numpy(rows.astype(np.int32)).cuda()
        after = torch.from_numpy((rows + 1).astype(np.int32)).cuda()
        iq.iq_decode_step_host(shape, rot, cb, h_in, d_in, pos, after, cache, ws, out_dev, out_host)
        # the call has waited for the output: no synchronize here
        got = out_host.numpy().astype(np.float64).copy()
        oracle.quantize_append(w.quats, th, kn, vn, rows.astype(np.int32), None, ref)
        rows += 1
        now = rows.astype(np.int32)
        r = oracle.decode_attention(w.quats, lv, qn, cache_to_numpy(cache), now, H_kv)
        tol = 2e-3 + 1e-3 * np.abs(r["out"]) + (2.0 ** -11 * np.abs(r["out"]) if out_dtype == "float16" else 0)
        assert np.all(np.abs(got - r["out"]) <= tol), float(np.max(np.abs(got - r["out"])))
    w2 = workloads.Workload("h", B, H_q, H_kv, d, t_cap, w.k, w.v, w.q, w.quats, rows.astype(np.int32))
    compare_caches(w2, th, cache_to_numpy(cache), ref, w2.seq_lens)
    # two more steps through the stepper that marshals every argument once (rows of one pinned tensor, one length table)
    more = 2
    h_all = torch.empty((more, n_in), dtype=torch.float16).pin_memory()
    tab = torch.from_numpy(np.stack([rows + j for j in range(more + 1)]).astype(np.int32)).cuda()
    qs, kns, vns = [], [], []
    for j in range(more):
        kn = np.stack([w.k[b, min(rows[b] + j, w.k.shape[1] - 1)] for b in range(B)])[:, None]
        vn = np.stack([w.v[b, min(rows[b] + j, w.k.shape[1] - 1)] for b in range(B)])[:, None]
        qn = workloads.to_fp16(g.standard_normal((B, H_q, d)))
        h_all[j].copy_(torch.from_numpy(np.concatenate([qn.reshape(-1), kn.reshape(-1), vn.reshape(-1)])))
        qs.append(qn); kns.append(kn); vns.append(vn)
    stepper = iq.HostStepper(shape, rot, cb, h_all, d_in, tab, cache, ws, out_dev, out_host)
    assert stepper.n_steps == more
    for j in range(more):
        stepper.step(j)
        got = out_host.numpy().astype(np.float64).copy()
        oracle.quantize_append(w.quats, th, kns[j], vns[j], rows.astype(np.int32), None, ref)
        rows += 1
        r = oracle.decode_attention(w.quats, lv, qs[j], cache_to_numpy(cache), rows.astype(np.int32), H_kv)
        tol = 2e-3 + 1e-3 * np.abs(r["out"]) + (2.0 ** -11 * np.abs(r["out"]) if out_dtype == "float16" else 0)
        assert np.all(np.abs(got - r["out"]) <= tol), float(np.max(np.abs(got - r["out"])))
    for b in range(B):
        assert np.array_equal(cache_to_numpy(cache)["k_codes"][b, :, :rows[b]], ref["k_codes"][b, :, :rows[b]])
    assert status.cpu().numpy()[0] == 0 and ws.status.cpu().numpy()[0] == 0


@pytest.mark.parametrize("d", [128, 256])
def test_calibration_histogram_and_fitted_codebook(iq, torch, d):
    """iq_rotated_histogram against the oracle's dense-rotation histogram on heavy-tailed rows (ragged row counts, a
    zero row, values beyond the range): the counts may differ only where fp32 puts a value on the other side of a bin
    edge (a vanishing fraction, neighbouring bins), the codebooks fitted to the two histograms agree, and a
    quantize + decode round trip with the fitted codebook is parity-exact and beats the default codebook's distortion."""
    from oracle import lloyd_max
    B, H_q, H_kv, T = 2, 4, 2, 700
    g = np.random.Generator(np.random.Philox(4100 + d))
    x = workloads.to_fp16(0.5 * g.standard_t(3.0, (B, T, H_kv, d)))
    x[0, 5] = 0
    n_rows = np.array([T, 333], np.int32)
    quats = workloads.quaternion_pairs(g, H_kv, d)
    bins, R = 2048, 6.0
    shape = iq.Shape(B, H_q, H_kv, d, workloads.cap128(T))
    rot = torch.empty(iq.iq_rotation_floats(d, H_kv), dtype=torch.float32, device="cuda")
    iq.iq_make_rotation(d, H_kv, 0, np.ascontiguousarray(quats), rot)
    hist = torch.zeros(bins, dtype=torch.int32, device="cuda")
    xd = torch.from_numpy(x).cuda()
    iq.iq_rotated_histogram(shape, rot, xd, torch.from_numpy(n_rows).cuda(), hist, R)
    torch.cuda.synchronize()
    got = hist.cpu().numpy().astype(np.int64)
    ref = lloyd_max.rotated_histogram(quats, x[0], bins, R) + lloyd_max.rotated_histogram(quats, x[1, :333], bins, R)
    assert got.sum() == ref.sum() == (T - 1 + 333) * H_kv * d
    moved = np.abs(np.cumsum(got - ref))                     # a value in the neighbouring bin shows as +1 / -1 next to each other
    assert moved.max() <= 3 and np.abs(got - ref).sum() <= 2e-4 * ref.sum()
    hist2 = torch.zeros(64, dtype=torch.int32, device="cuda")   # a narrow range: what falls outside is counted in the end bins
    iq.iq_rotated_histogram(shape, rot, xd, torch.from_numpy(n_rows).cuda(), hist2, 2.0)
    got2 = hist2.cpu().numpy().astype(np.int64)
    ref2 = lloyd_max.rotated_histogram(quats, x[0], 64, 2.0) + lloyd_max.rotated_histogram(quats, x[1, :333], 64, 2.0)
    assert got2.sum() == ref2.sum() and np.abs(np.cumsum(got2 - ref2)).max() <= 3
    assert got2[0] > 50 * got2[1] / 10 and got2[-1] > 50 * got2[-2] / 10
    for grid in ("int8", "fp16"):
        cb_g = iq.iq_fit_codebook(got.astype(np.uint32), R, grid=grid)
        cb_r = iq.iq_fit_codebook(ref.astype(np.uint32), R, grid=grid)
        assert np.allclose(cb_g.levels, cb_r.levels, atol=2e-3)
    # round trip with the fitted codebook (levels on the 8-bit grid): parity against the oracle, and a lower distortion
    cb = iq.iq_fit_codebook(got.astype(np.uint32), R, grid="int8")
    lv, th = np.array(cb.levels, np.float32), np.array(cb.thresholds, np.float32)
    w = workloads.Workload("cal", B, H_q, H_kv, d, shape.t_cap, x, x[:, ::-1].copy(), workloads.to_fp16(g.standard_normal((B, H_q, d))),
                           quats, n_rows)
    shape2, rot2, cache, status = gpu_quantize(iq, torch, w, cb, n_new=n_rows)
    cache_np = cache_to_numpy(cache)
    refc = oracle.new_cache(B, H_kv, d, shape.t_cap)
    oracle.quantize_append(quats, th, w.k, w.v, np.zeros(B, np.int32), n_rows, refc)
    compare_caches(w, th, cache_np, refc, n_rows)
    S = iq.iq_suggest_splits(shape2, T)
    res = gpu_decode(iq, torch, shape2, rot2, cb, w.q, cache, n_rows, S)
    check_decode(w, lv, w.q, res, cache_np, n_rows)
    dflt = iq.iq_int8_codebook(d)

    def distortion(levels, thresholds):
        c = oracle.new_cache(B, H_kv, d, shape.t_cap)
        oracle.quantize_append(quats, np.array(thresholds, np.float32), w.k, w.v, np.zeros(B, np.int32), n_rows, c)
        K, _ = oracle.reconstruct_rows(quats, np.array(levels, np.float32), c, n_rows, H_kv)
        xs = x[1, :333].astype(np.float64)
        return float(np.mean(np.sum((xs - K[1, :333]) ** 2, -1) / np.sum(xs * xs, -1)))

    assert distortion(cb.levels, cb.thresholds) < distortion(dflt.levels, dflt.thresholds)


def _gather_pages(cache, table, page_rows):
    """The paged pool read back as the contiguous cache [B][H_kv][t_cap] the oracle works on."""
    tb = np.asarray(table)
    out = {}
    for name in ("k_codes", "k_scales", "v_codes", "v_scales"):
        pool = getattr(cache, name).cpu().numpy()                                     # [pages][H_kv][page_rows](...)
        out[name] = np.ascontiguousarray(np.concatenate([pool[tb[:, j]] for j in range(tb.shape[1])], axis=2))
    return out


@pytest.mark.parametrize("d", [128, 256])
def test_rotation_calibration(iq, torch, codebooks, d):
    """The 'learnable' SO(4) parameters: iq_wht_coordinates (GPU) against the oracle's sqrt(d) H x^, the host fit on the
    GPU's coordinates against the oracle's fit, and the effect: rows quantised under the fitted rotation reconstruct
    with a lower error than under the rotation the fit started from, and decode stays parity-exact with it."""
    from oracle import so4_fit
    B, H_q, H_kv, T = 2, 4, 2, 640
    lv, th = codebooks[d]
    cb = codebook_for(iq, codebooks, d)
    lens = np.array([640, 500], np.int32)
    w = workloads.tiny(3100 + d, B, H_q, H_kv, d, T, lens)
    g = np.random.Generator(np.random.Philox(7 + d))
    scales = np.where(np.arange(d) % 2 == 1, 4.0, 1.0) * np.exp(0.5 * g.standard_normal(d))     # correlates neighbouring coordinates after H
    k = workloads.to_fp16(w.k.astype(np.float64) * scales)
    v = workloads.to_fp16(w.v.astype(np.float64) * scales)
    shape = iq.Shape(B, H_q, H_kv, d, workloads.cap128(T))
    kd = torch.from_numpy(k).cuda()
    z = torch.full((B, T, H_kv, d), float("nan"), dtype=torch.float32, device="cuda")
    iq.iq_wht_coordinates(shape, kd, torch.from_numpy(lens).cuda(), T, z)
    torch.cuda.synchronize()
    zc = z.cpu().numpy()
    assert np.isnan(zc[1, 500:]).all()                                                          # rows beyond a sequence's count are not written
    fitted = np.zeros_like(w.quats)
    for h in range(H_kv):
        rows = np.concatenate([zc[b, :lens[b], h] for b in range(B)])
        ref = np.concatenate([so4_fit.wht_coordinates(k[b, :lens[b], h]) for b in range(B)])
        assert np.all(np.abs(rows - ref) <= 1e-5 + 2e-6 * np.abs(ref))                          # fp32 butterfly against fp64
        q_lib, before, after = iq.iq_fit_rotation(rows, d, cb, w.quats[h])
        q_ref, b_ref, a_ref = so4_fit.fit_rotation(rows.astype(np.float64), w.quats[h], lv, th)
        assert abs(before - b_ref) < 1e-9 * b_ref and abs(after - a_ref) < 5e-3 * a_ref and after < 0.97 * before
        fitted[h] = q_lib
    # the same rows through Algorithm 1 under both rotations: reconstruction error of the K rows, and decode parity
    errs = []
    for quats in (w.quats, fitted):
        w2 = workloads.Workload("calib", B, H_q, H_kv, d, T, k, v, w.q, quats, lens)
        shape2, rot, cache, status = gpu_quantize(iq, torch, w2, cb, n_new=lens)
        gq = cache_to_numpy(cache)
        compare_caches(w2, th, gq, oracle_quantize(w2, th, n_new=lens), lens)
        K, _ = oracle.reconstruct_rows(quats, lv, gq, lens, H_kv)
        num = den = 0.0
        for b in range(B):
            xk = k[b, :lens[b]].astype(np.float64)
            num += np.sum((K[b, :lens[b]] - xk) ** 2)
            den += np.sum(xk ** 2)
        errs.append(num / den)
        res = gpu_decode(iq, torch, shape2, rot, cb, w.q, cache, lens, iq.iq_suggest_splits(shape2, T))
        check_decode(w2, lv, w.q, res, gq, lens)
    assert errs[1] < 0.98 * errs[0], errs


@pytest.mark.parametrize("d,page_rows", [(128, 128), (128, 256), (256, 128)])
def test_paged_cache_gives_the_contiguous_results(iq, torch, codebooks, d, page_rows):
    """A pool of pages in scrambled order behind a block table: bulk append with ragged lengths, two single-row steps
    (one of them lands on the first row of a fresh page), decode, and reconstruction must give exactly what the
    contiguous cache gives -- the gathered pool is compared with the oracle's cache and the oracle's decode."""
    B, H_q, H_kv, T = 3, 8, 2, 768
    lv, th = codebooks[d]
    cb = codebook_for(iq, codebooks, d)
    lens = np.array([700, 255, 0], np.int32)
    w = workloads.tiny(1200 + d + page_rows, B, H_q, H_kv, d, T, lens)
    n_tab = T // page_rows
    num_pages = B * n_tab + 3
    g = np.random.default_rng(page_rows + d)
    table = g.permutation(num_pages)[:B * n_tab].reshape(B, n_tab).astype(np.int32)   # every (sequence, slot) its own page
    shape = iq.Shape(B, H_q, H_kv, d, T)
    rot = torch.empty(iq.iq_rotation_floats(d, H_kv), dtype=torch.float32, device="cuda")
    iq.iq_make_rotation(d, H_kv, 0, np.ascontiguousarray(w.quats), rot)
    cache = iq.new_paged_cache(shape, num_pages, page_rows, torch.from_numpy(table).cuda())
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    k, v = torch.from_numpy(w.k).cuda(), torch.from_numpy(w.v).cuda()
    iq.iq_quantize_append(shape, rot, cb, k, v, torch.zeros(B, dtype=torch.int32, device="cuda"), torch.from_numpy(lens).cuda(), T, cache, status)
    ref = oracle.new_cache(B, H_kv, d, T)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(B, np.int32), lens, ref)
    now = lens.copy()
    for step in range(2):                                                            # sequence 1: rows 255 and 256
        kn = np.stack([w.k[b, now[b]] for b in range(B)])[:, None]
        vn = np.stack([w.v[b, now[b]] for b in range(B)])[:, None]
        iq.iq_quantize_append(shape, rot, cb, torch.from_numpy(kn).cuda(), torch.from_numpy(vn).cuda(),
                              torch.from_numpy(now).cuda(), None, 1, cache, status)
        oracle.quantize_append(w.quats, th, kn, vn, now, None, ref)
        now = now + 1
    torch.cuda.synchronize()
    assert status.cpu().numpy()[0] == 0
    gathered = _gather_pages(cache, table, page_rows)
    w2 = workloads.Workload("paged", B, H_q, H_kv, d, T, w.k, w.v, w.q, w.quats, now)
    compare_caches(w2, th, gathered, ref, now)
    used = np.zeros(num_pages, bool); used[table.ravel()] = True                     # pages outside the table stay untouched
    assert not cache.k_codes.cpu().numpy()[~used].any() and not cache.v_codes.cpu().numpy()[~used].any()
    S = iq.iq_suggest_splits(shape, T)
    res = gpu_decode(iq, torch, shape, rot, cb, w.q, cache, now, S)
    check_decode(w2, lv, w.q, res, gathered, now)
    k_out = torch.zeros((B, T, H_kv, d), dtype=torch.float16, device="cuda")
    v_out = torch.zeros_like(k_out)
    iq.iq_reconstruct_rows(shape, rot, cb, cache, torch.from_numpy(now).cuda(), k_out, v_out)
    K, V = oracle.reconstruct_rows(w.quats, lv, gathered, now, H_kv)
    for got, r in ((k_out.cpu().numpy().astype(np.float64), K), (v_out.cpu().numpy().astype(np.float64), V)):
        bound = 2.0 ** -11 * 1.001 * np.abs(r) + 1e-5 * np.abs(r).max(axis=-1, keepdims=True) + 1e-30
        assert np.all(np.abs(got - r) <= bound)
    # a block-table entry outside the pool is never turned into an address: flagged, read as page 0
    bad = table.copy(); bad[0, 1] = num_pages + 5
    cache_bad = iq.Cache(cache.k_codes, cache.k_scales, cache.v_codes, cache.v_scales, torch.from_numpy(bad).cuda(), page_rows)
    ws = iq.DecodeWorkspace(shape, S)
    iq.decode_step(shape, rot, cb, torch.from_numpy(w.q).cuda(), cache_bad, torch.from_numpy(now).cuda(), ws)
    torch.cuda.synchronize()
    assert int(ws.status[0].item()) & 4
    # quantize-append through such an entry (also a negative one) writes nothing anywhere: the rows are skipped and counted
    before = [t.clone() for t in (cache.k_codes, cache.k_scales, cache.v_codes, cache.v_scales)]
    for entry, n_new in ((num_pages + 5, 1), (-1, 1), (-1, 200)):
        bad = table.copy(); bad[0, 0] = entry
        cache_bad = iq.Cache(cache.k_codes, cache.k_scales, cache.v_codes, cache.v_scales, torch.from_numpy(bad).cuda(), page_rows)
        st2 = torch.zeros(4, dtype=torch.int32, device="cuda")
        nn = torch.tensor([n_new, 0, 0], dtype=torch.int32, device="cuda")
        iq.iq_quantize_append(shape, rot, cb, k, v, torch.zeros(B, dtype=torch.int32, device="cuda"), nn, n_new, cache_bad, st2)
        torch.cuda.synchronize()
        assert int(st2[0]) & 4 and int(st2[2]) == 2 * H_kv * min(n_new, page_rows)   # K and V rows of every KV head
        keep = torch.ones(num_pages, dtype=torch.bool, device="cuda")
        if n_new > page_rows:
            keep[int(table[0, 1])] = False                                  # rows beyond the missing page have a page and are written
        for a, bfr in zip((cache.k_codes, cache.k_scales, cache.v_codes, cache.v_scales), before):
            assert torch.equal(a[keep], bfr[keep])


def test_a_wait_that_nothing_completes_gives_up_and_reports(iq, torch):
    """The decode kernel's mbarrier waits are bounded: a one-warp kernel waits on a barrier that nothing arrives at
    (no copy, no tensor-core work in flight), gives up after its poll limit and reports IQ_STATUS_WAIT_TIMEOUT; the
    context stays usable."""
    import time
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    t0 = time.perf_counter()
    iq.iq_selftest_bounded_wait(status, 256)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    assert int(status[0]) == 2 and int(status[1]) == 256                    # the flag, and the polls it took
    assert dt < 1.0                                                         # 256 polls of at most 20 us each
    status.zero_()
    iq.iq_selftest_bounded_wait(status, 0)                                  # limit 0: the barrier is completed first
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    assert float(torch.ones(8, device="cuda").sum()) == 8.0


def test_context_sharded_decode_on_one_gpu(iq, torch, codebooks):
    """The context-sharded path with the two ranks' work done one after the other on one GPU: rows [0, 256) and
    [256, T) of every sequence in two caches, the fused decode over each, the partials laid out as the all-gather
    lays them out (rank after rank, argmax rows local to the slices, the slices' first rows beside them), one merge
    in place: the unsharded result. Then
    sharded_decode_step itself under a one-rank process group: the same as the plain step."""
    import torch.distributed as dist
    from paper_2608_08081_b200 import sharded
    d, B, H_q, H_kv, T, cut = 128, 2, 8, 2, 700, 256
    lv, th = codebooks[d]
    cb = codebook_for(iq, codebooks, d)
    lens = np.array([700, 130], np.int32)                                           # the second sequence ends inside the first slice
    w = workloads.tiny(77, B, H_q, H_kv, d, T, lens)
    t_cap = workloads.cap128(T)
    shape = iq.Shape(B, H_q, H_kv, d, t_cap)
    rot = torch.empty(iq.iq_rotation_floats(d, H_kv), dtype=torch.float32, device="cuda")
    iq.iq_make_rotation(d, H_kv, 0, np.ascontiguousarray(w.quats), rot)
    q = torch.from_numpy(w.q).cuda()
    S = 3
    parts = []
    for lo, hi in ((0, cut), (cut, T)):
        my = np.clip(lens - lo, 0, hi - lo).astype(np.int32)
        cache, status = iq.new_cache(shape), torch.zeros(4, dtype=torch.int32, device="cuda")
        iq.iq_quantize_append(shape, rot, cb, torch.from_numpy(w.k[:, lo:hi].copy()).cuda(), torch.from_numpy(w.v[:, lo:hi].copy()).cuda(),
                              torch.zeros(B, dtype=torch.int32, device="cuda"), torch.from_numpy(my).cuda(), hi - lo, cache, status)
        ws = iq.DecodeWorkspace(shape, S, want_argmax=True)
        iq.iq_decode_attention(shape, rot, cb, q, cache, torch.from_numpy(my).cuda(), S, ws.part_acc, ws.part_ml, ws.part_argmax, ws.status)
        parts.append((ws.part_acc.clone(), ws.part_ml.clone(), ws.part_argmax.clone(), cache, my, ws, lo))
    # the buffers as an all-gather into one tensor leaves them: rank after rank, argmax rows local to each slice
    acc = torch.stack([p[0] for p in parts])
    ml = torch.stack([p[1] for p in parts])
    am = torch.stack([p[2] for p in parts])
    offs = torch.tensor([[p[6]] * B for p in parts], dtype=torch.int32, device="cuda")
    out = torch.empty((B, H_q, d), dtype=torch.float32, device="cuda")
    lse = torch.empty((B, H_q), dtype=torch.float32, device="cuda")
    amx = torch.empty((B, H_q), dtype=torch.int32, device="cuda")
    iq.iq_combine_splits_sharded(shape, rot, S, 2, acc, ml, am, offs, out, lse, amx)
    torch.cuda.synchronize()
    full = oracle.new_cache(B, H_kv, d, t_cap)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(B, np.int32), lens, full)
    res = dict(out=out.cpu().numpy().astype(np.float64), lse=lse.cpu().numpy().astype(np.float64), argmax=amx.cpu().numpy())
    check_decode(w, lv, w.q, res, full, lens)
    # the library's function under a process group of one rank
    if not dist.is_initialized():
        dist.init_process_group("gloo", init_method="tcp://127.0.0.1:29557", rank=0, world_size=1)
    _, _, _, cache0, my0, ws0, _ = parts[0]
    bufs = sharded.ShardedBuffers(B, H_q, S, d, 1, True, "cuda")
    bufs.set_row_offsets(torch.zeros(B, dtype=torch.int32, device="cuda"))
    free_before = torch.cuda.mem_get_info()[0]
    o1, l1, a1 = sharded.sharded_decode_step(iq, shape, rot, cb, q, cache0, torch.from_numpy(my0).cuda(), ws0, bufs)
    o1, a1 = o1.clone(), a1.clone()
    assert torch.cuda.mem_get_info()[0] >= free_before - (4 << 20)                   # (the clones; the step itself takes nothing)
    iq.decode_step(shape, rot, cb, q, cache0, torch.from_numpy(my0).cuda(), ws0)
    torch.cuda.synchronize()
    assert torch.allclose(o1, ws0.out, atol=1e-5) and torch.equal(a1, ws0.argmax)
    dist.destroy_process_group()


@pytest.mark.parametrize("d", [128, 256])
def test_binary16_scales(iq, torch, codebooks, d):
    """The 50-bytes-per-row variant: scale arrays in binary16. Appends (bulk with ragged lengths and a partly filled
    block, then a single-row step), decode and reconstruction against the oracle with its stored norms rounded the same
    way; a row whose norm exceeds the binary16 range is stored as 65504 and flagged."""
    B, H_q, H_kv, T = 2, 8, 2, 300
    lv, th = codebooks[d]
    cb = codebook_for(iq, codebooks, d)
    lens = np.array([297, 130], np.int32)
    w = workloads.tiny(1500 + d, B, H_q, H_kv, d, T, lens)
    w.k[0, 11] = (w.k[0, 11].astype(np.float32) * 6000).astype(np.float16)             # norm ~ 6000 * sqrt(d) > 65504
    shape = iq.Shape(B, H_q, H_kv, d, w.t_cap)
    rot = torch.empty(iq.iq_rotation_floats(d, H_kv), dtype=torch.float32, device="cuda")
    iq.iq_make_rotation(d, H_kv, 0, np.ascontiguousarray(w.quats), rot)
    cache = iq.new_cache(shape, scales_dtype=torch.float16)
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    iq.iq_quantize_append(shape, rot, cb, torch.from_numpy(w.k).cuda(), torch.from_numpy(w.v).cuda(),
                          torch.zeros(B, dtype=torch.int32, device="cuda"), torch.from_numpy(lens).cuda(), T, cache, status)
    ref = oracle.new_cache(B, H_kv, d, w.t_cap)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(B, np.int32), lens, ref)
    kn = np.stack([w.k[b, lens[b]] for b in range(B)])[:, None]
    vn = np.stack([w.v[b, lens[b]] for b in range(B)])[:, None]
    iq.iq_quantize_append(shape, rot, cb, torch.from_numpy(kn).cuda(), torch.from_numpy(vn).cuda(), torch.from_numpy(lens).cuda(), None, 1, cache, status)
    oracle.quantize_append(w.quats, th, kn, vn, lens, None, ref)
    oracle.round_scales_fp16(ref)
    now = lens + 1
    torch.cuda.synchronize()
    assert status.cpu().numpy()[0] == 8                                               # IQ_STATUS_SCALE_OVERFLOW, nothing else
    g = dict(k_codes=cache.k_codes.cpu().numpy(), v_codes=cache.v_codes.cpu().numpy(),
             k_scales=cache.k_scales.float().cpu().numpy(), v_scales=cache.v_scales.float().cpu().numpy())
    assert g["k_scales"][0, :, 11].max() == 65504.0
    for name in ("k_scales", "v_scales"):                                             # equal but for norms that sit on a rounding boundary
        for b in range(B):
            a, r = g[name][b, :, :now[b]], ref[name][b, :, :now[b]]
            off = a != r
            assert off.mean() <= 2e-3 and np.all(np.abs(a - r)[off] <= 2.0 ** -10 * r[off])
    assert np.array_equal(g["k_codes"][0, :, :now[0]], ref["k_codes"][0, :, :now[0]])
    w2 = workloads.Workload("h16", B, H_q, H_kv, d, w.t_cap, w.k, w.v, w.q, w.quats, now)
    S = iq.iq_suggest_splits(shape, T)
    ws = iq.DecodeWorkspace(shape, S, want_argmax=True)
    iq.decode_step(shape, rot, cb, torch.from_numpy(w.q).cuda(), cache, torch.from_numpy(now).cuda(), ws)
    torch.cuda.synchronize()
    res = dict(out=ws.out.cpu().numpy().astype(np.float64), lse=ws.lse.cpu().numpy().astype(np.float64), argmax=ws.argmax.cpu().numpy())
    check_decode(w2, lv, w.q, res, g, now)                                            # the oracle on the GPU's own (rounded) cache
    k_out = torch.zeros((B, w.t_cap, H_kv, d), dtype=torch.float16, device="cuda")
    v_out = torch.zeros_like(k_out)
    iq.iq_reconstruct_rows(shape, rot, cb, cache, torch.from_numpy(now).cuda(), k_out, v_out)
    K, V = oracle.reconstruct_rows(w.quats, lv, g, now, H_kv)
    for got, r in ((k_out.cpu().numpy().astype(np.float64), K), (v_out.cpu().numpy().astype(np.float64), V)):
        fin = np.abs(r) < 6e4                                                         # (the blown-up row overflows binary16 outputs)
        bound = 2.0 ** -11 * 1.001 * np.abs(r) + 1e-5 * np.abs(r).max(axis=-1, keepdims=True) + 1e-30
        assert np.all((np.abs(got - r) <= bound)[fin])


@pytest.mark.parametrize("case", range(int(os.environ.get("IQ_RANDOM_CASES", "16"))))
def test_random_configurations(iq, torch, codebooks, case):
    """Seeded random shapes through the whole path: head counts and group sizes, head_dim, ragged lengths with empty
    sequences, split counts from 1 upwards, contiguous or paged cache, fp32 or binary16 scales, bulk append followed by
    single-row steps -- cache and decode output against the oracle every time."""
    g = np.random.Generator(np.random.Philox(9000 + case))
    d = int(g.choice([128, 128, 256]))
    H_kv = int(g.choice([1, 2, 3]))
    G = int(g.choice([1, 2, 4, 8, 12]))
    H_q = H_kv * G
    B = int(g.integers(1, 6))
    T = int(g.choice([128, 384, 640]))
    lens = g.integers(0, T - 3, size=B).astype(np.int32)
    if case % 4 == 0:
        lens[0] = T - 3
    paged = bool(case % 2)
    page_rows = int(g.choice([128, 128 * (T // 128)])) if paged else 0
    f16 = bool((case // 2) % 2)
    lv, th = codebooks[d]
    cb = codebook_for(iq, codebooks, d)
    w = workloads.tiny(9100 + case, B, H_q, H_kv, d, T, lens)
    shape = iq.Shape(B, H_q, H_kv, d, T)
    rot = torch.empty(iq.iq_rotation_floats(d, H_kv), dtype=torch.float32, device="cuda")
    iq.iq_make_rotation(d, H_kv, 0, np.ascontiguousarray(w.quats), rot)
    sdt = torch.float16 if f16 else torch.float32
    if paged:
        n_tab = T // page_rows
        table = g.permutation(B * n_tab + 2)[:B * n_tab].reshape(B, n_tab).astype(np.int32)
        cache = iq.new_paged_cache(shape, B * n_tab + 2, page_rows, torch.from_numpy(table).cuda(), scales_dtype=sdt)
    else:
        cache = iq.new_cache(shape, scales_dtype=sdt)
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    iq.iq_quantize_append(shape, rot, cb, torch.from_numpy(w.k).cuda(), torch.from_numpy(w.v).cuda(),
                          torch.zeros(B, dtype=torch.int32, device="cuda"), torch.from_numpy(lens).cuda(), T, cache, status)
    ref = oracle.new_cache(B, H_kv, d, T)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(B, np.int32), lens, ref)
    now = lens.copy()
    for step in range(int(g.integers(0, 3))):
        kn = np.stack([w.k[b, now[b]] for b in range(B)])[:, None]
        vn = np.stack([w.v[b, now[b]] for b in range(B)])[:, None]
        iq.iq_quantize_append(shape, rot, cb, torch.from_numpy(kn).cuda(), torch.from_numpy(vn).cuda(), torch.from_numpy(now).cuda(), None, 1, cache, status)
        oracle.quantize_append(w.quats, th, kn, vn, now, None, ref)
        now = now + 1
    if f16:
        oracle.round_scales_fp16(ref)
    torch.cuda.synchronize()
    assert status.cpu().numpy()[0] == 0
    if paged:
        got = _gather_pages(cache, table, page_rows)
    else:
        got = cache_to_numpy(cache)
    got["k_scales"] = got["k_scales"].astype(np.float32)
    got["v_scales"] = got["v_scales"].astype(np.float32)
    # the appended rows, wherever they came from: prefill rows 0 .. lens-1, then the step rows
    full_k, full_v = w.k.copy(), w.v.copy()
    w2 = workloads.Workload("rnd", B, H_q, H_kv, d, T, full_k, full_v, w.q, w.quats, now)
    if not f16:
        compare_caches(w2, th, got, ref, now)
    else:
        for b in range(B):
            assert np.array_equal(got["k_codes"][b, :, :now[b]], ref["k_codes"][b, :, :now[b]])   # codes do not depend on how the norm is stored
            nb = (int(now[b]) + 127) // 128
            vg = got["v_codes"][b].reshape(H_kv, -1)[:, :nb * 128 * oracle.row_bytes(d)]
            vr = ref["v_codes"][b].reshape(H_kv, -1)[:, :nb * 128 * oracle.row_bytes(d)]
            assert np.array_equal(vg, vr)
            a, r = got["k_scales"][b, :, :now[b]], ref["k_scales"][b, :, :now[b]]
            assert np.all(np.abs(a - r) <= 2.0 ** -10 * r)
    S = int(g.choice([1, 2, 3, iq.iq_suggest_splits(shape, T)]))
    res = gpu_decode(iq, torch, shape, rot, cb, w.q, cache, now, S)
    check_decode(w2, lv, w.q, res, got, now)
    # one more step through the one-call entry (the decode launch appends when the case is small, three launches otherwise)
    kn = np.ascontiguousarray(np.stack([w.k[b, now[b]] for b in range(B)]))
    vn = np.ascontiguousarray(np.stack([w.v[b, now[b]] for b in range(B)]))
    ws = torch.empty(iq.iq_decode_step_workspace_bytes(shape, S), dtype=torch.uint8, device="cuda")
    out = torch.empty((B, H_q, d), dtype=torch.float32, device="cuda")
    lse = torch.empty((B, H_q), dtype=torch.float32, device="cuda")
    am = torch.empty((B, H_q), dtype=torch.int32, device="cuda")
    iq.iq_decode_step_fused(shape, rot, cb, torch.from_numpy(w.q).cuda(), torch.from_numpy(kn).cuda(), torch.from_numpy(vn).cuda(), cache,
                            torch.from_numpy(now).cuda(), S, ws, out, lse, am, status)
    torch.cuda.synchronize()
    assert status.cpu().numpy()[0] == 0
    oracle.quantize_append(w.quats, th, kn[:, None], vn[:, None], now.copy(), None, ref)
    if f16:
        oracle.round_scales_fp16(ref)
    now = now + 1
    got = _gather_pages(cache, table, page_rows) if paged else cache_to_numpy(cache)
    got["k_scales"] = got["k_scales"].astype(np.float32)
    got["v_scales"] = got["v_scales"].astype(np.float32)
    for b in range(B):
        assert np.array_equal(got["k_codes"][b, :, :now[b]], ref["k_codes"][b, :, :now[b]])
    w3 = workloads.Workload("rnd", B, H_q, H_kv, d, T, full_k, full_v, w.q, w.quats, now)
    check_decode(w3, lv, w.q, dict(out=out.cpu().numpy().astype(np.float64), lse=lse.cpu().numpy().astype(np.float64), argmax=am.cpu().numpy()),
                 got, now)


def test_combine_splits_in_isolation(iq, torch, codebooks):
    d, B, H_q, H_kv, S = 128, 3, 8, 2, 5
    g = np.random.default_rng(7)
    pa = g.standard_normal((B, H_q, S, d)).astype(np.float32)
    pm = np.stack([g.standard_normal((B, H_q, S)) * 3, g.uniform(0.5, 40, (B, H_q, S))], -1).astype(np.float32)
    pg = g.integers(0, 10000, (B, H_q, S)).astype(np.int32)
    pm[0, 0, 2] = (-np.inf, 0); pg[0, 0, 2] = -1                                     # an empty split
    pm[1, 3, :] = (-np.inf, 0); pg[1, 3, :] = -1; pa[1, 3] = 0                        # an empty sequence
    pm[2, 1, 0, 0] = pm[2, 1, 4, 0] = 50.0; pg[2, 1, 0], pg[2, 1, 4] = 77, 12        # tie on the maximum: lowest row wins
    quats = workloads.quaternion_pairs(g, H_kv, d)
    ref = oracle.combine_splits(quats, pa, pm, pg, H_kv)
    shape = iq.Shape(B, H_q, H_kv, d, 128)
    rot = torch.empty(iq.iq_rotation_floats(d, H_kv), dtype=torch.float32, device="cuda")
    iq.iq_make_rotation(d, H_kv, 0, np.ascontiguousarray(quats), rot)
    out = torch.empty((B, H_q, d), dtype=torch.float32, device="cuda")
    lse = torch.empty((B, H_q), dtype=torch.float32, device="cuda")
    am = torch.empty((B, H_q), dtype=torch.int32, device="cuda")
    tt = lambda a: torch.from_numpy(a).cuda()
    iq.iq_combine_splits(shape, rot, S, tt(pa), tt(pm), tt(pg), out, lse, am)
    assert np.allclose(out.cpu().numpy(), ref["out"], atol=2e-5, rtol=1e-5)
    assert np.allclose(lse.cpu().numpy(), ref["lse"], atol=1e-4)
    assert np.array_equal(am.cpu().numpy(), ref["argmax"]) and am[2, 1].item() == 12 and am[1, 3].item() == -1
    out16 = torch.empty((B, H_q, d), dtype=torch.float16, device="cuda")
    iq.iq_combine_splits(shape, rot, S, tt(pa), tt(pm), None, out16)
    assert np.allclose(out16.float().cpu().numpy(), ref["out"], atol=2e-3, rtol=2e-3)


def test_make_rotation_from_seed(iq, torch):
    d, H = 128, 4
    a = torch.empty(iq.iq_rotation_floats(d, H), dtype=torch.float32, device="cuda")
    b = torch.empty_like(a); c = torch.empty_like(a)
    iq.iq_make_rotation(d, H, 1234, None, a)
    iq.iq_make_rotation(d, H, 1234, None, b)
    iq.iq_make_rotation(d, H, 1235, None, c)
    q = a.cpu().numpy().reshape(-1, 4)
    assert np.allclose(np.linalg.norm(q, axis=1), 1, atol=1e-6)
    assert torch.equal(a, b) and not torch.equal(a, c)
    assert abs(q.mean()) < 0.05 and abs(np.mean(q ** 2) - 0.25) < 0.02                # isotropic on S^3


def test_config2_prefill_then_64_decode_steps(iq, torch, codebooks):
    w = workloads.config2()
    lv, th = codebooks[w.d]
    cb = codebook_for(iq, codebooks, w.d)
    T, steps = 8192, w.extra["steps"]
    shape, rot, cache, status = gpu_quantize(iq, torch, w, cb, t_cap=w.t_cap)
    ref = oracle_quantize(w, th, t_cap=w.t_cap)
    S = iq.iq_suggest_splits(shape, T)
    ws = iq.DecodeWorkspace(shape, S, want_argmax=True)
    lens = torch.tensor([T], dtype=torch.int32, device="cuda")
    worst = 0.0
    for i in range(steps):
        k1 = torch.from_numpy(w.extra["step_k"][i]).cuda()
        v1 = torch.from_numpy(w.extra["step_v"][i]).cuda()
        q1 = torch.from_numpy(w.extra["step_q"][i]).cuda()
        iq.iq_quantize_append(shape, rot, cb, k1, v1, lens, None, 1, cache, status)
        lens += 1
        iq.decode_step(shape, rot, cb, q1, cache, lens, ws)
        torch.cuda.synchronize()
        oracle.quantize_append(w.quats, th, w.extra["step_k"][i], w.extra["step_v"][i], np.array([T + i], np.int32), None, ref)
        if i % 9 == 0 or i == steps - 1:                                              # every 9th step checked in full
            g = cache_to_numpy(cache)
            res = dict(out=ws.out.cpu().numpy().astype(np.float64), lse=ws.lse.cpu().numpy().astype(np.float64),
                       argmax=ws.argmax.cpu().numpy())
            worst = max(worst, check_decode(w, lv, w.extra["step_q"][i], res, g, np.array([T + i + 1], np.int32))["max_err"])
    g = cache_to_numpy(cache)
    full = workloads.Workload("c2", 1, w.H_q, w.H_kv, w.d, w.t_cap,
                              np.concatenate([w.k] + [w.extra["step_k"][i] for i in range(steps)], axis=1),
                              np.concatenate([w.v] + [w.extra["step_v"][i] for i in range(steps)], axis=1), w.q, w.quats,
                              np.array([T + steps], np.int32))
    print(compare_caches(full, th, g, ref, full.seq_lens), "worst decode err", worst)
    assert status.cpu().numpy()[0] == 0


def test_decode_step_replayed_from_a_cuda_graph(iq, torch, codebooks):
    """One decode step (append one row per sequence, attend, combine) captured once into a CUDA graph and replayed with
    new rows, new queries and growing lengths: the grids depend on the shape alone and every length is read on the
    device, so the replays must match the oracle step by step, across a 128-row block boundary, with one sequence
    that starts empty."""
    d, B, H_q, H_kv, T0, steps = 128, 3, 8, 2, 250, 12
    lv, th = codebooks[d]
    cb = codebook_for(iq, codebooks, d)
    w = workloads.tiny(77, B, H_q, H_kv, d, T0 + steps)
    lens0 = np.array([T0, 97, 0], np.int32)
    t_cap = workloads.cap128(T0 + steps)
    shape = iq.Shape(B, H_q, H_kv, d, t_cap)
    rot = torch.empty(iq.iq_rotation_floats(d, H_kv), dtype=torch.float32, device="cuda")
    iq.iq_make_rotation(d, H_kv, 0, np.ascontiguousarray(w.quats), rot)
    cache, status = iq.new_cache(shape), torch.zeros(4, dtype=torch.int32, device="cuda")
    iq.iq_quantize_append(shape, rot, cb, torch.from_numpy(w.k[:, :T0]).cuda(), torch.from_numpy(w.v[:, :T0]).cuda(),
                          torch.zeros(B, dtype=torch.int32, device="cuda"), torch.from_numpy(lens0).cuda(), T0, cache, status)
    ref = oracle.new_cache(B, H_kv, d, t_cap)
    oracle.quantize_append(w.quats, th, w.k[:, :T0], w.v[:, :T0], np.zeros(B, np.int32), lens0, ref)
    S = iq.iq_suggest_splits(shape, t_cap)
    ws = iq.DecodeWorkspace(shape, S, want_argmax=True)
    lens = torch.from_numpy(lens0).cuda()
    k1 = torch.zeros((B, 1, H_kv, d), dtype=torch.float16, device="cuda")
    v1, q1 = torch.zeros_like(k1), torch.zeros((B, H_q, d), dtype=torch.float16, device="cuda")

    def step():
        iq.iq_quantize_append(shape, rot, cb, k1, v1, lens, None, 1, cache, status)
        lens.add_(1)
        iq.decode_step(shape, rot, cb, q1, cache, lens, ws)

    g = np.random.default_rng(5)
    rows = lens0.astype(np.int64).copy()                  # next row of w.k / w.v each sequence appends
    graph = None
    for i in range(steps):
        kn = np.stack([w.k[b, rows[b]] for b in range(B)])[:, None]
        vn = np.stack([w.v[b, rows[b]] for b in range(B)])[:, None]
        qn = workloads.to_fp16(g.standard_normal((B, H_q, d)))
        k1.copy_(torch.from_numpy(kn)); v1.copy_(torch.from_numpy(vn)); q1.copy_(torch.from_numpy(qn))
        if i == 0:
            step()                                        # eager once: one-time kernel attributes are set outside a capture
        elif graph is None:
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            graph.replay()                                # capturing runs nothing
        else:
            graph.replay()
        torch.cuda.synchronize()
        oracle.quantize_append(w.quats, th, kn, vn, rows.astype(np.int32), None, ref)
        rows += 1
        now = rows.astype(np.int32)
        assert np.array_equal(lens.cpu().numpy(), now)
        res = dict(out=ws.out.cpu().numpy().astype(np.float64), lse=ws.lse.cpu().numpy().astype(np.float64),
                   argmax=ws.argmax.cpu().numpy())
        check_decode(w, lv, qn, res, cache_to_numpy(cache), now)
    gnp = cache_to_numpy(cache)
    w2 = workloads.Workload("g", B, H_q, H_kv, d, t_cap, w.k, w.v, w.q, w.quats, rows.astype(np.int32))
    compare_caches(w2, th, gnp, ref, w2.seq_lens)         # prefill rows and the rows the graph appended
    assert status.cpu().numpy()[0] == 0


def test_config3_wide_heads(iq, torch, codebooks):
    w = workloads.config3()
    S = None
    stats = _roundtrip(iq, torch, codebooks, w, [1, 19])
    print(stats)


def test_config4_long_context_retrieval(iq, torch, codebooks):
    w = workloads.config4()
    lv, th = codebooks[w.d]
    cb = codebook_for(iq, codebooks, w.d)
    shape, rot, cache, status = gpu_quantize(iq, torch, w, cb)
    g = cache_to_numpy(cache)
    ref = oracle_quantize(w, th)
    print(compare_caches(w, th, g, ref, w.seq_lens))
    S = iq.iq_suggest_splits(shape, w.t_cap)
    res = gpu_decode(iq, torch, shape, rot, cb, w.q, cache, w.seq_lens, S)
    chk = check_decode(w, lv, w.q, res, g, w.seq_lens)
    assert np.array_equal(res["argmax"][0], w.extra["needle_pos"])                    # identical to the planted positions
    assert np.array_equal(res["argmax"], chk["ref"]["argmax"])                        # and to the oracle's
    for h in range(w.H_q):
        o = res["out"][0, h]
        assert int(np.argmax(np.abs(o))) == int(w.extra["needle_chan"][h])            # dominant V channel = planted channel
        vn = w.v[0, w.extra["needle_pos"][h], h // w.G].astype(np.float64)
        assert (o @ vn) / (np.linalg.norm(o) * np.linalg.norm(vn)) > 0.9


@pytest.mark.parametrize("B,ctx", [(1, 4096), (8, 4096), (32, 4096), (1, 32768)])
def test_config5_small_points_in_full(iq, torch, codebooks, B, ctx):
    w = workloads.config5(B, ctx)
    lv, th = codebooks[w.d]
    cb = codebook_for(iq, codebooks, w.d)
    shape, rot, cache, status = gpu_quantize(iq, torch, w, cb, n_new=w.seq_lens)
    g = cache_to_numpy(cache)
    ref = oracle_quantize(w, th, n_new=w.seq_lens)
    print(compare_caches(w, th, g, ref, w.seq_lens))
    S = iq.iq_suggest_splits(shape, ctx)
    res = gpu_decode(iq, torch, shape, rot, cb, w.q, cache, w.seq_lens, S)
    c = check_decode(w, lv, w.q, res, g, w.seq_lens)
    print(c["max_err"], c["margin"])


@pytest.mark.parametrize("name", ["config5_B32_ctx32768", "config5_B8_ctx32768"])
def test_full_size_bench_configuration_sampled(iq, torch, codebooks, name):
    """Config 5 at ctx = 32768, B = 32 (the workload bench.py times) and B = 8, same launch configuration (library
    codebook, iq_suggest_splits, no argmax). The oracle checks sampled (sequence, KV head) slabs: their packed rows are
    re-quantised and every query head of the group is decoded from the GPU's own cache."""
    import bench

    assert bench.DEFAULT_WORKLOAD == "config5_B32_ctx32768"
    B, ctx, H_q, H_kv, d = bench.WORKLOADS[name]
    st = bench.build_state(name, torch.device("cuda", 0), 0)
    shape, cb, rot, cache = st["shape"], st["cb"], st["rot"], st["cache"]
    lv = np.array(cb.levels, np.float32)
    th = np.array(cb.thresholds, np.float32)
    S = iq.iq_suggest_splits(shape, ctx)
    ws = iq.DecodeWorkspace(shape, S, want_argmax=False)
    lens = torch.from_numpy(st["lens_np"]).cuda()
    q = st["q0"]
    iq.decode_step(shape, rot, cb, q, cache, lens, ws)
    torch.cuda.synchronize()
    assert int(ws.status[0]) == 0 and int(st["status"][0]) == 0
    out = ws.out.cpu().numpy().astype(np.float64)
    lse = ws.lse.cpu().numpy().astype(np.float64)
    G = H_q // H_kv
    g = np.random.default_rng(3)
    for b, kvh in [(0, 0), (int(np.argmax(st["lens_np"])), 7), (int(np.argmin(st["lens_np"])), 3), (int(g.integers(B)), int(g.integers(H_kv)))]:
        n = int(st["lens_np"][b])
        sub = {k: np.ascontiguousarray(getattr(cache, k)[b:b + 1, kvh:kvh + 1].cpu().numpy()) for k in ("k_codes", "k_scales", "v_codes", "v_scales")}
        qs = np.ascontiguousarray(q[b:b + 1, kvh * G:(kvh + 1) * G].cpu().numpy())
        ref = oracle.decode_attention(st["quats"][kvh:kvh + 1], lv, qs, sub, np.array([n], np.int32), 1)
        o = out[b, kvh * G:(kvh + 1) * G]
        err = np.abs(o - ref["out"][0])
        assert np.all(err <= 2e-3 + 1e-3 * np.abs(ref["out"][0])), f"(b={b}, kvh={kvh}) max err {err.max():.3e}"
        assert np.allclose(lse[b, kvh * G:(kvh + 1) * G], ref["lse"][0], atol=2e-3, rtol=1e-5)
    # quantize parity on sampled rows of the same cache: the generator is replayed for the first chunk of sequences
    gen = workloads.config5_device(B, ctx, torch.device("cuda", 0), H_q, H_kv, d)
    b0, k, v = next(iter(gen["chunks"]()))
    k, v = k.cpu().numpy(), v.cpu().numpy()
    kc = cache.k_codes[:k.shape[0]].cpu().numpy()
    vc = cache.v_codes[:k.shape[0]].cpu().numpy()
    ks = cache.k_scales[:k.shape[0]].cpu().numpy()
    Rs = {h: oracle.rotation_matrix(d, st["quats"][h]) for h in range(H_kv)}
    checked = 0
    for _ in range(400):
        b, h = int(g.integers(k.shape[0])), int(g.integers(H_kv))
        t = int(g.integers(int(st["lens_np"][b])))
        ck, sk, _ = oracle.quantize_row(d, Rs[h], th, k[b, t, h])
        cv, _, _ = oracle.quantize_row(d, Rs[h], th, v[b, t, h])
        assert np.array_equal(oracle.unpack_row(d, kc[b, h, t]), ck) and ks[b, h, t] == sk
        assert np.array_equal(oracle.v_row_codes(d, vc[b, h], t), cv)
        checked += 1
    assert checked == 400


def test_bench_line_keeps_its_contract():
    """bench.py on the smallest serving point: one JSON line with the keys the measurement contract names, a roofline
    object whose fraction is achieved / peak, an end-to-end leg that moved bytes both ways, and launches counted."""
    import json
    import os
    import subprocess
    import sys
    repo = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "bench.py", "--workload", "config5_B1_ctx4096", "--steps", "4", "--warmup", "3", "--no-cpu-baseline",
                        "--no-materialised"], cwd=repo, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline", "dtype",
                "data", "config", "roofline", "e2e", "gpu_launches", "clocks"):
        assert key in d, key
    assert d["steps"] == 4 and d["warmup"] == 3 and d["n_gpus"] == 1 and d["vs_baseline"] is None and d["data"] == "synthetic"
    assert d["config"]["workload"] == "config5_B1_ctx4096" and d["replays"] >= 1
    # 4 steps per replay: the bracketed one (first of every 4) by the three separate calls, the others by the one-call step (2 launches)
    assert d["gpu_launches"] == (3 + 3 * 2) * d["replays"]
    assert d["roofline"]["launches_timed"] >= 50 and d["clocks"]["samples"] >= 50
    rf = d["roofline"]
    assert rf["bound"] == "hbm" and rf["unit"] == "GB/s" and abs(rf["frac"] - rf["achieved"] / rf["peak"]) < 1e-3 and rf["traffic"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] > 0 and d["e2e"]["d2h_bytes_per_step"] > 0 and d["e2e"]["value"] > 0
    assert d["value"] > 0 and d["ms_per_step"] > 0


@pytest.mark.parametrize("d", [128, 256])
def test_empty_sequences_next_to_little_work(iq, torch, codebooks, d):
    """Many sequences without cached rows and hardly any blocks: only a few CTAs have work, and they must still define every
    partial slot of every empty sequence (the workspace is pre-filled with values a merge would take for live slots);
    likewise a batch in which no sequence has a row."""
    lv, th = codebooks[d]
    cb = codebook_for(iq, codebooks, d)
    for lens in ([5] + [0] * 199, [0] * 150 + [130, 0, 0, 1], [0] * 64):
        B = len(lens)
        w = workloads.tiny(2300 + B, B, 4, 2, d, 256, lens=lens)
        shape, rot, cache, status = gpu_quantize(iq, torch, w, cb, n_new=np.asarray(lens, np.int32))
        g = cache_to_numpy(cache)
        for S in (1, 3, 8, 24):
            ws = iq.DecodeWorkspace(shape, S, want_argmax=True)
            ws.part_acc.fill_(1.0); ws.part_ml.fill_(1.0); ws.part_argmax.fill_(7); ws.out.fill_(3.0); ws.lse.fill_(3.0)
            iq.decode_step(shape, rot, cb, torch.from_numpy(w.q).cuda(), cache, torch.from_numpy(np.asarray(lens, np.int32)).cuda(), ws)
            torch.cuda.synchronize()
            res = dict(out=ws.out.cpu().numpy().astype(np.float64), lse=ws.lse.cpu().numpy().astype(np.float64), argmax=ws.argmax.cpu().numpy())
            check_decode(w, lv, w.q, res, g, np.asarray(lens, np.int32))
            empty = np.asarray(lens) == 0
            assert np.all(res["argmax"][empty] == -1)


def test_very_many_slots(iq, torch, codebooks):
    """Slot counts beyond what one pass of the wide merge covers (more than 32 slots per warp), and odd ones."""
    lens = [700, 33, 0]
    w = workloads.tiny(2400, 3, 8, 2, 128, 768, lens=lens)
    print(_roundtrip(iq, torch, codebooks, w, [17, 33, 255, 257, 300, 1024], n_new=lens))


@pytest.mark.parametrize("d", [128, 256])
def test_softmax_scale_given_by_the_caller(iq, torch, codebooks, d):
    """iq_shape.sm_scale > 0 replaces 1/sqrt(d) (Appendix A's scale) in the plain step and in the one-call step."""
    lv, th = codebooks[d]
    cb = codebook_for(iq, codebooks, d)
    lens = np.array([300, 77], np.int32)
    w = workloads.tiny(2500 + d, 2, 8, 2, d, 304, lens=lens)
    for scale in (0.31, 0.02):
        shape = iq.Shape(w.B, w.H_q, w.H_kv, d, w.t_cap, sm_scale=scale)
        rot = torch.empty(iq.iq_rotation_floats(d, w.H_kv), dtype=torch.float32, device="cuda")
        iq.iq_make_rotation(d, w.H_kv, 0, np.ascontiguousarray(w.quats), rot)
        cache = iq.new_cache(shape)
        status = torch.zeros(4, dtype=torch.int32, device="cuda")
        iq.iq_quantize_append(shape, rot, cb, torch.from_numpy(w.k).cuda(), torch.from_numpy(w.v).cuda(),
                              torch.zeros(w.B, dtype=torch.int32, device="cuda"), torch.from_numpy(lens).cuda(), w.k.shape[1], cache, status)
        for S in (1, 8):
            res = gpu_decode(iq, torch, shape, rot, cb, w.q, cache, lens, S)
            check_decode(w, lv, w.q, res, cache_to_numpy(cache), lens, sm_scale=scale)
        ws = torch.empty(iq.iq_decode_step_workspace_bytes(shape, 8), dtype=torch.uint8, device="cuda")
        out = torch.empty((w.B, w.H_q, d), dtype=torch.float32, device="cuda")
        lse = torch.empty((w.B, w.H_q), dtype=torch.float32, device="cuda")
        am = torch.empty((w.B, w.H_q), dtype=torch.int32, device="cuda")
        kn = np.ascontiguousarray(np.stack([w.k[b, lens[b]] for b in range(w.B)]))
        vn = np.ascontiguousarray(np.stack([w.v[b, lens[b]] for b in range(w.B)]))
        iq.iq_decode_step_fused(shape, rot, cb, torch.from_numpy(w.q).cuda(), torch.from_numpy(kn).cuda(), torch.from_numpy(vn).cuda(), cache,
                                torch.from_numpy(lens).cuda(), 8, ws, out, lse, am, status)
        torch.cuda.synchronize()
        assert status.cpu().numpy()[0] == 0
        w2 = workloads.Workload("scale", w.B, w.H_q, w.H_kv, d, w.t_cap, w.k, w.v, w.q, w.quats, lens + 1)
        check_decode(w2, lv, w.q, dict(out=out.cpu().numpy().astype(np.float64), lse=lse.cpu().numpy().astype(np.float64), argmax=am.cpu().numpy()),
                     cache_to_numpy(cache), lens + 1, sm_scale=scale)


@pytest.mark.parametrize("seed", range(4))
def test_split_count_does_not_change_the_result(iq, torch, seed):
    """A property that holds at any size: which slots cover which rows is the library's choice, so the merged result
    of a launch must not depend on num_splits. Random caches (uniform codes, positive scales) with length mixes the
    oracle would take minutes for -- thousands of short sequences, many empty ones, a few long ones -- are decoded with
    one slot per head (one worker per item, no merge) and with balanced splits; outputs, lse and argmax must agree."""
    g = np.random.default_rng(500 + seed)
    for case in range(6):
        d = int(g.choice([128, 256]))
        H_kv = int(g.choice([1, 2, 4]))
        G = int(g.choice([1, 4, 8, 12]))
        H_q = H_kv * G
        B, T = [(2, 20000), (500, 256), (60, 2048), (2500, 128), (12, 8192), (300, 640)][case]
        lens = g.integers(0, T + 1, size=B).astype(np.int32)
        lens[g.random(B) < g.choice([0.0, 0.3, 0.9])] = 0
        lens[g.integers(0, B)] = T
        t_cap = workloads.cap128(T)
        shape = iq.Shape(B, H_q, H_kv, d, t_cap)
        cb = iq.iq_int8_codebook(d) if (case + seed) % 2 == 0 else iq.iq_default_codebook(d)
        rot = torch.empty(iq.iq_rotation_floats(d, H_kv), dtype=torch.float32, device="cuda")
        iq.iq_make_rotation(d, H_kv, case, None, rot)
        cache = iq.new_cache(shape)
        gen = torch.Generator(device="cuda")
        gen.manual_seed(1000 * seed + case)
        cache.k_codes.copy_(torch.randint(0, 256, cache.k_codes.shape, dtype=torch.uint8, device="cuda", generator=gen))
        cache.v_codes.copy_(torch.randint(0, 256, cache.v_codes.shape, dtype=torch.uint8, device="cuda", generator=gen))
        cache.k_scales.copy_(torch.rand(cache.k_scales.shape, device="cuda", generator=gen) * 3 + 0.1)
        cache.v_scales.copy_(torch.rand(cache.v_scales.shape, device="cuda", generator=gen) * 3 + 0.1)
        q = torch.randn((B, H_q, d), device="cuda", generator=gen).half()
        sl = torch.from_numpy(lens).cuda()
        ref = None
        for S in (1, 2, int(g.choice([8, 16, 24])), iq.iq_suggest_splits(shape, T), int(g.choice([9, 33, 100]))):
            ws = iq.DecodeWorkspace(shape, S, want_argmax=True)
            ws.part_ml.fill_(1.0); ws.part_acc.fill_(1.0); ws.part_argmax.fill_(5)   # what a merge would take for live slots
            iq.decode_step(shape, rot, cb, q, cache, sl, ws)
            torch.cuda.synchronize()
            assert int(ws.status[0]) == 0
            if ref is None:
                ref = (ws.out.clone(), ws.lse.clone(), ws.argmax.clone())
                continue
            nz = sl > 0
            assert float((ws.out - ref[0]).abs().max()) <= 2e-3, (case, S)
            assert float((ws.lse[nz] - ref[1][nz]).abs().max()) <= 2e-3, (case, S)
            assert int((ws.argmax != ref[2]).sum()) <= 0.02 * ref[2].numel() + 1, (case, S)
            assert bool((ws.out[~nz] == 0).all()) and bool(torch.isneginf(ws.lse[~nz]).all()) and bool((ws.argmax[~nz] == -1).all())
        del cache
        torch.cuda.empty_cache()
