"""Parity of the decode step whose decode launch also appends the step's new rows (two launches instead of three) with the
oracle: the cache after the step must equal the oracle's cache after its own append, and the output must equal the
oracle's attention over that cache, the new row included."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
import workloads
from helpers import cache_to_numpy, check_decode, codebook_for, compare_caches, gpu_quantize

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


def _step(iq, torch, codebooks, w, lens_before, S, append=True, want_argmax=True, t_cap=None, steps=1):
    """Prefill lens_before[b] rows, then `steps` one-launch steps (each appending the next row of the workload when
    `append`), each checked against the oracle."""
    lv, th = codebooks[w.d]
    cb = codebook_for(iq, codebooks, w.d)
    lens = np.asarray(lens_before, np.int32).copy()
    t_cap = t_cap or w.t_cap
    shape, rot, cache, status = gpu_quantize(iq, torch, w, cb, t_cap=t_cap, n_new=lens)
    ref = oracle.new_cache(w.B, w.H_kv, w.d, t_cap)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(w.B, np.int32), lens, ref)
    ws = torch.full((iq.iq_decode_step_workspace_bytes(shape, S),), 0xA5, dtype=torch.uint8, device="cuda")   # needs no initialisation
    out = torch.full((w.B, w.H_q, w.d), 7.0, dtype=torch.float32, device="cuda")
    lse = torch.full((w.B, w.H_q), 7.0, dtype=torch.float32, device="cuda")
    am = torch.full((w.B, w.H_q), 7, dtype=torch.int32, device="cuda") if want_argmax else None
    q = torch.from_numpy(w.q).cuda()
    stats = []
    for step in range(steps):
        T = w.k.shape[1]
        idx = np.minimum(lens, T - 1)
        k_new = np.ascontiguousarray(w.k[np.arange(w.B), idx])   # [B][H_kv][d]
        v_new = np.ascontiguousarray(w.v[np.arange(w.B), idx])
        sl = torch.from_numpy(lens).cuda()
        status.zero_()
        iq.iq_decode_step_fused(shape, rot, cb, q, torch.from_numpy(k_new).cuda() if append else None,
                                torch.from_numpy(v_new).cuda() if append else None, cache, sl, S, ws, out, lse, am, status)
        torch.cuda.synchronize()
        st = status.cpu().numpy()
        full = lens >= t_cap
        if append:
            assert (st[0] != 0) == bool(full.any()) and st[2] == 2 * w.H_kv * int(full.sum()), st
            oracle.quantize_append(w.quats, th, k_new[:, None], v_new[:, None], lens.copy(), (~full).astype(np.int32), ref)
            lens = np.where(full, lens, lens + 1).astype(np.int32)
        else:
            assert st[0] == 0
        g = cache_to_numpy(cache)
        compare_caches(w, th, g, ref, lens)
        res = dict(out=out.cpu().numpy().astype(np.float64), lse=lse.cpu().numpy().astype(np.float64),
                   argmax=None if am is None else am.cpu().numpy())
        c = check_decode(w, lv, w.q, res, g, lens)
        stats.append((c["max_err"], c["margin"], c["argmax_exact"], c["argmax_ties"]))
    return stats


@pytest.mark.parametrize("d", [128, 256])
@pytest.mark.parametrize("T", [0, 1, 127, 128, 129, 1000])
def test_single_sequence_context_lengths(iq, torch, codebooks, d, T):
    w = workloads.tiny(700 + T, 1, 8 if d == 128 else 4, 2, d, T + 4)
    for S in (1, 3, 8, 16):
        print(T, S, _step(iq, torch, codebooks, w, [T], S, steps=2))


def test_ragged_batch_with_empty_and_full_sequences(iq, torch, codebooks):
    lens = [0, 1, 64, 257, 512, 100, 0, 511, 127, 128]
    w = workloads.tiny(730, 10, 8, 2, 128, 520, lens=lens)
    for S in (1, 4, 9, 16, 33):
        print(S, _step(iq, torch, codebooks, w, lens, S, t_cap=512, steps=3))   # sequence 4 is full: no new row, flagged


@pytest.mark.parametrize("G", [1, 4, 16])
def test_group_sizes(iq, torch, codebooks, G):
    w = workloads.tiny(740 + G, 2, 2 * G, 2, 128, 400)
    print(_step(iq, torch, codebooks, w, [300, 123], 8, steps=2))
    print(_step(iq, torch, codebooks, w, [300, 123], 2, steps=2, want_argmax=False))
    print(_step(iq, torch, codebooks, w, [300, 123], 40, steps=2))   # many slots: the merge spreads a head over a CTA


@pytest.mark.parametrize("d", [128, 256])
def test_long_single_sequence(iq, torch, codebooks, d):
    T = 32768 if d == 128 else 16384
    w = workloads.tiny(750, 1, 8, 2, d, T + 2)
    shape = iq.Shape(1, 8, 2, d, w.t_cap)
    S = iq.iq_suggest_splits(shape, T)
    print(S, _step(iq, torch, codebooks, w, [T], S, steps=2))


def test_more_sequences_than_sms(iq, torch, codebooks):
    B = 400
    g = np.random.default_rng(5)
    lens = g.integers(0, 200, size=B).astype(np.int32)
    w = workloads.tiny(760, B, 4, 2, 128, 256, lens=lens)
    print(_step(iq, torch, codebooks, w, lens, 8, steps=2)[-1])
    print(_step(iq, torch, codebooks, w, lens, 3, steps=1)[-1])


def test_paged_cache_and_binary16_scales(iq, torch, codebooks):
    """The step's append inside the decode launch on a pool of scrambled pages with binary16 scale arrays: the new rows
    land in the right pages (one of them on the first row of a fresh page), the output equals the oracle's with its
    stored norms rounded the same way, and a page that is missing from the table costs the row, not another page."""
    d, B, H_q, H_kv, T, page_rows = 128, 3, 8, 2, 768, 128
    lv, th = codebooks[d]
    cb = codebook_for(iq, codebooks, d)
    lens = np.array([700, 255, 0], np.int32)
    w = workloads.tiny(770, B, H_q, H_kv, d, T, lens)
    n_tab = T // page_rows
    num_pages = B * n_tab + 2
    table = np.random.default_rng(3).permutation(num_pages)[:B * n_tab].reshape(B, n_tab).astype(np.int32)
    shape = iq.Shape(B, H_q, H_kv, d, T)
    rot = torch.empty(iq.iq_rotation_floats(d, H_kv), dtype=torch.float32, device="cuda")
    iq.iq_make_rotation(d, H_kv, 0, np.ascontiguousarray(w.quats), rot)
    cache = iq.new_paged_cache(shape, num_pages, page_rows, torch.from_numpy(table).cuda(), scales_dtype=torch.float16)
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    iq.iq_quantize_append(shape, rot, cb, torch.from_numpy(w.k).cuda(), torch.from_numpy(w.v).cuda(),
                          torch.zeros(B, dtype=torch.int32, device="cuda"), torch.from_numpy(lens).cuda(), T, cache, status)
    ref = oracle.new_cache(B, H_kv, d, T)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(B, np.int32), lens, ref)
    S = 8
    ws = torch.empty(iq.iq_decode_step_workspace_bytes(shape, S), dtype=torch.uint8, device="cuda")
    out = torch.empty((B, H_q, d), dtype=torch.float32, device="cuda")
    lse = torch.empty((B, H_q), dtype=torch.float32, device="cuda")
    am = torch.empty((B, H_q), dtype=torch.int32, device="cuda")
    now = lens.copy()
    q = torch.from_numpy(w.q).cuda()

    def gathered():
        def pool(a):
            a = a.cpu().numpy()
            return np.stack([np.concatenate([a[table[b, j]] for j in range(n_tab)], axis=1) for b in range(B)])
        g = dict(k_codes=pool(cache.k_codes), v_codes=pool(cache.v_codes),
                 k_scales=pool(cache.k_scales).astype(np.float32), v_scales=pool(cache.v_scales).astype(np.float32))
        return g

    for step in range(2):                                                # sequence 1: rows 255 and 256 (a fresh page)
        kn = np.ascontiguousarray(np.stack([w.k[b, now[b]] for b in range(B)]))
        vn = np.ascontiguousarray(np.stack([w.v[b, now[b]] for b in range(B)]))
        iq.iq_decode_step_fused(shape, rot, cb, q, torch.from_numpy(kn).cuda(), torch.from_numpy(vn).cuda(), cache,
                                torch.from_numpy(now).cuda(), S, ws, out, lse, am, status)
        torch.cuda.synchronize()
        assert status.cpu().numpy()[0] == 0
        oracle.quantize_append(w.quats, th, kn[:, None], vn[:, None], now.copy(), None, ref)
        now = now + 1
        ref16 = {k_: v_.copy() for k_, v_ in ref.items()}
        oracle.round_scales_fp16(ref16)
        g = gathered()
        assert np.array_equal(g["k_codes"][0, :, :now[0]], ref16["k_codes"][0, :, :now[0]])
        for b in range(B):
            n = int(now[b])
            assert np.array_equal(g["k_codes"][b, :, :n], ref16["k_codes"][b, :, :n])
            assert np.mean(g["k_scales"][b, :, :n] != ref16["k_scales"][b, :, :n]) <= 2e-3 + 1.0 / max(n * H_kv, 1)
        w2 = workloads.Workload("paged", B, H_q, H_kv, d, T, w.k, w.v, w.q, w.quats, now)
        res = dict(out=out.cpu().numpy().astype(np.float64), lse=lse.cpu().numpy().astype(np.float64), argmax=am.cpu().numpy())
        check_decode(w2, lv, w.q, res, g, now)
    # a page missing from the table: the new row of that sequence is skipped and counted, every page stays as it was
    bad = table.copy(); bad[1, int(now[1]) // page_rows] = -1
    cache_bad = iq.Cache(cache.k_codes, cache.k_scales, cache.v_codes, cache.v_scales, torch.from_numpy(bad).cuda(), page_rows)
    if True:
        before = [t.clone() for t in (cache.k_codes, cache.v_codes)]
        only1 = torch.tensor([-5, int(now[1]), -5], dtype=torch.int32, device="cuda")     # the other sequences: out of range, no row either
        status.zero_()
        kn = torch.from_numpy(np.ascontiguousarray(w.k[:, 0])).cuda()
        iq.iq_decode_step_fused(shape, rot, cb, q, kn, kn, cache_bad, only1, S, ws, out, lse, am, status)
        torch.cuda.synchronize()
        st = status.cpu().numpy()
        assert st[0] & 4 and st[0] & 1 and st[2] == 3 * 2 * H_kv
        assert torch.equal(cache.k_codes, before[0]) and torch.equal(cache.v_codes, before[1])


@pytest.mark.parametrize("bits", [2, 4])
def test_other_bit_widths_take_the_three_launch_route(iq, torch, bits):
    """The one-call step at 2 and 4 bits (the three launches behind the same contract) against the oracle."""
    from oracle import lloyd_max
    d, B, H_q, H_kv, T = 128, 2, 8, 2, 300
    lv, th = lloyd_max.int8_codebook(d, 1 << bits)
    cb = iq.Codebook(tuple(map(float, lv)), tuple(map(float, th)))
    lens = np.array([259, 128], np.int32)
    w = workloads.tiny(780 + bits, B, H_q, H_kv, d, T + 2, lens)
    shape = iq.Shape(B, H_q, H_kv, d, w.t_cap, bits=bits)
    rot = torch.empty(iq.iq_rotation_floats(d, H_kv), dtype=torch.float32, device="cuda")
    iq.iq_make_rotation(d, H_kv, 0, np.ascontiguousarray(w.quats), rot)
    cache = iq.new_cache(shape)
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    iq.iq_quantize_append(shape, rot, cb, torch.from_numpy(w.k).cuda(), torch.from_numpy(w.v).cuda(),
                          torch.zeros(B, dtype=torch.int32, device="cuda"), torch.from_numpy(lens).cuda(), w.k.shape[1], cache, status)
    ref = oracle.new_cache(B, H_kv, d, w.t_cap, bits)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(B, np.int32), lens, ref)
    S = 8
    ws = torch.empty(iq.iq_decode_step_workspace_bytes(shape, S), dtype=torch.uint8, device="cuda")
    out = torch.empty((B, H_q, d), dtype=torch.float32, device="cuda")
    lse = torch.empty((B, H_q), dtype=torch.float32, device="cuda")
    am = torch.empty((B, H_q), dtype=torch.int32, device="cuda")
    kn = np.ascontiguousarray(np.stack([w.k[b, lens[b]] for b in range(B)]))
    vn = np.ascontiguousarray(np.stack([w.v[b, lens[b]] for b in range(B)]))
    iq.iq_decode_step_fused(shape, rot, cb, torch.from_numpy(w.q).cuda(), torch.from_numpy(kn).cuda(), torch.from_numpy(vn).cuda(), cache,
                            torch.from_numpy(lens).cuda(), S, ws, out, lse, am, status)
    torch.cuda.synchronize()
    assert status.cpu().numpy()[0] == 0
    oracle.quantize_append(w.quats, th, kn[:, None], vn[:, None], lens.copy(), None, ref)
    now = lens + 1
    g = cache_to_numpy(cache)
    for b in range(B):
        assert np.array_equal(g["k_codes"][b, :, :now[b]], ref["k_codes"][b, :, :now[b]])
    w2 = workloads.Workload("bits", B, H_q, H_kv, d, w.t_cap, w.k, w.v, w.q, w.quats, now)
    res = dict(out=out.cpu().numpy().astype(np.float64), lse=lse.cpu().numpy().astype(np.float64), argmax=am.cpu().numpy())
    check_decode(w2, lv, w.q, res, g, now)
