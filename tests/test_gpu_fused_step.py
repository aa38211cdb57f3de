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
