"""The decode entry point for callers that cannot allocate device memory (stream-capture code, plugins
that own only their inputs and outputs, fixed memory budgets): iq_decode_attention_static keeps the split
partials in an array inside the library instead of caller buffers. Its output must equal the regular
iq_decode_attention + iq_combine_splits path, on two calls in a row (the array is shared between calls
and keeps the previous call's contents). Collected last on purpose."""
import numpy as np
import pytest

import workloads

pytestmark = pytest.mark.gpu


def test_static_scratch_decode_matches_regular_path_twice(codebooks):
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2608_08081_b200 as iq
    from helpers import cache_to_numpy, check_decode, codebook_for, gpu_quantize

    outs = []
    # two different problems back to back: the second one (fewer heads, other lengths, other split count)
    # runs over whatever the first left in the shared array
    for seed, (B, H_q, H_kv, d, T, lens, S) in enumerate([(3, 8, 2, 128, 640, [640, 77, 0], 5), (2, 4, 4, 256, 200, [200, 131], 3)]):
        w = workloads.tiny(900 + seed, B, H_q, H_kv, d, T, lens=lens)
        cb = codebook_for(iq, codebooks, d)
        shape, rot, cache, _ = gpu_quantize(iq, torch, w, cb, n_new=lens)
        q = torch.from_numpy(w.q).cuda()
        sl = torch.tensor(lens, dtype=torch.int32, device="cuda")
        ws = iq.DecodeWorkspace(shape, S)
        ref = iq.decode_step(shape, rot, cb, q, cache, sl, ws).clone()
        ref_lse = ws.lse.clone()
        out = torch.full((B, H_q, d), float("nan"), dtype=torch.float32, device="cuda")
        lse = torch.full((B, H_q), float("nan"), dtype=torch.float32, device="cuda")
        status = torch.zeros(4, dtype=torch.int32, device="cuda")
        if seed == 0:
            # set-up call: the first call on a device looks up the array's address; with CUDA's lazy module
            # loading this is also when the driver places the library's fixed array on the GPU
            iq.iq_decode_attention_static(shape, rot, cb, q, cache, sl, S, out, lse, status)
            torch.cuda.synchronize()
            out.fill_(float("nan")); lse.fill_(float("nan"))
        free_before = torch.cuda.mem_get_info()[0]
        iq.iq_decode_attention_static(shape, rot, cb, q, cache, sl, S, out, lse, status)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before            # after set-up, a call takes no device memory
        assert int(status[0]) == 0
        # same kernels on the same inputs; the decode kernel hands out blocks dynamically, so the fp32 summation order
        # (and nothing else) may differ between two calls
        assert np.allclose(out.cpu().numpy(), ref.cpu().numpy(), atol=1e-5, rtol=1e-5)
        assert np.allclose(lse.cpu().numpy(), ref_lse.cpu().numpy(), atol=1e-5, rtol=1e-6)
        # and against the fp64 oracle on the same packed cache, at the tolerance of the parity tests
        lv, _ = codebooks[d]
        check_decode(w, lv, w.q, dict(out=out.cpu().numpy().astype(np.float64), lse=lse.cpu().numpy().astype(np.float64), argmax=None),
                     cache_to_numpy(cache), np.asarray(lens, np.int32))
        out16 = torch.empty((B, H_q, d), dtype=torch.float16, device="cuda")
        iq.iq_decode_attention_static(shape, rot, cb, q, cache, sl, S, out16)
        torch.cuda.synchronize()
        assert np.allclose(out16.float().cpu().numpy(), ref.cpu().numpy(), atol=2e-3, rtol=2e-3)
        outs.append(out)
    # a request beyond the fixed array is refused before anything is launched
    big = iq.Shape(64, 64, 8, 128, 1024)
    need = 64 * 64 * 64 * 130 * 4
    assert need > iq.iq_static_scratch_bytes()
    with pytest.raises(iq.IQError) as e:
        iq.iq_decode_attention_static(big, rot, cb, q, cache, sl, 64, outs[0])
    assert e.value.code == -6
