"""C-ABI boundary on the CPU: the library loads, exports every declared symbol, validates arguments
before any launch, and its host-side codebook matches the oracle-side tool. No kernel is launched."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def iq():
    import paper_2608_08081_b200 as m
    return m


def test_library_exports_every_declared_symbol(iq):
    header = open(os.path.join(ROOT, "include", "isoquant.h")).read()
    names = set(re.findall(r"\b(iq_[a-z_0-9]+)\s*\(", header))
    assert {"iq_make_rotation", "iq_quantize_append", "iq_decode_attention", "iq_combine_splits"} <= names
    lib = ctypes.CDLL(iq.lib_path())
    for n in sorted(names):
        assert hasattr(lib, n), f"{n} declared in isoquant.h but not exported"
    assert iq.iq_version() == 300 and iq.iq_format_version() == 3
    for n in sorted(names):
        assert hasattr(iq, n) or n in ("iq_shape", "iq_codebook", "iq_cache"), f"binding lacks {n}"


def test_sizes(iq):
    assert iq.iq_row_bytes(128) == 48 and iq.iq_row_bytes(256) == 96 and iq.iq_row_bytes(64) == 0
    assert iq.iq_rotation_floats(128, 1) == 256 and iq.iq_rotation_floats(256, 8) == 8 * 512


def test_default_codebook_matches_oracle_tool(iq, codebooks):
    for d in (128, 256):
        cb = iq.iq_default_codebook(d) if codebooks["kind"] == "fp16" else iq.iq_int8_codebook(d)
        lv, th = codebooks[d]
        assert np.array_equal(np.array(cb.levels, np.float32), lv)      # two independent Lloyd-Max implementations
        assert np.allclose(np.array(cb.thresholds, np.float32), th, atol=0)
    with pytest.raises(iq.IQError):
        iq.iq_default_codebook(96)


def test_codebook_fitted_to_a_histogram_matches_the_oracle(iq):
    """iq_fit_codebook is host code: Lloyd's iteration on a histogram against the oracle's independent implementation,
    for a Gaussian, a heavy-tailed and a skewed histogram, with and without the symmetry constraint, on both grids."""
    from oracle import lloyd_max
    bins, R = 2048, 8.0
    c = (np.arange(bins) + 0.5) * (2 * R / bins) - R
    hists = {"gauss": np.exp(-0.5 * c * c), "student_t3": (1 + c * c / 3) ** -2.0, "skewed": np.exp(-0.5 * (c - 0.4) ** 2) + 0.3 * np.exp(-2 * (c + 1.5) ** 2)}
    for name, dens in hists.items():
        h = np.rint(dens * 1e8).astype(np.uint32)
        for symmetric in (True, False):
            lv, _, _ = lloyd_max.fit_histogram(h, R, symmetric=symmetric)
            cb16 = iq.iq_fit_codebook(h, R, symmetric=symmetric, grid="fp16")
            assert np.array_equal(np.array(cb16.levels, np.float32), lv.astype(np.float16).astype(np.float32)), (name, symmetric)
            th16 = 0.5 * (np.array(cb16.levels, np.float64)[1:] + np.array(cb16.levels, np.float64)[:-1])
            assert np.array_equal(np.array(cb16.thresholds, np.float32), th16.astype(np.float32))
            cb8 = iq.iq_fit_codebook(h, R, symmetric=symmetric, grid="int8")
            delta = np.float32(np.max(np.abs(lv)) / 127.0)
            n = np.rint(lv / np.float64(delta))
            assert np.array_equal(np.array(cb8.levels, np.float32), (n.astype(np.float32) * delta).astype(np.float32)), (name, symmetric)
            if symmetric:
                assert np.array_equal(np.array(cb8.levels)[::-1], -np.array(cb8.levels)) and cb8.thresholds[3] == 0.0
    with pytest.raises(iq.IQError):
        iq.iq_fit_codebook(np.zeros(bins, np.uint32), R)                 # no data
    # 4 and 16 levels (Algorithm 1's b = 2 and 4)
    for bits in (2, 4):
        h = np.rint(hists["skewed"] * 1e8).astype(np.uint32)
        for symmetric in (True, False):
            lv, _, _ = lloyd_max.fit_histogram(h, R, n_levels=1 << bits, symmetric=symmetric)
            cb16 = iq.iq_fit_codebook(h, R, symmetric=symmetric, grid="fp16", bits=bits)
            assert cb16.bits == bits and len(cb16.levels) == 1 << bits
            assert np.allclose(np.array(cb16.levels, np.float64), lv.astype(np.float16).astype(np.float64), rtol=0, atol=2e-3), (bits, symmetric)
            cb8 = iq.iq_fit_codebook(h, R, symmetric=symmetric, grid="int8", bits=bits)
            delta = np.max(np.abs(cb8.levels)) / 127.0
            assert np.allclose(np.array(cb8.levels) / delta, np.rint(np.array(cb8.levels) / delta), atol=1e-4)
            assert np.allclose(cb8.levels, lv, rtol=0, atol=0.6 * delta + 2e-3)
    # the library's Lloyd-Max codebooks for the post-rotation marginal, every width and both grids
    for d in (128, 256):
        for bits in (2, 3, 4):
            for kind, make in (("int8", lloyd_max.int8_codebook), ("fp16", lloyd_max.fp16_codebook)):
                cb = iq.iq_lloyd_max_codebook(d, bits, kind)
                lv, th = make(d, 1 << bits)
                assert np.allclose(cb.levels, lv, rtol=0, atol=2e-3) and np.allclose(cb.thresholds, th, rtol=0, atol=2e-3), (d, bits, kind)
    two = iq.iq_codebook_set_v(iq.iq_lloyd_max_codebook(128, 4, "int8"), iq.iq_lloyd_max_codebook(128, 4, "fp16"))
    assert two.v_levels == iq.iq_lloyd_max_codebook(128, 4, "fp16").levels and two.levels == iq.iq_lloyd_max_codebook(128, 4, "int8").levels
    with pytest.raises(iq.IQError):
        iq.iq_codebook_set_v(iq.iq_lloyd_max_codebook(128, 4, "int8"), iq.iq_lloyd_max_codebook(128, 2, "int8"))


class _P:
    """Fake tensor: just a device-pointer-like integer (never dereferenced: validation fails first)."""
    def __init__(self, p): self._p = p
    def data_ptr(self): return self._p


def _call(iq, fn, *a):
    try:
        fn(*a)
    except iq.IQError as e:
        return e.code
    return 0


def test_argument_validation_happens_before_any_launch(iq, monkeypatch):
    import paper_2608_08081_b200.binding as B
    monkeypatch.setattr(B, "_stream", lambda s=None: None)
    lib = B._lib
    cb = iq.iq_default_codebook(128).c()
    good = B._IqShape(1, 4, 1, 128, 1024, 3, 0.0)
    cache = B._IqCache(0x1000, 0x2000, 0x3000, 0x4000)
    A = 0x10000  # aligned fake pointer
    def qa(shape, rot=A, cbk=cb, k=A, v=A, sb=1024 * 128, st=128, sh=128, pos=A, nn=None, n=1, c=cache):
        return lib.iq_quantize_append(ctypes.byref(shape), rot, ctypes.byref(cbk), k, v, sb, st, sh, pos, nn, n, ctypes.byref(c), None, None)
    assert qa(B._IqShape(1, 4, 1, 64, 1024, 3, 0.0)) == -2          # head_dim
    assert qa(B._IqShape(1, 4, 1, 128, 1024, 5, 0.0)) == -2         # bits
    assert qa(B._IqShape(1, 4, 1, 128, 1024, 4, 0.0)) == -4         # bits that the codebook is not for
    assert qa(B._IqShape(1, 5, 2, 128, 1024, 3, 0.0)) == -2         # n_q % n_kv
    assert qa(B._IqShape(1, 4, 1, 128, 1022, 3, 0.0)) == -2         # t_cap % 4
    assert qa(good, rot=None) == -1
    assert qa(good, k=None) == -1
    assert qa(good, k=A + 2) == -3
    assert qa(good, st=130) == -3
    assert qa(good, n=-1) == -2
    assert qa(good, c=B._IqCache(0x1000, 0x2004, 0x3000, 0x4000)) == -3
    assert qa(good, c=B._IqCache(0x1000, 0, 0x3000, 0x4000)) == -1
    assert qa(good, n=0) == 0                                        # no-op, nothing launched
    bad = iq.iq_default_codebook(128).c(); bad.levels[3] = -0.2443    # ascending but not fp16-representable: fine for quantize...
    assert qa(good, cbk=bad, n=0) == 0
    bad2 = iq.iq_default_codebook(128).c(); bad2.thresholds[2] = 5.0  # ...but thresholds must ascend
    assert qa(good, cbk=bad2) == -4

    def da(shape, cbk=cb, q=A, S=2, pa=A, pm=A, lens=A):
        return lib.iq_decode_attention(ctypes.byref(shape), A, ctypes.byref(cbk), q, ctypes.byref(cache), lens, S, pa, pm, None, None, None)
    assert da(good, cbk=bad) == -4                                   # decode needs fp16-exact levels
    assert da(good, S=0) == -2
    assert da(good, q=None) == -1
    assert da(good, pa=A + 4) == -3
    assert da(B._IqShape(0, 4, 1, 128, 1024, 3, 0.0)) == 0           # empty batch: nothing launched

    def cs(shape, S=2, out=A, pg=None, ao=None):
        return lib.iq_combine_splits(ctypes.byref(shape), A, S, A, A, pg, out, 0, None, ao, None)
    assert cs(good, S=0) == -2
    assert cs(good, out=None) == -1
    assert cs(good, ao=A) == -1                                      # argmax_out without part_argmax
    assert "binary16" in iq.iq_strerror(-4) and "8-bit grid" in iq.iq_strerror(-4)

    # the no-allocation entry point: its size limit and its output pointer are checked before any CUDA call
    def ds(shape, S=2, out=A):
        return lib.iq_decode_attention_static(ctypes.byref(shape), A, ctypes.byref(cb), A, ctypes.byref(cache), A, S, out, 0, None, None, None)
    assert ds(B._IqShape(64, 64, 8, 128, 1024, 3, 0.0), S=64) == -6   # 64 * 64 * 64 * 130 floats > the fixed array
    assert ds(good, out=None) == -1
    assert ds(good, out=A + 4) == -3
    assert ds(good, S=0) == -2
    assert ds(B._IqShape(1, 4, 1, 64, 1024, 3, 0.0)) == -2
    assert lib.iq_decode_attention_static(None, A, ctypes.byref(cb), A, ctypes.byref(cache), A, 2, A, 0, None, None, None) == -1

    # the host-buffer step refuses what its three parts would refuse before it enqueues the copy and the append
    def hs(shape, cbk=cb, S=2, pa=A, out=A):
        return lib.iq_decode_step_host(ctypes.byref(shape), A, ctypes.byref(cbk), A, A, A, A, ctypes.byref(cache), S, pa, A, out, A, 0, None, None)
    assert hs(good, cbk=bad) == -4
    assert hs(good, S=0) == -2
    assert hs(good, pa=None) == -1
    assert hs(good, out=A + 8) == -3
    assert lib.iq_make_rotation(96, 1, 0, None, A, None) == -2
    assert lib.iq_make_rotation(128, 1, 0, None, None, None) == -1


def test_suggest_splits_is_sane(iq):
    # one slot per piece of an item and group of the CTA that holds it (4 groups at head_dim 128, 2 at 256): a multiple
    # of the group count, at least two pieces, no more pieces than groups' worth of 128-row blocks
    s = iq.iq_suggest_splits(iq.Shape(1, 32, 8, 128, 32768), 32768)
    assert s % 4 == 0 and 8 <= s <= 4 * 64
    assert iq.iq_suggest_splits(iq.Shape(1, 4, 1, 128, 1024), 100) == 8
    assert iq.iq_suggest_splits(iq.Shape(32, 64, 8, 128, 32768), 32768) == 8
    assert iq.iq_suggest_splits(iq.Shape(1, 16, 8, 256, 16384), 16384) % 2 == 0


def test_rotation_fit_on_the_host_matches_the_oracle(iq, codebooks):
    """iq_fit_rotation is host code: the same pattern search as the oracle's, written independently in C++. On structured
    calibration rows both must end at the same distortion (the two evaluate the same fp64 sums in a different order, so a
    comparison at a near-tie may go the other way: distortions are compared, not paths), the product's quaternion pairs
    must give, under the oracle's distortion, what the product reports, and no block may end above its start."""
    import oracle
    import workloads
    from oracle import lloyd_max, so4_fit
    d = 128
    lv, th = codebooks[d]
    cb = iq.Codebook(tuple(float(x) for x in lv), tuple(float(x) for x in th))
    g = np.random.Generator(np.random.Philox(21))
    scales = np.where(np.arange(d) % 2 == 1, 4.0, 1.0) * np.exp(0.5 * g.standard_normal(d))   # channel scales that correlate the block's coordinates
    x = workloads.to_fp16(g.standard_normal((768, d)) * scales)
    z = so4_fit.wht_coordinates(x).astype(np.float32)
    q0 = workloads.quaternion_pairs(g, 1, d)[0]
    q_ref, b_ref, a_ref = so4_fit.fit_rotation(z.astype(np.float64), q0, lv, th)
    q_lib, b_lib, a_lib = iq.iq_fit_rotation(z, d, cb, q0)
    assert abs(b_lib - b_ref) < 1e-12 * b_ref
    assert a_lib <= b_lib and a_ref <= b_ref and a_ref < 0.97 * b_ref          # the fit pays on such data
    assert abs(a_lib - a_ref) < 2e-3 * a_ref
    again = sum(so4_fit.block_distortion(z[:, 4 * b:4 * b + 4].astype(np.float64), oracle.so4_block(q_lib[b]), lv, th) for b in range(d // 4)) / d
    assert abs(again - a_lib) < 1e-5 * a_lib                                   # the pairs it returns are the rotation it found
    for bits in (2, 4):                                                        # the same with 4 and 16 levels
        lvb, thb = lloyd_max.int8_codebook(d, 1 << bits)
        cbb = iq.Codebook(tuple(float(x) for x in lvb), tuple(float(x) for x in thb))
        _, b_r, a_r = so4_fit.fit_rotation(z[:256].astype(np.float64), q0, lvb, thb)
        _, b_l, a_l = iq.iq_fit_rotation(np.ascontiguousarray(z[:256]), d, cbb, q0)
        assert abs(b_l - b_r) < 1e-12 * b_r and a_l <= b_l and abs(a_l - a_r) < 5e-3 * a_r, (bits, b_l, b_r, a_l, a_r)
    assert np.allclose(np.linalg.norm(q_lib.reshape(-1, 2, 4), axis=-1), 1.0, atol=1e-6)
    # argument checks, no CUDA involved
    import ctypes
    import paper_2608_08081_b200.binding as B
    c = cb.c()
    assert B._lib.iq_fit_rotation(None, 4, 128, 128, ctypes.byref(c), q_lib.ctypes.data, None) == -1
    assert B._lib.iq_fit_rotation(z.ctypes.data, 0, 128, 128, ctypes.byref(c), q_lib.ctypes.data, None) == -2
    assert B._lib.iq_fit_rotation(z.ctypes.data, 4, 64, 128, ctypes.byref(c), q_lib.ctypes.data, None) == -2
