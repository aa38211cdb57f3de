"""Pins for the fp64 oracle: every check here is against something other than the oracle itself --
the paper's printed counts, mathematical invariants, library routines, closed forms typed out
independently, or brute force on tiny inputs. CPU only."""
import math
import os

import numpy as np
import pytest
import scipy.linalg

import oracle
import workloads
from oracle import lloyd_max

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _counts():
    out = {}
    for line in open(os.path.join(GOLD, "paper_counts.txt")):
        line = line.split("#")[0].split()
        if len(line) == 2:
            out[line[0]] = float(line[1])
    return out


def _rand_quats(seed, n=1):
    g = np.random.default_rng(seed)
    q = g.standard_normal((n, 2, 4))
    q /= np.linalg.norm(q, axis=-1, keepdims=True)
    return q.reshape(n, 8).astype(np.float32)


# ---------------------------------------------------------------- binary16 inputs
def test_half_to_double_on_every_bit_pattern():
    """Every input of both sides passes through the oracle's binary16 reader: all 65536 patterns (subnormals,
    infinities, NaNs included) against numpy's float16 -> float64 conversion."""
    L = oracle.lib()
    bits = np.arange(65536, dtype=np.uint16)
    want = bits.view(np.float16).astype(np.float64)
    got = np.array([L.iqo_half_to_double(int(b)) for b in bits])
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan]) and np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))


# ---------------------------------------------------------------- H_d (Eq. 2)
@pytest.mark.parametrize("d", [4, 32, 128, 256])
def test_hadamard_matches_library_and_is_orthogonal(d):
    H = oracle.hadamard(d)
    Hint = np.rint(H * math.sqrt(d)).astype(np.int64)
    assert np.array_equal(Hint @ Hint.T, d * np.eye(d, dtype=np.int64))       # H H^T = d I exactly
    assert np.array_equal(Hint, scipy.linalg.hadamard(d))                      # Sylvester order
    assert np.allclose(H, H.T, atol=0) and np.allclose(H @ H, np.eye(d), atol=1e-14)
    assert np.allclose(H[:, 0], 1 / math.sqrt(d), atol=1e-16)


# ---------------------------------------------------------------- SO(4) block (Section 3.3, Appendix B)
def _closed_form_block(q8):
    q8 = np.asarray(q8, np.float64)
    a, b, c, d = q8[:4] / np.linalg.norm(q8[:4])
    e, f, g, h = q8[4:] / np.linalg.norm(q8[4:])
    L = np.array([[a, -b, -c, -d], [b, a, -d, c], [c, d, a, -b], [d, -c, b, a]])           # v -> qL v
    Rm = np.array([[e, f, g, h], [-f, e, -h, g], [-g, h, e, -f], [-h, -g, f, e]])          # v -> v conj(qR)
    return L @ Rm


def test_so4_block_is_a_rotation_and_matches_closed_form():
    for q8 in _rand_quats(1, 50):
        M = oracle.so4_block(q8)
        assert np.allclose(M.T @ M, np.eye(4), atol=1e-14)
        assert abs(np.linalg.det(M) - 1.0) < 1e-13
        assert np.allclose(M, _closed_form_block(q8), atol=1e-15)
        assert np.allclose(oracle.so4_block(-q8), M, atol=1e-15)                # double cover (Appendix B)


def test_so4_special_cases():
    ident = np.array([1, 0, 0, 0, 1, 0, 0, 0], np.float32)
    assert np.allclose(oracle.so4_block(ident), np.eye(4), atol=0)
    for q8 in _rand_quats(2, 10):
        q8[4:] = q8[:4]                                                         # single-quaternion conjugation
        M = oracle.so4_block(q8)
        assert np.allclose(M[0], [1, 0, 0, 0], atol=1e-15) and np.allclose(M[:, 0], [1, 0, 0, 0], atol=1e-15)
        assert abs(np.linalg.det(M[1:, 1:]) - 1) < 1e-13                        # acts as SO(3) on the imaginary part
    # unnormalised input is renormalised
    q8 = _rand_quats(3, 1)[0]
    assert np.allclose(oracle.so4_block(3.0 * q8), oracle.so4_block(q8), atol=1e-7)
    # a known rotation: qL = qR = (cos t/2, sin t/2, 0, 0) rotates the (j,k) plane by t, fixes (1,i)
    t = 0.7
    q = np.array([math.cos(t / 2), math.sin(t / 2), 0, 0] * 2, np.float64)
    M = _closed_form_block(q)
    expect = np.eye(4)
    expect[2:, 2:] = [[math.cos(t), -math.sin(t)], [math.sin(t), math.cos(t)]]
    assert np.allclose(M, expect, atol=1e-15)
    assert np.allclose(oracle.so4_block(q.astype(np.float32)), expect, atol=1e-7)


# ---------------------------------------------------------------- R = R_SO4 o H_d (Eq. 2, Appendix A)
@pytest.mark.parametrize("d", [128, 256])
def test_rotation_is_orthogonal_and_composed_in_the_stated_order(d):
    quats = workloads.quaternion_pairs(np.random.default_rng(5), 1, d)[0]
    R = oracle.rotation_matrix(d, quats)
    assert np.allclose(R.T @ R, np.eye(d), atol=1e-13)
    g = np.random.default_rng(6)
    x, y = g.standard_normal(d), g.standard_normal(d)
    assert abs((R @ x) @ (R @ y) - x @ y) < 1e-12                               # inner products preserved
    # independent composition: WHT first, then each block on its four contiguous coordinates
    hx = scipy.linalg.hadamard(d) @ x / math.sqrt(d)
    ref = np.concatenate([_closed_form_block(quats[b]) @ hx[4 * b:4 * b + 4] for b in range(d // 4)])
    assert np.allclose(R @ x, ref, atol=1e-13)
    # identity quaternions leave the WHT alone
    ident = np.tile(np.array([1, 0, 0, 0, 1, 0, 0, 0], np.float32), (d // 4, 1))
    assert np.allclose(oracle.rotation_matrix(d, ident), scipy.linalg.hadamard(d) / math.sqrt(d), atol=1e-16)


def test_post_wht_coordinate_variance_is_one_over_d():
    d = 128
    g = np.random.default_rng(7)
    x = g.standard_normal((20000, d)) * np.exp(g.standard_normal(d))            # anisotropic rows
    x /= np.linalg.norm(x, axis=1, keepdims=True)
    y = x @ oracle.hadamard(d).T
    assert abs(np.mean(y ** 2) * d - 1) < 1e-12                                  # exact by orthogonality
    assert np.all(np.abs(np.mean(y ** 2, axis=0) * d - 1) < 0.6)                 # energy spread, no hot channel


# ---------------------------------------------------------------- the paper's counts
def test_paper_counts():
    c = _counts()
    d = 128
    assert oracle.row_bytes(d) == c["packed_row_bytes_d128"] == 3 * d // 8
    assert 2 * d == c["fp16_row_bytes_d128"]
    assert round(2 * d / oracle.row_bytes(d), 1) == c["compression_ratio"]
    quats = workloads.quaternion_pairs(np.random.default_rng(0), 1, d)
    assert quats.size == c["stored_params_d128"] == c["blocks_d128"] * c["floats_per_block"]
    assert d * d == c["dense_params_d128"]
    assert (d // 4) * 6 == c["effective_dof_d128"]
    assert d * int(math.log2(d)) == c["wht_fmas_d128"]
    assert (d // 4) * c["so4_fmas_per_block"] == c["so4_fmas_d128"]
    assert c["wht_fmas_d128"] + c["so4_fmas_d128"] == c["total_fmas_d128"]
    assert round(c["dense_fmas_d128"] / c["total_fmas_d128"], 1) == c["fma_reduction"]
    transient_mb = 2 * 28 * 8 * 128 * 2048 * 2 / 1e6                             # Appendix C formula
    assert abs(transient_mb - c["prefill_transient_mb"]) / c["prefill_transient_mb"] < 0.03
    assert c["total_fmas_d128"] / (2 * 2048 * 128) < c["inverse_rotation_share_max"]


# ---------------------------------------------------------------- Lloyd-Max codebook (Step 3)
def test_lloyd_max_gaussian_limit_matches_the_textbook_table():
    rows = [l.split() for l in open(os.path.join(GOLD, "gauss_lloyd_max_8.txt")) if not l.startswith("#")]
    lv_ref, th_ref, mse_ref = [float(x) for x in rows[0]], [float(x) for x in rows[1]], float(rows[2][0])
    lv, th, mse = lloyd_max.lloyd_max(0)
    assert np.allclose(lv[4:], lv_ref, atol=6e-4) and np.allclose(-lv[:4][::-1], lv_ref, atol=6e-4)
    assert np.allclose(th[4:], th_ref, atol=6e-4) and abs(th[3]) < 1e-9
    assert abs(mse - mse_ref) < 5e-5


@pytest.mark.parametrize("d", [128, 256])
def test_lloyd_max_is_a_fixed_point_for_the_sphere_marginal(d):
    from scipy import integrate

    lv, th, mse = lloyd_max.lloyd_max(d)
    pdf, lim = lloyd_max.sphere_marginal_pdf(d)
    edges = np.concatenate(([-lim], th, [lim]))
    for i in range(8):                                                           # centroid condition, independent quadrature
        xs = np.linspace(edges[i], edges[i + 1], 200001)
        w = np.array([pdf(x) for x in xs])
        assert abs(integrate.simpson(xs * w, x=xs) / integrate.simpson(w, x=xs) - lv[i]) < 1e-7
    assert np.allclose(th, 0.5 * (lv[1:] + lv[:-1]), atol=1e-12)                 # midpoint condition
    assert np.allclose(lv, -lv[::-1], atol=1e-9)                                 # symmetry
    g_lv, _, g_mse = lloyd_max.lloyd_max(0)
    assert np.all(np.abs(lv) < np.abs(g_lv) + 1e-12) and mse < g_mse             # lighter tails than the Gaussian
    assert np.allclose(lv, g_lv, atol=0.03)
    # variance of the marginal is 1 in these units (each coordinate of a unit vector has variance 1/d)
    xs = np.linspace(-lim, lim, 400001)
    w = np.array([pdf(x) for x in xs])
    assert abs(integrate.simpson(xs * xs * w, x=xs) / integrate.simpson(w, x=xs) - 1) < 1e-6


def test_codebook_as_handed_to_both_sides(codebooks):
    from oracle import lloyd_max
    for d in (128, 256):
        lv, th = codebooks[d]
        assert lv.dtype == np.float32 and th.dtype == np.float32
        if codebooks["kind"] == "fp16":
            assert np.array_equal(lv.astype(np.float16).astype(np.float32), lv)  # exactly fp16-representable
        else:                                                                    # integer multiples of max / 127
            delta = np.float32(lv[-1]) / np.float32(127.0)
            n = lv.astype(np.float64) / np.float64(delta)
            assert np.allclose(n, np.rint(n), atol=1e-4) and np.abs(np.rint(n)).max() == 127
            exact, _, mse = lloyd_max.lloyd_max(d)
            assert np.abs(lv - exact).max() <= 0.5 * delta * 1.0001              # each level moved by at most half a grid step
            pdf = lambda u: (1 - u * u / d) ** ((d - 3) / 2) if u * u < d else 0.0
            from scipy import integrate
            edges = np.concatenate(([-np.sqrt(d)], th.astype(np.float64), [np.sqrt(d)]))
            tot = integrate.quad(pdf, -np.sqrt(d), np.sqrt(d))[0]
            mse8 = sum(integrate.quad(lambda u: (u - lv[i]) ** 2 * pdf(u), edges[i], edges[i + 1])[0] for i in range(8)) / tot
            assert mse8 <= mse * 1.002                                           # the snapping costs < 0.2 % of the distortion
        assert np.all(np.diff(lv) > 0) and np.all(np.diff(th) > 0) and th[3] == 0


# ---------------------------------------------------------------- quantise + pack (Algorithm 1)
@pytest.mark.parametrize("d", [128, 256])
def test_pack_unpack_roundtrip_and_layout(d):
    g = np.random.default_rng(11)
    assert oracle.row_bytes(d) == 3 * d // 8
    for pattern in [np.zeros(d), np.full(d, 7), np.arange(d) % 8, g.integers(0, 8, d), g.integers(0, 8, d)]:
        codes = pattern.astype(np.uint8)
        row = oracle.pack_row(d, codes)
        assert row.shape == (3 * d // 8,)
        assert np.array_equal(oracle.unpack_row(d, row), codes)
    # independent statement of the layout: one coordinate set at a time, every bit accounted for
    seen = np.zeros(3 * d, dtype=np.int64)
    for i in range(d):
        for bit in range(3):
            codes = np.zeros(d, np.uint8)
            codes[i] = 1 << bit
            words = oracle.pack_row(d, codes).view("<u4")
            grp, c = divmod(i, 32)
            if c < 24:
                w, pos = 3 * grp + c // 8, 4 * (c % 8) + bit
            else:
                w, pos = 3 * grp + bit, 4 * (c - 24) + 3
            expect = np.zeros(3 * d // 32, np.uint32)
            expect[w] = np.uint32(1) << np.uint32(pos)
            assert np.array_equal(words, expect)
            seen[32 * w + pos] += 1
    assert np.all(seen == 1)                                                    # a bijection onto the 3d bits


def test_transposed_v_layout(codebooks):
    """V codes are stored per 128-row block and coordinate: record ((t // 128) * d + c) * 48 holds the 128 codes of
    coordinate c, arranged like a packed row of 128 entries (entry = row within the block)."""
    d, T = 128, 300
    lv, th = codebooks[d]
    w = workloads.tiny(9, 1, 1, 1, d, T)
    cache = oracle.new_cache(1, 1, d, w.t_cap)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(1, np.int32), None, cache)
    R = oracle.rotation_matrix(d, w.quats[0])
    area = cache["v_codes"][0, 0].reshape(-1)
    expect = np.stack([oracle.quantize_row(d, R, th, w.v[0, t, 0])[0] for t in range(T)])          # [T][d] codes
    for j in range(w.t_cap // 128):
        for c in (0, 1, 77, 127):
            rec = area[(j * d + c) * 48:(j * d + c + 1) * 48]
            col = oracle.unpack_row(128, rec)                                                        # 128 entries = rows of block j
            rows = np.arange(128 * j, min(128 * j + 128, T))
            assert np.array_equal(col[:len(rows)], expect[rows, c])
            assert np.all(col[len(rows):] == 0)                                                      # rows never appended stay zero
    for t in (0, 31, 32, 127, 128, 299):
        assert np.array_equal(oracle.v_row_codes(d, cache["v_codes"][0, 0], t), expect[t])
    # appending row by row gives the same bytes as one bulk append
    c2 = oracle.new_cache(1, 1, d, w.t_cap)
    for t in range(T):
        oracle.quantize_append(w.quats, th, w.k[:, t:t + 1], w.v[:, t:t + 1], np.array([t], np.int32), None, c2)
    assert all(np.array_equal(cache[k], c2[k]) for k in cache)


def test_quantize_row_against_an_independent_numpy_statement(codebooks):
    d = 128
    lv, th = codebooks[d]
    w = workloads.config1(T=64)
    R = oracle.rotation_matrix(d, w.quats[0])
    for t in range(64):
        x16 = w.k[0, t, 0]
        codes, scale, u = oracle.quantize_row(d, R, th, x16)
        x = x16.astype(np.float64)
        s = math.sqrt(float(np.sum(x * x)))
        assert scale == np.float32(s)
        hx = scipy.linalg.hadamard(d) @ (x / s) / math.sqrt(d)
        xt = np.concatenate([_closed_form_block(w.quats[0, b]) @ hx[4 * b:4 * b + 4] for b in range(d // 4)])
        u_ref = math.sqrt(d) * xt
        assert np.allclose(u, u_ref, atol=1e-12)
        assert abs(np.sum(u * u) - d) < 1e-9                                     # rotation preserves the unit norm
        far = np.min(np.abs(u_ref[:, None] - th[None, :].astype(np.float64)), axis=1) > 1e-9
        nearest = np.argmin(np.abs(u_ref[:, None] - lv[None, :].astype(np.float64)), axis=1)
        assert np.array_equal(codes[far], nearest[far].astype(np.uint8))        # threshold rule == nearest level
        assert np.array_equal(codes, np.sum(u_ref[:, None] > th[None, :].astype(np.float64), axis=1))


def test_quantizer_ties_and_zero_row(codebooks):
    d = 128
    lv, th = codebooks[d]
    ident = np.tile(np.array([1, 0, 0, 0, 1, 0, 0, 0], np.float32), (d // 4, 1))
    R = oracle.rotation_matrix(d, ident)
    codes, scale, u = oracle.quantize_row(d, R, th, np.zeros(d, np.float16))
    assert scale == 0 and np.all(u == 0) and np.all(codes == 3)                  # 0 > t_3 = 0 is false: lower code
    # a row whose rotated image sits exactly on thresholds: use R = I-like probe through the definition
    codes2 = np.sum(np.array([th[5], np.nextafter(th[5], np.float32(9))], np.float64)[:, None] > th[None, :].astype(np.float64), axis=1)
    assert list(codes2) == [5, 6]


@pytest.mark.parametrize("maker,lo,hi", [
    (lambda: workloads.tiny(1, 1, 1, 1, 128, 512), 0.030, 0.038),               # Gaussian rows: the codebook's own MSE
    (lambda: workloads.config1(T=512), 0.025, 0.045),                            # x20 outlier channels
    (lambda: workloads.config3(T=256), 0.02, 0.08),                              # Student-t, d = 256
])
def test_roundtrip_reconstruction_error(codebooks, maker, lo, hi):
    w = maker()
    lv, th = codebooks[w.d]
    cache = oracle.new_cache(w.B, w.H_kv, w.d, w.t_cap)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(w.B, np.int32), None, cache)
    errs = []
    for g in range(w.H_kv):
        R = oracle.rotation_matrix(w.d, w.quats[g])
        for t in range(0, w.k.shape[1], 7):
            codes = oracle.unpack_row(w.d, cache["k_codes"][0, g, t])
            xr = R.T @ (float(cache["k_scales"][0, g, t]) * lv[codes].astype(np.float64) / math.sqrt(w.d))
            x = w.k[0, t, g].astype(np.float64)
            errs.append(np.sum((x - xr) ** 2) / np.sum(x * x))
    assert lo < float(np.mean(errs)) < hi


# ---------------------------------------------------------------- attention (Appendix A)
def _reconstruct_then_attend(w, lv, cache, sm_scale=None):
    """Brute force in numpy: dequantise every row, undo the rotation per row, textbook softmax attention."""
    d = w.d
    out = np.zeros((w.B, w.H_q, d))
    am = np.zeros((w.B, w.H_q), np.int64)
    for b in range(w.B):
        n = int(w.seq_lens[b])
        for h in range(w.H_q):
            g = h // w.G
            R = oracle.rotation_matrix(d, w.quats[g])
            K = np.stack([R.T @ (float(cache["k_scales"][b, g, t]) * lv[oracle.unpack_row(d, cache["k_codes"][b, g, t])].astype(np.float64) / math.sqrt(d)) for t in range(n)]) if n else np.zeros((0, d))
            V = np.stack([R.T @ (float(cache["v_scales"][b, g, t]) * lv[oracle.v_row_codes(d, cache["v_codes"][b, g], t)].astype(np.float64) / math.sqrt(d)) for t in range(n)]) if n else np.zeros((0, d))
            if n == 0:
                am[b, h] = -1
                continue
            z = (K @ w.q[b, h].astype(np.float64)) * (sm_scale or 1 / math.sqrt(d))
            p = np.exp(z - z.max())
            p /= p.sum()
            out[b, h] = p @ V
            am[b, h] = int(np.argmax(z))
    return out, am


@pytest.mark.parametrize("d,T,H_q,H_kv,lens", [(128, 64, 4, 1, None), (128, 37, 4, 2, [37, 5]), (256, 16, 2, 2, None),
                                               (128, 8, 2, 1, [0])])
def test_compressed_space_attention_equals_reconstruct_then_compute(codebooks, d, T, H_q, H_kv, lens):
    B = 1 if lens is None else len(lens)
    w = workloads.tiny(3, B, H_q, H_kv, d, T, lens)
    lv, th = codebooks[d]
    cache = oracle.new_cache(B, H_kv, d, w.t_cap)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(B, np.int32), w.seq_lens, cache)
    r = oracle.decode_attention(w.quats, lv, w.q, cache, w.seq_lens, H_kv, want_rot=True)
    ref, am = _reconstruct_then_attend(w, lv, cache)
    assert np.allclose(r["out"], ref, atol=1e-12)
    assert np.array_equal(r["argmax"], am)
    # omitting the inverse rotation must NOT reproduce the output (the paper's PPL 7.05 -> 15,369 remark)
    if w.seq_lens.max() > 0:
        assert np.max(np.abs(r["o_rot"] - ref)) > 0.05


@pytest.mark.parametrize("d,T,H_q,H_kv,lens", [(128, 150, 4, 2, [150, 33, 0]), (256, 40, 2, 2, None)])
def test_reconstructed_rows_give_the_same_attention_and_the_codebook_error(codebooks, d, T, H_q, H_kv, lens):
    """The reconstruct-then-compute model (Figure 1, top) pinned from three sides: rows are the quantiser's input up to
    the codebook's distortion, K and V agree with the row-by-row numpy statement, and textbook softmax attention on
    the reconstructed tensors reproduces the compressed-space result (Appendix A) -- a transposed rotation, a V row
    read from the wrong record or a missing 1/sqrt(d) fails at least one of them."""
    B = 1 if lens is None else len(lens)
    w = workloads.tiny(11, B, H_q, H_kv, d, T, lens)
    lv, th = codebooks[d]
    cache = oracle.new_cache(B, H_kv, d, w.t_cap)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(B, np.int32), w.seq_lens, cache)
    K, V = oracle.reconstruct_rows(w.quats, lv, cache, w.seq_lens, H_kv)
    assert K.shape == (B, w.t_cap, H_kv, d)
    for b in range(B):
        n = int(w.seq_lens[b])
        assert not K[b, n:].any() and not V[b, n:].any()                          # rows beyond the length stay zero
        if n == 0:
            continue
        for x, xr in ((w.k[b, :n].astype(np.float64), K[b, :n]), (w.v[b, :n].astype(np.float64), V[b, :n])):
            rel = np.sum((x - xr) ** 2, axis=-1) / np.sum(x * x, axis=-1)
            assert 0.028 < float(rel.mean()) < 0.040                              # 3-bit Lloyd-Max on N(0,1): 0.0345
        g, t = H_kv - 1, n - 1                                                    # one row, restated with the dense rotation
        R = oracle.rotation_matrix(d, w.quats[g])
        xt = float(cache["v_scales"][b, g, t]) * lv[oracle.v_row_codes(d, cache["v_codes"][b, g], t)].astype(np.float64) / math.sqrt(d)
        assert np.allclose(V[b, t, g], R.T @ xt, atol=1e-13)
    r = oracle.decode_attention(w.quats, lv, w.q, cache, w.seq_lens, H_kv)
    for b in range(B):
        n = int(w.seq_lens[b])
        for h in range(H_q):
            if n == 0:
                assert not r["out"][b, h].any()
                continue
            z = K[b, :n, h // w.G] @ w.q[b, h].astype(np.float64) / math.sqrt(d)
            p = np.exp(z - z.max())
            assert np.allclose((p / p.sum()) @ V[b, :n, h // w.G], r["out"][b, h], atol=1e-12)
            assert np.isclose(z.max() + math.log(p.sum()), r["lse"][b, h], atol=1e-12)


def test_histogram_fit_reproduces_closed_forms():
    """Lloyd's iteration on a histogram, pinned by three densities with known optima: uniform on [-1, 1) (the uniform
    quantiser: levels (2k+1)/8 - 1, mse (1/4)^2 / 12), the Gaussian (the textbook 8-level table) and a shifted Gaussian
    fitted without the symmetry constraint (the same table, shifted)."""
    lv, th, mse = lloyd_max.fit_histogram(np.ones(4096), 1.0)
    assert np.allclose(lv, (2 * np.arange(8) + 1) / 8 - 1, atol=1e-9) and np.allclose(th, np.arange(1, 8) / 4 - 1, atol=1e-9)
    assert abs(mse - 1 / 192) < 1e-12
    rows = [l.split() for l in open(os.path.join(GOLD, "gauss_lloyd_max_8.txt")) if not l.startswith("#")]
    lv_ref, mse_ref = np.array([float(x) for x in rows[0]]), float(rows[2][0])     # the textbook table (4 positive levels)
    centres = (np.arange(4096) + 0.5) * (16.0 / 4096) - 8.0
    lv, th, mse = lloyd_max.fit_histogram(np.exp(-0.5 * centres ** 2) * 1e9, 8.0)
    assert np.allclose(lv[4:], lv_ref, atol=6e-4) and np.allclose(lv[:4], -lv_ref[::-1], atol=6e-4)
    assert abs(mse - mse_ref) < 5e-5
    lv2, _, _ = lloyd_max.fit_histogram(np.exp(-0.5 * (centres - 0.3) ** 2) * 1e9, 8.0, symmetric=False)
    assert np.allclose(lv2 - 0.3, lv, atol=1e-4)
    assert np.max(np.abs(lv2 + lv2[::-1])) > 0.5                                  # and it is not symmetric about zero


def test_rotated_histogram_counts_what_the_quantiser_sees(codebooks):
    """The calibration histogram bins u = sqrt(d) R x^ -- the quantity Algorithm 1 compares with the thresholds: its
    counts equal a direct binning of the u values the row quantiser reports, zero rows are left out, and for Gaussian
    rows its first two moments are those of the post-rotation marginal (mean 0, variance 1)."""
    d, T, H_kv = 128, 300, 2
    w = workloads.tiny(21, 1, 2, H_kv, d, T)
    x = w.k[0].copy()
    x[7] = 0                                                                      # a zero row (both heads)
    bins, R = 256, 6.0
    h = lloyd_max.rotated_histogram(w.quats, x, bins, R)
    assert h.sum() == (T - 1) * H_kv * d
    _, th = codebooks[d]
    direct = np.zeros(bins, np.int64)
    for g in range(H_kv):
        Rm = oracle.rotation_matrix(d, w.quats[g])
        for t in (0, 1, 150, 299):
            _, _, u = oracle.quantize_row(d, Rm, th, x[t, g])
            direct += np.bincount(np.clip(np.floor((u + R) * bins / (2 * R)).astype(np.int64), 0, bins - 1), minlength=bins)
    part = lloyd_max.rotated_histogram(w.quats, x[[0, 1, 150, 299]], bins, R)
    assert np.array_equal(part, direct)
    centres = (np.arange(bins) + 0.5) * (2 * R / bins) - R
    mean = float((h * centres).sum() / h.sum())
    var = float((h * centres ** 2).sum() / h.sum())
    assert abs(mean) < 0.02 and abs(var - 1.0) < 0.01                             # sum of u^2 over a row is exactly d


def test_binary16_scales_variant(codebooks):
    """round_scales_fp16: the stored norms become binary16 values within 2^-11 of the exact ones (saturating at 65504),
    codes are untouched, the rounding is idempotent, and the attention output moves by no more than the scales did."""
    d = 128
    lv, th = codebooks[d]
    w = workloads.tiny(5, 1, 4, 2, d, 200)
    w.k[0, 3] = np.clip(w.k[0, 3].astype(np.float32) * 9000, -65504, 65504).astype(np.float16)
    cache = oracle.new_cache(1, 2, d, w.t_cap)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(1, np.int32), None, cache)
    exact = {k: v.copy() for k, v in cache.items()}
    oracle.round_scales_fp16(cache)
    for name in ("k_scales", "v_scales"):
        a, e = cache[name], exact[name]
        assert np.array_equal(a.astype(np.float16).astype(np.float32), a)
        ok = e <= 65504
        assert np.all(np.abs(a - e)[ok] <= 2.0 ** -11 * e[ok]) and np.all(a[~ok] == 65504.0) and (~ok).sum() == (2 if name == "k_scales" else 0)
    assert np.array_equal(cache["k_codes"], exact["k_codes"]) and np.array_equal(cache["v_codes"], exact["v_codes"])
    again = {k: v.copy() for k, v in cache.items()}
    oracle.round_scales_fp16(again)
    assert all(np.array_equal(again[k], cache[k]) for k in cache)
    lens = np.array([200], np.int32)
    keep = np.ones(200, bool); keep[3] = False                       # (leave the saturated row out of the comparison)
    for c in (cache, exact):
        c["k_scales"][0, :, 3] = 0
    r16 = oracle.decode_attention(w.quats, lv, w.q, cache, lens, 2)["out"]
    r32 = oracle.decode_attention(w.quats, lv, w.q, exact, lens, 2)["out"]
    assert np.max(np.abs(r16 - r32)) <= 4e-3 * np.max(np.abs(r32)) and np.max(np.abs(r16 - r32)) > 0


def test_attention_special_cases(codebooks):
    d = 128
    lv, th = codebooks[d]
    w = workloads.tiny(4, 1, 2, 1, d, 16)
    cache = oracle.new_cache(1, 1, d, w.t_cap)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(1, np.int32), None, cache)
    R = oracle.rotation_matrix(d, w.quats[0])
    recon = lambda t: R.T @ (float(cache["v_scales"][0, 0, t]) * lv[oracle.v_row_codes(d, cache["v_codes"][0, 0], t)].astype(np.float64) / math.sqrt(d))
    # T = 1: the output is the reconstruction of v_0
    r = oracle.decode_attention(w.quats, lv, w.q, cache, np.array([1], np.int32), 1)
    assert np.allclose(r["out"][0, 0], recon(0), atol=1e-13)
    assert np.all(r["argmax"] == 0)
    # all keys equal: uniform weights -> mean of reconstructed V, argmax = lowest index
    cache["k_codes"][0, 0, :] = cache["k_codes"][0, 0, 0]
    cache["k_scales"][0, 0, :] = cache["k_scales"][0, 0, 0]
    r = oracle.decode_attention(w.quats, lv, w.q, cache, np.array([16], np.int32), 1)
    mean_v = np.mean([recon(t) for t in range(16)], axis=0)
    assert np.allclose(r["out"][0, 1], mean_v, atol=1e-13) and np.all(r["argmax"] == 0)
    for h in range(2):
        assert abs(r["lse"][0, h] - (oracle.scores(w.quats, lv, w.q, cache, 0, h, 16, 1)[0] + math.log(16))) < 1e-12
    # empty sequence
    r = oracle.decode_attention(w.quats, lv, w.q, cache, np.array([0], np.int32), 1)
    assert np.all(r["out"] == 0) and np.all(r["argmax"] == -1) and np.all(np.isneginf(r["lse"]))


def test_score_error_statistics_against_the_bound(codebooks):
    """Eq. 3 / Appendix A: E|q.k - q.k_hat|^2 = sigma_q^2 ||q||^2 (derivation), <= d_k sigma_q^2 ||q||^2 (as printed),
    with sigma_q^2 the per-coordinate quantisation variance of the de-normalised rotated key."""
    d = 128
    lv, th = codebooks[d]
    w = workloads.tiny(5, 1, 1, 1, d, 4096)
    cache = oracle.new_cache(1, 1, d, w.t_cap)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(1, np.int32), None, cache)
    z = oracle.scores(w.quats, lv, w.q, cache, 0, 0, 4096, 1, sm_scale=1.0)
    q = w.q[0, 0].astype(np.float64)
    exact = w.k[0, :, 0].astype(np.float64) @ q
    s2 = np.mean(cache["k_scales"][0, 0].astype(np.float64) ** 2)
    _, _, mse = lloyd_max.lloyd_max(d)
    sigma2 = s2 * mse / d
    measured = float(np.mean((z - exact) ** 2))
    tight = sigma2 * float(q @ q)
    assert 0.7 * tight < measured < 1.3 * tight
    assert measured < d * tight


def test_split_merge_equals_unsplit_softmax(codebooks):
    d = 128
    lv, th = codebooks[d]
    w = workloads.tiny(6, 2, 4, 2, d, 100, lens=[100, 63])
    cache = oracle.new_cache(2, 2, d, w.t_cap)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(2, np.int32), w.seq_lens, cache)
    full = oracle.decode_attention(w.quats, lv, w.q, cache, w.seq_lens, 2, want_rot=True)
    g = np.random.default_rng(1)
    for S in (1, 3, 7):
        pa = np.zeros((2, 4, S, d), np.float32)
        pm = np.zeros((2, 4, S, 2), np.float32)
        pg = np.full((2, 4, S), -1, np.int32)
        for b in range(2):
            n = int(w.seq_lens[b])
            cuts = np.sort(np.concatenate(([0, n], g.integers(0, n + 1, S - 1))))     # arbitrary partition, may have empty splits
            for h in range(4):
                z = oracle.scores(w.quats, lv, w.q, cache, b, h, n, 2)
                R = oracle.rotation_matrix(d, w.quats[h // 2])
                for s in range(S):
                    lo, hi = cuts[s], cuts[s + 1]
                    if hi == lo:
                        pm[b, h, s] = (-np.inf, 0)
                        continue
                    m = z[lo:hi].max()
                    p = np.exp(z[lo:hi] - m)
                    vt = np.stack([float(cache["v_scales"][b, h // 2, t]) * lv[oracle.v_row_codes(d, cache["v_codes"][b, h // 2], t)].astype(np.float64) / math.sqrt(d) for t in range(lo, hi)])
                    pa[b, h, s] = p @ vt
                    pm[b, h, s] = (m, p.sum())
                    pg[b, h, s] = lo + int(np.argmax(z[lo:hi]))
        r = oracle.combine_splits(w.quats, pa, pm, pg, 2)
        assert np.allclose(r["out"], full["out"], atol=2e-6)                      # fp32 partials
        assert np.allclose(r["lse"], full["lse"], atol=1e-5)
        assert np.array_equal(r["argmax"], full["argmax"])


def test_retrieval_margins_config4_shape(codebooks):
    """Planted key scores ~ 4 ||q||^2 / sqrt(d) ~ 45, far above the Gaussian background: argmax is unambiguous."""
    d = 128
    lv, th = codebooks[d]
    w = workloads.config4(T=2048, H_q=8, H_kv=2)
    cache = oracle.new_cache(1, 2, d, w.t_cap)
    oracle.quantize_append(w.quats, th, w.k, w.v, np.zeros(1, np.int32), None, cache)
    r = oracle.decode_attention(w.quats, lv, w.q, cache, w.seq_lens, 2)
    assert np.array_equal(r["argmax"][0], w.extra["needle_pos"])
    for h in range(8):
        z = oracle.scores(w.quats, lv, w.q, cache, 0, h, 2048, 2)
        top2 = np.sort(z)[-2:]
        assert top2[1] - top2[0] > 15
        o = r["out"][0, h]
        assert int(np.argmax(np.abs(o))) == int(w.extra["needle_chan"][h])
        vn = w.v[0, w.extra["needle_pos"][h], h // 4].astype(np.float64)
        assert (o @ vn) / (np.linalg.norm(o) * np.linalg.norm(vn)) > 0.9


# ---------------------------------------------------------------- fitting the SO(4) blocks (Section 3.2: 192 learnable parameters)
def test_quaternion_pair_decomposition_inverts_the_block_matrix():
    from oracle import so4_fit
    q = _rand_quats(6, 64)
    for q8 in q:
        M = oracle.so4_block(q8)
        back = so4_fit.matrix_to_quaternion_pair(M)
        assert abs(np.linalg.norm(back[:4]) - 1) < 1e-12 and abs(np.linalg.norm(back[4:]) - 1) < 1e-12
        assert np.allclose(oracle.so4_block(back.astype(np.float32)), M, atol=5e-7)      # (the block is built from fp32 parameters)
        # the pair is determined up to a common sign (double cover)
        s = np.sign(back[:4] @ q8[:4].astype(np.float64))
        assert np.allclose(s * back, q8.astype(np.float64), atol=1e-6)
    assert np.allclose(so4_fit.matrix_to_quaternion_pair(np.eye(4)) ** 2, [1, 0, 0, 0, 1, 0, 0, 0], atol=1e-12)


def test_block_distortion_of_isotropic_data_does_not_depend_on_the_rotation():
    from oracle import so4_fit
    lv, th, mse = lloyd_max.lloyd_max(0)                       # the Gaussian-limit codebook and its distortion
    z = np.random.Generator(np.random.Philox(5)).standard_normal((200000, 4))
    q = _rand_quats(7, 3)
    ds = [so4_fit.block_distortion(z, oracle.so4_block(q8), lv, th) for q8 in q] + [so4_fit.block_distortion(z, np.eye(4), lv, th)]
    for dist in ds:
        assert abs(dist - 4 * mse) < 0.02 * 4 * mse            # four coordinates, each at the codebook's distortion
    assert max(ds) - min(ds) < 0.01 * 4 * mse


def test_rotation_fit_finds_a_planted_rotation_and_never_ends_above_its_start(codebooks):
    from oracle import so4_fit
    lv, th = codebooks[128]
    lv64 = np.asarray(lv, np.float64)
    g = np.random.Generator(np.random.Philox(11))
    Mstar = oracle.so4_block(_rand_quats(12, 1)[0])
    c = lv64[g.integers(0, 8, size=(4000, 4))]                 # points that sit exactly on levels after the planted rotation
    z = c @ Mstar                                              # u = M* z = c: zero distortion at M*
    assert so4_fit.block_distortion(z, Mstar, lv, th) < 1e-24
    start = so4_fit.givens(0, 2, 0.17) @ so4_fit.givens(1, 3, -0.11) @ Mstar
    M, before, after = so4_fit.fit_block(z, start, lv, th)
    assert before > 1e-2 and after < 1e-3 * before
    assert np.allclose(M @ M.T, np.eye(4), atol=1e-12) and abs(np.linalg.det(M) - 1) < 1e-12
    # structured (non-isotropic) data: the search improves on its start and beats most random rotations
    zz = g.standard_normal((3000, 4)) * np.array([2.0, 0.3, 1.0, 0.2])
    zz *= 2.0 / np.sqrt(np.mean(np.sum(zz * zz, axis=1)))      # mean squared norm 4, as for sqrt(d) H x^
    M2, b2, a2 = so4_fit.fit_block(zz, np.eye(4), lv, th)
    rand = sorted(so4_fit.block_distortion(zz, oracle.so4_block(q8), lv, th) for q8 in _rand_quats(13, 200))
    assert a2 <= b2 and a2 <= rand[len(rand) // 10]             # at least as good as the best tenth of 200 random rotations


def test_wht_coordinates_have_unit_variance_units():
    from oracle import so4_fit
    x = workloads.to_fp16(np.random.Generator(np.random.Philox(3)).standard_normal((64, 128)))
    z = so4_fit.wht_coordinates(x)
    assert np.allclose(np.sum(z * z, axis=1), 128.0, rtol=1e-12)          # sqrt(d) times a unit vector
    R = oracle.rotation_matrix(128, np.tile(np.array([1, 0, 0, 0, 1, 0, 0, 0], np.float32), (32, 1)))   # identity blocks: R = H
    xs = x.astype(np.float64)
    assert np.allclose(z, math.sqrt(128) * (xs / np.linalg.norm(xs, axis=1, keepdims=True)) @ R.T, atol=1e-12)


# ---------------------------------------------------------------- other bit widths (Algorithm 1 is written for a general b)
def _gauss_table(n):
    out = {}
    for line in open(os.path.join(GOLD, "gauss_lloyd_max_4_16.txt")):
        f = line.split("#")[0].split()
        if len(f) >= 3 and f[0] == str(n):
            out[f[1]] = np.array([float(x) for x in f[2:]])
    return out


@pytest.mark.parametrize("n", [4, 16])
def test_lloyd_max_gaussian_limit_matches_the_textbook_tables_for_2_and_4_bits(n):
    lv, th, mse = lloyd_max.lloyd_max(0, n_levels=n)
    t = _gauss_table(n)
    assert np.allclose(lv[n // 2:], t["levels"], atol=6e-4) and np.allclose(lv[:n // 2], -t["levels"][::-1], atol=6e-4)
    assert abs(th[n // 2 - 1]) < 1e-9 and np.allclose(th[n // 2:], t["thresholds"], atol=6e-4)
    assert abs(mse - t["mse"][0]) < 6e-5


@pytest.mark.parametrize("bits", [2, 4])
@pytest.mark.parametrize("d", [128, 256])
def test_pack_unpack_roundtrip_and_layout_other_bit_widths(d, bits):
    g = np.random.default_rng(bits * 100 + d)
    codes = g.integers(0, 1 << bits, size=d, dtype=np.uint8)
    row = oracle.pack_row(d, codes, bits)
    assert row.size == bits * d // 8 and np.array_equal(oracle.unpack_row(d, row, bits), codes)
    words = row.view("<u4")
    # the layout, stated bit by bit
    for c in range(d):
        if bits == 4:      # entry c: bits [4n, 4n+4) of word c / 8, n = c mod 8
            got = (int(words[c // 8]) >> (4 * (c % 8))) & 15
        else:              # groups of 16 entries, one word each: entry e < 8 at bits [4e, 4e+2), entry e >= 8 at bits [4(e-8)+2, 4(e-8)+4)
            e = c % 16
            got = (int(words[c // 16]) >> (4 * e if e < 8 else 4 * (e - 8) + 2)) & 3
        assert got == codes[c]
    # every bit of the row belongs to exactly one entry: flipping one code changes only that entry's bits
    for c in (0, 7, 8, 15, 16, d - 1):
        c2 = codes.copy()
        c2[c] ^= (1 << bits) - 1
        diff = np.unpackbits(oracle.pack_row(d, c2, bits) ^ row).sum()
        assert diff == bits


@pytest.mark.parametrize("bits", [2, 4])
def test_quantize_roundtrip_and_attention_identity_other_bit_widths(bits):
    """Round-trip error = the codebook's distortion, threshold rule = nearest level, the token-transposed V records, and
    compressed-space attention = reconstruct-then-compute, at 2 and 4 bits, with separate K and V codebooks."""
    d, T, H_kv, H_q = 128, 300, 2, 4
    n = 1 << bits
    lv_k, th_k = lloyd_max.int8_codebook(d, n)
    lv_f, _, mse = lloyd_max.lloyd_max(d, n)
    lv_v = (lv_k.astype(np.float64) * 1.07).astype(np.float32)                     # a different codebook for the V side
    th_v = (0.5 * (lv_v[1:].astype(np.float64) + lv_v[:-1].astype(np.float64))).astype(np.float32)
    w = workloads.tiny(500 + bits, 1, H_q, H_kv, d, T)
    cache = oracle.new_cache(1, H_kv, d, workloads.cap128(T), bits)
    assert cache["k_codes"].shape[-1] == bits * d // 8
    oracle.quantize_append(w.quats, th_k, w.k, w.v, np.zeros(1, np.int32), None, cache, thresholds_v=th_v)
    R = [oracle.rotation_matrix(d, w.quats[g]) for g in range(H_kv)]
    err = 0.0
    for t in (0, 1, 127, 128, 129, 299):
        for g in range(H_kv):
            ck, s, u = oracle.quantize_row(d, R[g], th_k, w.k[0, t, g])
            assert np.array_equal(oracle.unpack_row(d, cache["k_codes"][0, g, t], bits), ck)
            assert np.array_equal(ck, np.argmin(np.abs(u[:, None] - lv_k[None, :].astype(np.float64)), axis=1))   # nearest level
            cv, sv, uv = oracle.quantize_row(d, R[g], th_v, w.v[0, t, g])
            assert np.array_equal(oracle.v_row_codes(d, cache["v_codes"][0, g], t, bits), cv)
            # the V record of (block, coordinate), stated independently: 16 * bits bytes, entry = row in the block
            for c in (0, 5, d - 1):
                rec = cache["v_codes"][0, g].reshape(-1)[((t // 128) * d + c) * 16 * bits:][:16 * bits].view("<u4")
                e = t % 128
                if bits == 4:
                    got = (int(rec[e // 8]) >> (4 * (e % 8))) & 15
                else:
                    ee = e % 16
                    got = (int(rec[e // 16]) >> (4 * ee if ee < 8 else 4 * (ee - 8) + 2)) & 3
                assert got == cv[c]
            err += np.mean((u - lv_k.astype(np.float64)[ck]) ** 2)
    err /= 12
    assert abs(err - mse) < 0.12 * mse                                             # distortion of Gaussian rows = the codebook's
    # attention identity against a dense numpy restatement with the two codebooks
    lens = np.array([T], np.int32)
    res = oracle.decode_attention(w.quats, lv_k, w.q, cache, lens, H_kv, levels_v=lv_v)
    K, V = oracle.reconstruct_rows(w.quats, lv_k, cache, lens, H_kv, levels_v=lv_v, d=d)
    for h in range(H_q):
        g = h // (H_q // H_kv)
        q = w.q[0, h].astype(np.float64)
        z = (K[0, :T, g] @ q) / math.sqrt(d)
        a = np.exp(z - z.max()); a /= a.sum()
        assert np.allclose(res["out"][0, h], a @ V[0, :T, g], atol=1e-11)
        # and the reconstruction itself: x_hat = R^T (s * level[code] / sqrt(d))
        t = 17
        ck = oracle.unpack_row(d, cache["k_codes"][0, g, t], bits)
        assert np.allclose(K[0, t, g], R[g].T @ (cache["k_scales"][0, g, t].astype(np.float64) * lv_k.astype(np.float64)[ck] / math.sqrt(d)), atol=1e-12)
        cv = oracle.v_row_codes(d, cache["v_codes"][0, g], t, bits)
        assert np.allclose(V[0, t, g], R[g].T @ (cache["v_scales"][0, g, t].astype(np.float64) * lv_v.astype(np.float64)[cv] / math.sqrt(d)), atol=1e-12)
