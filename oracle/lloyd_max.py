"""Lloyd-Max scalar quantiser for the post-rotation marginal (test infrastructure only).

Step 3 of the compression pipeline quantises each rotated coordinate with a codebook that minimises
the expected squared error under the post-rotation marginal. After normalisation and an orthogonal
rotation the vector is (for isotropic data) a uniform point on the unit sphere S^{d-1}; one
coordinate, in unit-variance units u = sqrt(d) * x, then has density proportional to
(1 - u^2/d)^((d-3)/2) on |u| < sqrt(d). Lloyd's iteration (Lloyd 1982; Max 1960): each level is the
centroid of its cell, each threshold the midpoint of neighbouring levels.

Everything is fp64 with adaptive quadrature (scipy.integrate.quad). The paper prints no codebook
values and its codebook files are not available: parity with the authors' files is unpinned. The
iteration itself is pinned by its fixed-point property and by the Gaussian limit d -> inf, which must
reproduce the textbook 8-level Gaussian Lloyd-Max table.
"""
from __future__ import annotations

import math

import numpy as np
from scipy import integrate


def sphere_marginal_pdf(d: int):
    """Unnormalised density of sqrt(d) * (one coordinate of a uniform point on S^{d-1})."""
    if d <= 0:  # Gaussian limit
        return (lambda u: math.exp(-0.5 * u * u)), math.inf
    e = 0.5 * (d - 3)
    return (lambda u: (max(0.0, 1.0 - u * u / d)) ** e), math.sqrt(d)


def lloyd_max(d: int, n_levels: int = 8, iters: int = 2000, tol: float = 1e-13):
    """Returns (levels[n_levels], thresholds[n_levels-1], mse) in fp64. d <= 0 selects the Gaussian limit."""
    pdf, lim = sphere_marginal_pdf(d)
    hi = lim if math.isfinite(lim) else 12.0
    levels = np.linspace(-2.0, 2.0, n_levels)
    for _ in range(iters):
        th = 0.5 * (levels[1:] + levels[:-1])
        edges = np.concatenate(([-hi], th, [hi]))
        new = np.empty_like(levels)
        for i in range(n_levels):
            a, b = edges[i], edges[i + 1]
            mass = integrate.quad(pdf, a, b, epsabs=1e-15, epsrel=1e-13)[0]
            mom = integrate.quad(lambda u: u * pdf(u), a, b, epsabs=1e-15, epsrel=1e-13)[0]
            new[i] = mom / mass
        delta = float(np.max(np.abs(new - levels)))
        levels = new
        if delta < tol:
            break
    th = 0.5 * (levels[1:] + levels[:-1])
    edges = np.concatenate(([-hi], th, [hi]))
    total = integrate.quad(pdf, -hi, hi, epsabs=1e-15, epsrel=1e-13)[0]
    err = 0.0
    for i in range(n_levels):
        err += integrate.quad(lambda u: (u - levels[i]) ** 2 * pdf(u), edges[i], edges[i + 1], epsabs=1e-15, epsrel=1e-13)[0]
    return levels, th, err / total


def fp16_codebook(d: int, n_levels: int = 8):
    """Codebook in the form handed to both the oracle and the CUDA library: levels rounded to values
    exactly representable in binary16 (stored as fp32), thresholds = midpoints of those levels (fp32)."""
    lv, _, _ = lloyd_max(d, n_levels)
    lv16 = lv.astype(np.float16).astype(np.float32)
    th = (0.5 * (lv16[1:].astype(np.float64) + lv16[:-1].astype(np.float64))).astype(np.float32)
    return lv16, th


def int8_codebook(d: int, n_levels: int = 8):
    """The same codebook with its levels snapped to an 8-bit grid: level_j = n_j * delta with integer |n_j| <= 127 and
    delta = max|level| / 127 (all in fp32, as handed to the oracle and the CUDA library); thresholds = midpoints of the
    snapped levels. The decode kernel's integer tensor-core path needs levels of this form."""
    lv, _, _ = lloyd_max(d, n_levels)
    a = 0.5 * (lv - lv[::-1])                      # exact symmetry first (ascending, a[-1] = -a[0] > 0)
    delta = np.float32(a[-1] / 127.0)
    n = np.rint(a / np.float64(delta)).astype(np.int32)
    lv8 = (n.astype(np.float32) * delta).astype(np.float32)
    th = (0.5 * (lv8[1:].astype(np.float64) + lv8[:-1].astype(np.float64))).astype(np.float32)
    return lv8, th


# ---------------------------------------------------------------- fitting the codebook to data (Section 3.2, Step 3)
# The paper calls the codebook "Lloyd-Max for the post-rotation distribution" without saying how that distribution is
# obtained. Reading taken here: the empirical marginal of u = sqrt(d) * R x^ over a calibration set of K/V rows, as a
# histogram with uniform bins on [-range, range) (values outside fall into the end bins), and Lloyd's iteration on
# that histogram read as a piecewise-constant density.
def rotated_histogram(quats, x_half, bins: int, rng_half: float) -> np.ndarray:
    """Counts [bins] (int64) of the rotated normalised coordinates of the rows x_half, fp16 [..., H_kv, d]; zero rows
    are skipped. quats: fp32 [H_kv][d/4][8]."""
    import oracle

    x = np.asarray(x_half)
    H_kv, d = x.shape[-2], x.shape[-1]
    rows = x.reshape(-1, H_kv, d).astype(np.float64)
    counts = np.zeros(bins, dtype=np.int64)
    for g in range(H_kv):
        R = oracle.rotation_matrix(d, np.asarray(quats)[g])
        xg = rows[:, g, :]
        s = np.sqrt(np.sum(xg * xg, axis=1))
        xg = xg[s > 0] / s[s > 0, None]
        u = math.sqrt(d) * (xg @ R.T)
        idx = np.floor((u + rng_half) * (bins / (2.0 * rng_half))).astype(np.int64)
        counts += np.bincount(np.clip(idx, 0, bins - 1).ravel(), minlength=bins)
    return counts


def fit_histogram(counts, rng_half: float, n_levels: int = 8, symmetric: bool = True, iters: int = 5000, tol: float = 1e-13):
    """Lloyd's iteration on a histogram read as a piecewise-constant density (a bin cut by a threshold contributes to
    both cells in proportion): returns (levels, thresholds, mse) in fp64, in the histogram's units.
    symmetric: the histogram is first averaged with its mirror image, which makes the codebook symmetric about 0."""
    c = np.asarray(counts, dtype=np.float64)
    if symmetric:
        c = 0.5 * (c + c[::-1])
    bins = c.size
    w = 2.0 * rng_half / bins
    edges = np.arange(bins + 1) * w - rng_half
    total = c.sum()
    assert total > 0
    mass0 = np.concatenate(([0.0], np.cumsum(c)))                                   # mass below edge i
    mom0 = np.concatenate(([0.0], np.cumsum(c * 0.5 * (edges[1:] + edges[:-1]))))   # first moment below edge i
    sq0 = np.concatenate(([0.0], np.cumsum(c * (edges[1:] ** 3 - edges[:-1] ** 3) / (3.0 * w))))  # second moment

    def below(t):
        """(mass, first moment, second moment) of the density below t."""
        t = min(max(t, -rng_half), rng_half)
        i = min(int((t + rng_half) / w), bins - 1)
        dens = c[i] / w
        return (mass0[i] + dens * (t - edges[i]), mom0[i] + dens * 0.5 * (t * t - edges[i] ** 2),
                sq0[i] + dens * (t ** 3 - edges[i] ** 3) / 3.0)

    qs = np.interp((np.arange(n_levels) + 0.5) / n_levels, mass0 / total, edges)    # start: quantiles
    levels = qs.copy()
    for _ in range(iters):
        cuts = [-rng_half] + list(0.5 * (levels[1:] + levels[:-1])) + [rng_half]
        st = [below(t) for t in cuts]
        new = levels.copy()
        for i in range(n_levels):
            m = st[i + 1][0] - st[i][0]
            if m > 0:
                new[i] = (st[i + 1][1] - st[i][1]) / m
        if symmetric:
            new = 0.5 * (new - new[::-1])
        delta = float(np.max(np.abs(new - levels)))
        levels = new
        if delta < tol:
            break
    th = 0.5 * (levels[1:] + levels[:-1])
    cuts = [-rng_half] + list(th) + [rng_half]
    st = [below(t) for t in cuts]
    mse = 0.0
    for i in range(n_levels):   # sum over cells of E[(u - l)^2] = second - 2 l first + l^2 mass
        m, f, q = (st[i + 1][k] - st[i][k] for k in range(3))
        mse += q - 2.0 * levels[i] * f + levels[i] ** 2 * m
    return levels, th, float(mse / total)
