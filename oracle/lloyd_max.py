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


def fp16_codebook(d: int):
    """Codebook in the form handed to both the oracle and the CUDA library: levels rounded to values
    exactly representable in binary16 (stored as fp32), thresholds = midpoints of those levels (fp32)."""
    lv, _, _ = lloyd_max(d)
    lv16 = lv.astype(np.float16).astype(np.float32)
    th = (0.5 * (lv16[1:].astype(np.float64) + lv16[:-1].astype(np.float64))).astype(np.float32)
    return lv16, th


def int8_codebook(d: int):
    """The same codebook with its levels snapped to an 8-bit grid: level_j = n_j * delta with integer |n_j| <= 127 and
    delta = max|level| / 127 (all in fp32, as handed to the oracle and the CUDA library); thresholds = midpoints of the
    snapped levels. The decode kernel's integer tensor-core path needs levels of this form."""
    lv, _, _ = lloyd_max(d)
    a = 0.5 * (lv - lv[::-1])                      # exact symmetry first (ascending, a[7] = -a[0] > 0)
    delta = np.float32(a[-1] / 127.0)
    n = np.rint(a / np.float64(delta)).astype(np.int32)
    lv8 = (n.astype(np.float32) * delta).astype(np.float32)
    th = (0.5 * (lv8[1:].astype(np.float64) + lv8[:-1].astype(np.float64))).astype(np.float32)
    return lv8, th
