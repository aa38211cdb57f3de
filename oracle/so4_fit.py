"""Fitting the SO(4) blocks of the rotation to calibration data (test infrastructure only).

Section 3.2 counts 192 learnable parameters at d = 128: the 6 rotational degrees of freedom of each of the 32
quaternion-pair blocks (Appendix B stores them as 8 floats per block). The paper does not say how they are learned.
The reading taken here: for a calibration set of rows, block b's rotation M is chosen to minimise the mean squared
quantisation error of the block's four rotated coordinates under the codebook in use,

    D_b(M) = 1/N sum_n sum_{i<4} (u_i - level[code(u_i)])^2,   u = M z_n,

where z_n holds coordinates 4b .. 4b+3 of sqrt(d) * H_d x^_n (Algorithm 1 up to the Walsh-Hadamard transform, in the
unit-variance units of the codebook) and code(u) = #{j : u > t_j}. The minimiser is a deterministic pattern search over
the six coordinate planes: rotate by +-delta in plane (i, j), keep the move if D decreases; delta starts at pi/8 and
is halved whenever a sweep over the planes improves nothing, down to 1e-3 rad. The result is returned as a unit
quaternion pair (q_L, q_R) with M = L(q_L) R(conj q_R) (Section 3.3).

Plain numpy, fp64. Pinned in tests/test_oracle_pins.py: the quaternion-pair decomposition inverts the oracle's block
matrix; the distortion of isotropic Gaussian data does not depend on the rotation and equals four times the
codebook's Gaussian distortion; the search never ends above its starting point and is at least as good as the best
of a dense random sample of rotations on a small set.
"""
from __future__ import annotations

import math

import numpy as np

PLANES = [(0, 1), (0, 2), (0, 3), (1, 2), (1, 3), (2, 3)]
DELTA0 = math.pi / 8
DELTA_MIN = 1e-3


def wht_coordinates(x_half) -> np.ndarray:
    """z = sqrt(d) * H_d x^ for rows x_half [n][d] (fp16 values): Algorithm 1, lines 1-2. Zero rows give zeros."""
    import oracle

    x = np.asarray(x_half).astype(np.float64)
    d = x.shape[-1]
    s = np.sqrt(np.sum(x * x, axis=-1, keepdims=True))
    xh = np.divide(x, s, out=np.zeros_like(x), where=s > 0)
    return math.sqrt(d) * (xh @ oracle.hadamard(d).T)


def quantise(u, levels, thresholds):
    """level[#{j : u > t_j}] element-wise."""
    lv = np.asarray(levels, np.float64)
    th = np.asarray(thresholds, np.float64)
    code = np.sum(u[..., None] > th, axis=-1)
    return lv[code]


def block_distortion(z4, M, levels, thresholds) -> float:
    """D_b(M) for z4 [n][4]."""
    u = z4 @ np.asarray(M, np.float64).T
    e = u - quantise(u, levels, thresholds)
    return float(np.sum(e * e) / z4.shape[0])


def givens(i: int, j: int, angle: float) -> np.ndarray:
    G = np.eye(4)
    c, s = math.cos(angle), math.sin(angle)
    G[i, i] = c; G[j, j] = c; G[i, j] = -s; G[j, i] = s
    return G


def fit_block(z4, M0, levels, thresholds):
    """Pattern search from M0; returns (M, distortion at M0, distortion at M)."""
    M = np.asarray(M0, np.float64).copy()
    best = start = block_distortion(z4, M, levels, thresholds)
    delta = DELTA0
    while delta >= DELTA_MIN:
        improved = False
        for (i, j) in PLANES:
            for sign in (1.0, -1.0):
                cand = givens(i, j, sign * delta) @ M
                dist = block_distortion(z4, cand, levels, thresholds)
                if dist < best:
                    M, best, improved = cand, dist, True
                    break
        if not improved:
            delta *= 0.5
    return M, start, best


def _basis():
    """T[a][b] = L(e_a) R(conj e_b): the 16 matrices a block matrix is bilinear in (q_L, q_R) over."""
    import oracle

    T = np.zeros((4, 4, 4, 4))
    for a in range(4):
        for b in range(4):
            q8 = np.zeros(8, np.float32)
            q8[a] = 1.0
            q8[4 + b] = 1.0
            T[a, b] = oracle.so4_block(q8)
    return T


def matrix_to_quaternion_pair(M) -> np.ndarray:
    """(q_L.wxyz, q_R.wxyz), both of unit length, with L(q_L) R(conj q_R) = M for M in SO(4). The 16 matrices
    L(e_a) R(conj e_b) are orthogonal under the Frobenius product (norm^2 = 4), so <M, T_ab> / 4 = l_a r_b: a rank-one
    matrix whose largest row gives r up to sign, and l follows."""
    T = _basis()
    P = np.einsum("abij,ij->ab", T, np.asarray(M, np.float64)) / 4.0
    a = int(np.argmax(np.sum(P * P, axis=1)))
    r = P[a] / np.linalg.norm(P[a])
    l = P @ r
    l /= np.linalg.norm(l)
    return np.concatenate([l, r])


def fit_rotation(z, quats0, levels, thresholds):
    """Fits every block of one head: z [n][d] (wht_coordinates of the calibration rows), quats0 [d/4][8] the starting
    rotation. Returns (quats [d/4][8] fp64, mean distortion per coordinate before, after)."""
    import oracle

    z = np.asarray(z, np.float64)
    d = z.shape[1]
    out = np.zeros((d // 4, 8))
    before = after = 0.0
    for b in range(d // 4):
        M0 = oracle.so4_block(np.asarray(quats0, np.float32)[b])
        M, s, e = fit_block(z[:, 4 * b:4 * b + 4], M0, levels, thresholds)
        out[b] = matrix_to_quaternion_pair(M)
        before += s
        after += e
    return out, before / d, after / d
