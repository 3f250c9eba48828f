"""Plain CPU oracle of the calibration of the inter-block rotation: block covariance and
Algorithm 1 ("Givens Rotation for Variance Equalization", Section 5.1) in float64.

TEST INFRASTRUCTURE, like the rest of this package: never on the product path.

What is computed.  For calibration activations X [T, d] viewed per token as [B, K] (B = d/32
blocks of K = 32), the covariance across blocks, pooled over tokens and positions,
    Sigma[b, b'] = (1 / (T K)) sum_t sum_k x[t, b, k] x[t, b', k]
(the mean inside blocks is taken as zero, as Section 5.1 assumes), and an orthogonal Q with
    diag(Q Sigma Q^T) = c 1,   c = tr(Sigma) / B
(Theorem 1: equal block variances minimise a convex block error).  Q is the matrix R_B that the
structured rotation applies to a token's blocks, Y = R_B X, so the covariance of Y is Q Sigma Q^T.

Readings of points where Algorithm 1 as printed is silent or at odds with its own stated output:
  * the angle.  The printed angle, half the arctangent of 2 sigma_ij / (sigma_ii - sigma_jj), is
    the Jacobi angle that zeroes sigma_ij; it moves the two diagonal entries APART (to the
    eigenvalues of the 2 x 2 block), which cannot reach the stated output.  The angle used here
    is the one of the Schur-Horn construction the section is named after: rotate in the (i, j)
    plane until sigma_ii equals the target c exactly, which is possible because the two
    deviations have opposite signs.  With t = tan(theta):
        (sigma_jj - c) t^2 - 2 sigma_ij t + (sigma_ii - c) = 0,
    the root of smaller magnitude, t = (sigma_ii - c) / (sigma_ij + sgn(sigma_ij) sqrt(D)),
    D = sigma_ij^2 - (sigma_ii - c)(sigma_jj - c) > 0.  Every rotation settles one block for good,
    so at most B - 1 rotations are needed: the O(B^2) total the section states.
  * the pair.  "A pair with opposite deviation signs" is any such pair; here i is the block with
    the largest deviation, j the one with the smallest (most negative); ties go to the lowest
    index.
  * the accumulated matrix.  The listing updates Sigma <- G^T Sigma G and R <- R G, for which the
    final Sigma is R^T Sigma_0 R, while its output line asks for diag(R Sigma R^T); the matrix
    returned here is Q = (G_1 G_2 ...)^T, the one that satisfies the output line.
  * the threshold is absolute, as printed: stop when max_i |sigma_ii - c| <= eps.
  * pooling over positions: one matrix shared by all K positions (the structure the structured
    rotation kernel takes); a per-position matrix would run the same routine on each Sigma_k.

Pins (tests/test_oracle_givens.py): closed form for 2 x 2, the stated output on random and
outlier-heavy covariances, orthogonality, invariance of the spectrum and the trace, rotation
count, identity on an already equal diagonal, and brute-force covariance loops.
"""
from __future__ import annotations

import math

import numpy as np

from .torq_oracle import K_BLOCK, decode_bf16

__all__ = ["block_covariance", "givens_equalize", "block_variances"]


def block_covariance(x_bits: np.ndarray) -> np.ndarray:
    """X [T, d] bfloat16 bit patterns -> Sigma [B, B] float64, pooled over tokens and positions."""
    x = decode_bf16(x_bits)
    t, d = x.shape
    assert d % K_BLOCK == 0
    nb = d // K_BLOCK
    a = x.reshape(t, nb, K_BLOCK).transpose(0, 2, 1).reshape(t * K_BLOCK, nb)    # rows = (token, position)
    return (a.T @ a) / float(t * K_BLOCK)


def block_variances(z: np.ndarray) -> np.ndarray:
    """Mean square of each block of Z [T, d] (float64): the diagonal of its block covariance."""
    t, d = z.shape
    return (np.asarray(z, dtype=np.float64).reshape(t, d // K_BLOCK, K_BLOCK) ** 2).mean(axis=(0, 2))


def givens_equalize(sigma: np.ndarray, eps: float, max_rotations: int | None = None):
    """Algorithm 1 with the readings in the module header.
    Returns (Q [B,B] with diag(Q sigma Q^T) = c 1 to eps, the rotated covariance, number of rotations).
    Every scalar step is a single float64 operation written out, so that another implementation
    can follow it operation by operation."""
    s = np.array(sigma, dtype=np.float64, copy=True)
    nb = s.shape[0]
    assert s.shape == (nb, nb)
    q = np.eye(nb, dtype=np.float64)
    tr = 0.0
    for b in range(nb):                                   # in index order
        tr = tr + s[b, b]
    c = tr / nb
    limit = 4 * nb if max_rotations is None else max_rotations
    n = 0
    while n < limit:
        dev = np.diagonal(s) - c
        i = int(np.argmax(dev))                           # first index of the largest deviation
        j = int(np.argmin(dev))                           # first index of the smallest
        if max(dev[i], -dev[j]) <= eps:
            break
        if i == j:                                        # cannot happen while a deviation exceeds eps
            break
        da, dd, b = dev[i], dev[j], s[i, j]
        disc = b * b - da * dd                            # da > 0 >= dd or da >= 0 > dd: disc >= b^2
        root = math.sqrt(disc)
        den = b + root if b >= 0.0 else b - root
        if den == 0.0:                                    # both deviations and the coupling vanish
            break
        t = da / den
        cs = 1.0 / math.sqrt(1.0 + t * t)
        sn = t * cs
        # Sigma <- G^T Sigma G,  G = I except G[i,i] = G[j,j] = cs, G[i,j] = sn, G[j,i] = -sn
        ci, cj = s[:, i].copy(), s[:, j].copy()
        s[:, i] = ci * cs - cj * sn
        s[:, j] = ci * sn + cj * cs
        ri, rj = s[i, :].copy(), s[j, :].copy()
        s[i, :] = ri * cs - rj * sn
        s[j, :] = ri * sn + rj * cs
        # Q <- G^T Q
        qi, qj = q[i, :].copy(), q[j, :].copy()
        q[i, :] = qi * cs - qj * sn
        q[j, :] = qi * sn + qj * cs
        n += 1
    return q, s, n
