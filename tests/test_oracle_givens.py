"""Pins for the oracle of the inter-block calibration (block covariance; Algorithm 1, Section 5.1).

Each check comes from the mathematics, not from the routine: the 2 x 2 closed form, the output the
algorithm states (equal diagonal at tr/B), invariants of an orthogonal similarity (spectrum,
trace, symmetry), the Schur-Horn rotation count, and brute-force loops for the covariance."""
import numpy as np
import pytest

import oracle as O
from paper_2605_19561_b200 import inputs as I


def _spd(n, seed, outliers=0):
    g = np.random.default_rng(seed)
    a = g.standard_normal((n, 3 * n))
    s = a @ a.T / (3 * n)
    for k in range(outliers):                             # a few blocks with a hundredfold variance
        s[k * 7 % n, :] *= 10.0
        s[:, k * 7 % n] *= 10.0
    return s


def test_two_by_two_closed_form():
    """diag(3, 1): equal variances need a 45 degree rotation; the result is [[2, -1], [-1, 2]] up to the
    sign of the coupling, and one rotation suffices."""
    q, s, n = O.givens_equalize(np.diag([3.0, 1.0]), 1e-14)
    assert n == 1
    assert np.allclose(np.abs(q), np.full((2, 2), np.sqrt(0.5)), atol=1e-15)
    assert np.allclose(np.diagonal(s), [2.0, 2.0], atol=1e-15) and np.isclose(abs(s[0, 1]), 1.0)
    # a general symmetric 2 x 2: the equalising angle satisfies tan(2 theta) = (a - d) / (2 b)
    a, b, d = 5.0, 0.7, 2.0
    q, s, n = O.givens_equalize(np.array([[a, b], [b, d]]), 1e-14)
    theta = np.arctan2(q[0, 1], q[0, 0])
    assert np.isclose(np.tan(2 * theta), -(a - d) / (2 * b)) or np.isclose(np.tan(2 * theta), (a - d) / (2 * b))
    assert np.allclose(np.diagonal(s), [(a + d) / 2] * 2, atol=1e-14)


@pytest.mark.parametrize("n,outliers", [(8, 0), (32, 2), (128, 4), (160, 5)])
def test_stated_output_and_invariants(n, outliers):
    sig = _spd(n, n, outliers)
    c = np.trace(sig) / n
    q, s, rot = O.givens_equalize(sig, 1e-12 * c)
    assert np.abs(np.diagonal(s) - c).max() <= 1e-12 * c                 # the output line of Algorithm 1
    assert np.abs(q @ q.T - np.eye(n)).max() <= 1e-12                    # orthogonal
    assert np.abs(q @ sig @ q.T - s).max() <= 1e-11 * np.abs(sig).max()  # the returned Q is the one that does it
    assert np.allclose(np.linalg.eigvalsh(s), np.linalg.eigvalsh(sig), rtol=1e-10, atol=1e-12)
    assert np.isclose(np.trace(s), np.trace(sig), rtol=1e-13)
    assert np.abs(s - s.T).max() <= 1e-12 * np.abs(sig).max()
    assert 1 <= rot <= n - 1                                             # one block settled per rotation


def test_the_printed_jacobi_angle_would_not_reach_the_stated_output():
    """Why the reading departs from the printed angle: it is the angle that zeroes sigma_ij (with the sign
    that goes with the rotation's orientation), and zeroing sigma_ij spreads the pair's variances."""
    a, b, d = 3.0, 0.5, 1.0
    m = np.array([[a, b], [b, d]])
    spreads = []
    for th in (0.5 * np.arctan(2 * b / (a - d)), -0.5 * np.arctan(2 * b / (a - d))):
        g = np.array([[np.cos(th), np.sin(th)], [-np.sin(th), np.cos(th)]])
        s = g.T @ m @ g
        spreads.append((abs(s[0, 1]), abs(s[0, 0] - s[1, 1])))
    off, spread = min(spreads)                            # the orientation for which it is the Jacobi angle
    assert off < 1e-15 and spread > abs(a - d)


def test_equal_diagonal_needs_no_rotation():
    sig = _spd(16, 3)
    q0, s0, _ = O.givens_equalize(sig, 1e-13)
    q, s, n = O.givens_equalize(s0, 1e-10)
    assert n == 0 and np.array_equal(q, np.eye(16)) and np.array_equal(s, s0)


def test_block_covariance_against_loops():
    g = np.random.default_rng(5)
    xb = I.to_bf16_bits(g.standard_normal((3, 64)).astype(np.float32))
    x = O.decode_bf16(xb)
    want = np.zeros((2, 2))
    for t in range(3):
        for k in range(32):
            for b in range(2):
                for b2 in range(2):
                    want[b, b2] += x[t, 32 * b + k] * x[t, 32 * b2 + k]
    want /= 3 * 32
    assert np.allclose(O.block_covariance(xb), want, rtol=1e-13, atol=0)
    assert np.allclose(np.diagonal(O.block_covariance(xb)), O.block_variances(x), rtol=1e-13)


def test_calibrated_rotation_flattens_block_variances_and_lowers_the_quantization_error():
    """The claim of Section 5.1 on synthetic activations with outlier channels: after Y = R_B X the block
    variances are equal, the block maxima (hence the shared scales) drop, and the MXFP4 error with them."""
    cfg = I.CONFIGS["tiny"]
    xb = I.activations(cfg, M=128, d=1024)                # 4 outlier channels x50
    x = O.decode_bf16(xb)
    sig = O.block_covariance(xb)
    c = np.trace(sig) / sig.shape[0]
    q, _, _ = O.givens_equalize(sig, 1e-10 * c)
    rb = I.to_bf16_bits(q.astype(np.float32))
    z = O.rotate_structured(xb, rb, None)
    v0, v1 = O.block_variances(x), O.block_variances(z)
    assert v0.max() / v0.min() > 50                       # outlier blocks dominate before
    assert v1.max() / v1.min() < 1.05                     # flat after (bf16 rounding of R_B leaves ~1e-2)

    def mse(a):
        codes, sb = O.quantize_mxfp4(a.astype(np.float32))
        return ((O.dequantize(codes, sb) - a) ** 2).mean()

    assert mse(z) < 0.95 * mse(x)                         # about 10 % lower on this input (inter-block step alone)
