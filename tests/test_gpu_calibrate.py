"""GPU parity of the inter-block calibration (Section 5.1, Algorithm 1) against the oracle.

Covariance: float64 accumulation in a different order from the oracle's matrix product: 1e-12 relative.
Algorithm 1: both sides take the same float64 steps with one rounding per operation, so the rotation
matrix, the rotated covariance and the rotation count are compared bit for bit; the properties that
define the result (equal diagonal, orthogonality) are checked on their own as well."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import dev_bf16
from paper_2605_19561_b200 import inputs as I
from paper_2605_19561_b200 import torq

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T,d", [(128, 1024), (5, 96), (33, 4096), (128, 5120)])
def test_block_covariance(T, d):
    xb = I.activations(I.CONFIGS["tiny"], M=T, d=d)
    got = torq.torq_block_covariance(dev_bf16(xb)).cpu().numpy()
    want = O.block_covariance(xb)
    assert np.abs(got - want).max() <= 1e-12 * np.abs(want).max()
    assert np.array_equal(got, got.T)                      # same products, same order, on both sides of the diagonal


def _covariance(n, seed, outliers):
    g = np.random.default_rng(seed)
    a = g.standard_normal((n, 3 * n))
    s = a @ a.T / (3 * n)
    for k in range(outliers):
        s[k * 7 % n, :] *= 10.0
        s[:, k * 7 % n] *= 10.0
    return s


@pytest.mark.parametrize("n,outliers", [(2, 0), (8, 1), (128, 4), (160, 5), (448, 8), (600, 3)])
def test_givens_equalize_matches_the_oracle(n, outliers):
    sig = _covariance(n, 100 + n, outliers)
    c = np.trace(sig) / n
    eps = 1e-12 * c
    S = torch.from_numpy(sig.copy()).cuda()
    Q, Qb, nrot = torq.torq_givens_equalize(S, eps)
    torch.cuda.synchronize()
    q, s, rot = O.givens_equalize(sig, eps)
    gq, gs = Q.cpu().numpy(), S.cpu().numpy()
    # what defines the result
    assert np.abs(np.diagonal(gs) - c).max() <= eps
    assert np.abs(gq @ gq.T - np.eye(n)).max() <= 1e-12
    assert np.abs(gq @ sig @ gq.T - gs).max() <= 1e-11 * np.abs(sig).max()
    # and the same steps as the oracle
    assert int(nrot.item()) == rot
    assert np.array_equal(gq, q)
    assert np.array_equal(gs, s)
    want_b = I.to_bf16_bits(q.astype(np.float32))
    assert np.array_equal(Qb.view(torch.int16).cpu().numpy().view(np.uint16), want_b)


def test_equal_diagonal_returns_identity():
    S = torch.eye(64, dtype=torch.float64, device="cuda") * 3.0
    Q, _, nrot = torq.torq_givens_equalize(S, 1e-12)
    assert int(nrot.item()) == 0 and bool((Q == torch.eye(64, dtype=torch.float64, device="cuda")).all())


def test_calibrate_then_rotate_flattens_block_variances():
    """The whole calibration on the device feeding the structured rotation kernel: block variances of the
    dequantized output are flat where the input's differ by more than 50x (Section 5.1's aim)."""
    cfg = I.CONFIGS["tiny"]
    T, d = 128, 1024
    xb = I.activations(cfg, M=T, d=d)
    X = dev_bf16(xb)
    S = torq.torq_block_covariance(X)
    c = float(torch.diagonal(S).sum().item()) / (d // 32)
    _, Qb, _ = torq.torq_givens_equalize(S, 1e-10 * c)
    torch.cuda.synchronize()
    codes_t, scales_t = torq.torq_rotate_quantize_structured(X, Qb, None)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    codes = O.unpack_codes(codes_t.cpu().numpy())
    sb = O.unswizzle_scales(scales_t.cpu().numpy(), T, d)
    v_in = O.block_variances(O.decode_bf16(xb))
    v_out = O.block_variances(O.dequantize(codes, sb))
    assert v_in.max() / v_in.min() > 50
    assert v_out.max() / v_out.min() < 1.3               # 4-bit quantization noise on top of the flat variances
    # parity of the rotated, quantized activations with the oracle fed the same R_B
    rb = Qb.view(torch.int16).cpu().numpy().view(np.uint16)
    o_codes, o_sb = O.quantize_mxfp4(O.round_to_f32(O.rotate_structured(xb, rb, None)))
    same = (sb == o_sb)
    assert (~same).mean() <= 1e-4
    assert ((codes != o_codes) & np.repeat(same, 32, axis=1)).mean() <= 1e-4
