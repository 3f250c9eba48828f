"""GPU parity: block-scaled MXFP4 GEMM (Algorithm 3 step 5) against the oracle's fp64 product of
the dequantized operands.  Bound: relative Frobenius error <= 1e-3 (fp32 output); bit-exact in
the regime where fp32 accumulation is exact."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import dev_u8
from paper_2605_19561_b200 import torq

pytestmark = pytest.mark.gpu


def _rand_operand(rows, k, seed, scale_lo=118, scale_hi=134):
    g = np.random.default_rng(seed)
    codes = g.integers(0, 16, size=(rows, k), dtype=np.uint8)
    sb = g.integers(scale_lo, scale_hi, size=(rows, k // 32), dtype=np.uint8)
    return codes, sb


def _gpu_gemm(ac, asb, wc, wsb, out_dtype):
    K = ac.shape[1]
    y = torq.torq_mxfp4_gemm(dev_u8(O.pack_codes(ac)), dev_u8(O.swizzle_scales(asb, K, fill=0)),
                             dev_u8(O.pack_codes(wc)), dev_u8(O.swizzle_scales(wsb, K, fill=0)),
                             out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    return y.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("M,N,K", [(64, 256, 256), (128, 256, 128), (1, 8, 128), (33, 24, 384),
                                   (129, 264, 512), (200, 136, 1024), (256, 512, 4096), (130, 640, 640)])
def test_random_operands_fp32_output(M, N, K):
    ac, asb = _rand_operand(M, K, 1)
    wc, wsb = _rand_operand(N, K, 2)
    ref = O.gemm_dequant(ac, asb, wc, wsb)
    got = _gpu_gemm(ac, asb, wc, wsb, torch.float32)
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert rel <= 1e-3, rel
    assert rel <= 1e-5, rel          # fp32 accumulation should do far better than the bound


def test_exact_integer_regime_is_bit_exact():
    """Equal scales on each side: every product is a multiple of 0.25, partial sums stay below
    2^24 units, so fp32 accumulation is exact whatever its order."""
    M, N, K = 160, 272, 512
    ac, _ = _rand_operand(M, K, 3)
    wc, _ = _rand_operand(N, K, 4)
    asb = np.full((M, K // 32), 127, np.uint8)
    wsb = np.full((N, K // 32), 127, np.uint8)
    ref = O.gemm_dequant(ac, asb, wc, wsb)
    got = _gpu_gemm(ac, asb, wc, wsb, torch.float32)
    assert (got == ref).all()


def test_one_hot_rows_select_weight_columns_and_scales_are_per_row_and_block():
    """A one-hot activation row with value 1.0 returns one dequantized weight column: any mix-up
    of row<->scale or K-block<->scale assignment on either side shows up exactly."""
    M, N, K = 128, 256, 1024
    wc, wsb = _rand_operand(N, K, 5, 100, 150)
    g = np.random.default_rng(6)
    ac = np.zeros((M, K), np.uint8)
    hot = g.integers(0, K, size=M)
    ac[np.arange(M), hot] = 2
    asb = g.integers(100, 150, size=(M, K // 32)).astype(np.uint8)
    ref = O.gemm_dequant(ac, asb, wc, wsb)
    got = _gpu_gemm(ac, asb, wc, wsb, torch.float32)
    assert (got == ref).all()


def test_bf16_output_is_the_rounded_fp32_result():
    M, N, K = 96, 320, 768
    ac, asb = _rand_operand(M, K, 7)
    wc, wsb = _rand_operand(N, K, 8)
    ref = O.gemm_dequant(ac, asb, wc, wsb)
    got = _gpu_gemm(ac, asb, wc, wsb, torch.bfloat16)
    want = O.round_to_bf16(ref)
    # every element within one bf16 ulp of the rounded oracle value, almost all identical
    ulp = np.ldexp(1.0, np.frexp(np.maximum(np.abs(want), 1e-30))[1] - 8)
    assert (np.abs(got - want) <= ulp).all()
    assert (got == want).mean() > 0.99
    assert np.linalg.norm(got - want) / np.linalg.norm(want) <= 1e-3


def test_full_size_sampled_outputs_llama3_qkv_shape():
    """Benchmark size (M=2048, K=4096, N=6144, bf16 out): sampled rows/columns against the oracle."""
    M, N, K = 2048, 6144, 4096
    ac, asb = _rand_operand(M, K, 9, 120, 131)
    wc, wsb = _rand_operand(N, K, 10, 120, 131)
    y = torq.torq_mxfp4_gemm(dev_u8(O.pack_codes(ac)), dev_u8(O.swizzle_scales(asb, K, fill=0)),
                             dev_u8(O.pack_codes(wc)), dev_u8(O.swizzle_scales(wsb, K, fill=0)),
                             out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    rows = np.array([0, 127, 128, 1000, 2047])
    cols = np.array([0, 255, 256, 3000, 6143])
    ref = O.gemm_dequant(ac[rows], asb[rows], wc, wsb)
    got = y.cpu().numpy()[rows].astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5
    ref2 = O.gemm_dequant(ac, asb, wc[cols], wsb[cols])
    got2 = y.cpu().numpy()[:, cols].astype(np.float64)
    assert np.linalg.norm(got2 - ref2) / np.linalg.norm(ref2) <= 1e-5


def test_fp4_peak_probe_reports_a_plausible_rate():
    """The measurement tool behind the GEMM's roofline denominator: finite, positive, and not above
    what the instruction can do at the maximum clock (about 9.3 PFLOP/s on 148 SMs at 1965 MHz)."""
    rate = torq.torq_probe_fp4_peak(20000)
    assert torq.torq_last_device_error() == 0
    assert 1000.0 < rate < 9500.0, rate
