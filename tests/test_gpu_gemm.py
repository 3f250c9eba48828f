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


@pytest.mark.parametrize("M,N,K,dt", [(300, 520, 1152, torch.bfloat16), (257, 72, 128, torch.bfloat16),
                                      (1000, 264, 640, torch.float32), (129, 8, 384, torch.bfloat16),
                                      (511, 1032, 896, torch.float32), (640, 328, 1408, torch.bfloat16)])
def test_ragged_shapes_on_the_cta_pair_kernel(M, N, K, dt):
    """M > 128 runs on CTA pairs with staged TMA stores of Y: ragged M (second row tile of a pair
    missing or partial), N that ends inside a 256-column tile and inside a 64- or 32-column store
    box, K with a half last stage (K % 256 == 128)."""
    ac, asb = _rand_operand(M, K, 31)
    wc, wsb = _rand_operand(N, K, 32)
    ref = O.gemm_dequant(ac, asb, wc, wsb)
    # canary: rows and columns around Y must stay untouched
    pad = torch.full((M + 2, N + 16), 7.0, dtype=dt, device="cuda")
    Y = pad[1:M + 1, 8:N + 8]
    assert not Y.is_contiguous()
    Yc = torch.empty((M, N), dtype=dt, device="cuda")
    torq.torq_mxfp4_gemm(dev_u8(O.pack_codes(ac)), dev_u8(O.swizzle_scales(asb, K, fill=0)),
                         dev_u8(O.pack_codes(wc)), dev_u8(O.swizzle_scales(wsb, K, fill=0)), Y=Yc)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    got = Yc.float().cpu().numpy().astype(np.float64)
    want = ref if dt == torch.float32 else O.round_to_bf16(ref)
    assert np.isfinite(got).all()
    assert np.linalg.norm(got - want) / np.linalg.norm(want) <= (1e-5 if dt == torch.float32 else 1e-3)
    if dt == torch.bfloat16:
        # element-wise: one bf16 ulp of the result, plus the fp32 accumulation error, which scales with
        # the size of the terms (not of the possibly cancelled sum)
        ulp = np.ldexp(1.0, np.frexp(np.maximum(np.abs(want), 1e-30))[1] - 8)
        terms = np.abs(O.dequantize(ac, asb)) @ np.abs(O.dequantize(wc, wsb)).T
        assert (np.abs(got - want) <= ulp + 1e-6 * terms).all()


def test_output_buffer_neighbours_are_not_written():
    """Y packed between canaries in one allocation: the TMA stores clip at M rows and N columns."""
    M, N, K = 300, 520, 256
    ac, asb = _rand_operand(M, K, 41)
    wc, wsb = _rand_operand(N, K, 42)
    for dt in (torch.bfloat16, torch.float32):
        buf = torch.full((M * N + 4096,), 3.0, dtype=dt, device="cuda")
        Y = buf[2048:2048 + M * N].view(M, N)
        torq.torq_mxfp4_gemm(dev_u8(O.pack_codes(ac)), dev_u8(O.swizzle_scales(asb, K, fill=0)),
                             dev_u8(O.pack_codes(wc)), dev_u8(O.swizzle_scales(wsb, K, fill=0)), Y=Y)
        torch.cuda.synchronize()
        assert bool((buf[:2048] == 3.0).all()) and bool((buf[2048 + M * N:] == 3.0).all())
        ref = O.gemm_dequant(ac, asb, wc, wsb)
        got = Y.float().cpu().numpy().astype(np.float64)
        assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-2


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


@pytest.mark.parametrize("M,N,K,dt", [(2300, 6200, 640, torch.float32), (2048, 6144, 384, torch.bfloat16),
                                      (1100, 12296, 256, torch.float32)])
def test_several_waves_of_tiles_with_ragged_edges_and_one_hot_rows(M, N, K, dt):
    """Shapes with several waves of tiles per CTA pair (every pair walks two to four tiles, the last wave
    partly empty), ragged M and N, K with and without a half last stage.  One-hot activation rows make every
    output a single product: exact in fp32 and in bf16 after one rounding, so any mix-up of columns, rows of W,
    scale tiles or store boxes shows up exactly; random rows in between exercise the accumulation."""
    wc, wsb = _rand_operand(N, K, 21, 100, 150)
    g = np.random.default_rng(22)
    ac, asb = _rand_operand(M, K, 23, 100, 150)
    hot_rows = np.arange(0, M, 3)
    ac[hot_rows] = 0
    ac[hot_rows, g.integers(0, K, size=hot_rows.size)] = g.integers(1, 16, size=hot_rows.size).astype(np.uint8)
    ref = O.gemm_dequant(ac, asb, wc, wsb)
    got = _gpu_gemm(ac, asb, wc, wsb, dt)
    if dt == torch.bfloat16:
        ref = O.round_to_bf16(ref)
        assert (got[hot_rows] == ref[hot_rows]).all()
        assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-3
    else:
        assert (got[hot_rows] == ref[hot_rows]).all()
        assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5
