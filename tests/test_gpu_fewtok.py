"""GPU parity of the few-token kernels (rotation up to 256 tokens, GEMM up to 128; the regime where the layer
streams R_inter and W from HBM once): the rotation that splits its contraction over a cluster and reduces the
partial sums through distributed shared memory, and the GEMM built the same way, against the oracle.
Same bounds as everywhere else: rotate + quantize at most 1e-4 of the elements one lattice step off
and 1e-4 of the block scales one step off (one element / block at sizes where 1e-4 is less than
one); GEMM <= 1e-5 relative Frobenius error in fp32, bit-exact where fp32 accumulation is exact."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import dev_bf16, dev_u8, gpu_quantized_to_numpy, lattice, mismatch_report
from paper_2605_19561_b200 import inputs as I
from paper_2605_19561_b200 import torq

pytestmark = pytest.mark.gpu


def _rand_rotation(d, seed):
    """Any well-scaled matrix serves parity (orthogonality is not used by the path); QR only when cheap."""
    g = np.random.default_rng(seed)
    if d <= 1024:
        return I.to_bf16_bits(I.orthogonal(d, g))
    return I.to_bf16_bits(g.standard_normal((d, d)) / np.sqrt(d))


# cluster sizes reached on 148 SMs: d = 128 -> 1, 256 -> 2, 640 -> 5, 1536 -> 8, 2560 -> 7, 4096 -> 4, 5120 -> 3
@pytest.mark.parametrize("M,d", [(1, 128), (16, 256), (17, 256), (32, 640), (33, 640), (64, 1536), (5, 2560),
                                 (48, 4096), (1, 5120), (64, 5120),
                                 # 128 and 256 tokens per instruction (one CTA per SM), two row tiles of scales
                                 (65, 256), (100, 1536), (128, 640), (129, 256), (200, 5120), (256, 2560), (130, 4096)])
def test_rotation_alone_without_any_workspace(M, d):
    g = np.random.default_rng(1000 * M + d)
    xb = I.to_bf16_bits(g.standard_t(3.0, size=(M, d)))
    rb = _rand_rotation(d, d)
    rib = I.to_bf16_bits(I.orthogonal(32, g, batch=d // 32))
    for intra in (rib, None):
        codes_t = torch.full((M, d // 2), 0xEE, dtype=torch.uint8, device="cuda")
        scales_t = torch.full((torq.torq_scales_bytes(M, d),), 0xEE, dtype=torch.uint8, device="cuda")
        before = torq.torq_launch_count()
        torq.torq_rotate_quantize(dev_bf16(xb), dev_bf16(rb), None if intra is None else dev_bf16(intra),
                                  out_codes=codes_t, out_scales=scales_t)
        torch.cuda.synchronize()
        assert torq.torq_launch_count() - before == 1
        assert torq.torq_last_device_error() == 0
        g_codes, g_sb = gpu_quantized_to_numpy(codes_t, scales_t, M, d)
        o_codes, o_sb = O.quantize_mxfp4(O.round_to_f32(O.rotate(xb, rb, intra)))
        rep = mismatch_report(g_codes, g_sb, o_codes, o_sb)
        assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
        assert rep["elem_mismatch_frac"] <= max(1e-4, 33.0 / g_codes.size), rep
        assert rep["block_scale_mismatch_frac"] <= max(1e-4, 1.5 / g_sb.size), rep
        # every byte of the scale buffer was written: real rows hold scales, padding rows zero
        raw = scales_t.cpu().numpy().copy()
        rr, cc = np.meshgrid(np.arange(M), np.arange(d // 32), indexing="ij")
        raw[O.scale_layout_offset(rr, cc, d)] = 0
        assert not raw.any()


def test_rotation_exact_cases_are_bit_exact():
    """Permutation and identity rotations with integer activations: every partial sum is exact in any
    order, so codes and scales must equal the oracle's bit for bit through the split and the reduction."""
    d, M = 1536, 40
    g = np.random.default_rng(7)
    x = g.integers(-8, 9, size=(M, d)).astype(np.float64)
    xb = I.to_bf16_bits(x)
    perm = g.permutation(d)
    P = np.zeros((d, d))
    P[np.arange(d), perm] = 1.0
    pin = np.stack([np.eye(32)[g.permutation(32)] for _ in range(d // 32)])
    for rb, rib in ((I.to_bf16_bits(P), I.to_bf16_bits(pin)), (I.to_bf16_bits(np.eye(d)), None)):
        codes_t, scales_t = torq.torq_rotate_quantize(dev_bf16(xb), dev_bf16(rb), None if rib is None else dev_bf16(rib))
        torch.cuda.synchronize()
        g_codes, g_sb = gpu_quantized_to_numpy(codes_t, scales_t, M, d)
        o_codes, o_sb = O.quantize_mxfp4(O.round_to_f32(O.rotate(xb, rb, rib)))
        assert np.array_equal(g_sb, o_sb) and np.array_equal(g_codes, o_codes)
    assert torq.torq_last_device_error() == 0


# ------------------------------------------------------------------------------------- GEMM
def _rand_operand(rows, k, seed, scale_lo=118, scale_hi=134):
    g = np.random.default_rng(seed)
    codes = g.integers(0, 16, size=(rows, k), dtype=np.uint8)
    sb = g.integers(scale_lo, scale_hi, size=(rows, k // 32), dtype=np.uint8)
    return codes, sb


def _gpu_gemm(ac, asb, wc, wsb, out_dtype):
    K = ac.shape[1]
    before = torq.torq_launch_count()
    y = torq.torq_mxfp4_gemm(dev_u8(O.pack_codes(ac)), dev_u8(O.swizzle_scales(asb, K, fill=0)),
                             dev_u8(O.pack_codes(wc)), dev_u8(O.swizzle_scales(wsb, K, fill=0)), out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert torq.torq_launch_count() - before == 1
    assert torq.torq_last_device_error() == 0
    return y.float().cpu().numpy().astype(np.float64)


# K = 128 (one half stage), 384 (a half last stage), 640 and 5120 (several stages per split); N ragged in the
# last 128-row tile; cluster sizes 1 .. 8
@pytest.mark.parametrize("M,N,K", [(1, 8, 128), (16, 136, 384), (17, 640, 640), (33, 2560, 1024), (64, 5120, 5120),
                                   (5, 4096, 4096), (64, 264, 2048), (40, 1000, 896),
                                   (65, 136, 384), (100, 2560, 1024), (128, 5120, 5120), (97, 1000, 896)])
def test_gemm_random_operands(M, N, K):
    ac, asb = _rand_operand(M, K, 1)
    wc, wsb = _rand_operand(N, K, 2)
    ref = O.gemm_dequant(ac, asb, wc, wsb)
    got = _gpu_gemm(ac, asb, wc, wsb, torch.float32)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5
    # bf16 output: the same fp32 sums, rounded once to nearest even
    gotb = _gpu_gemm(ac, asb, wc, wsb, torch.bfloat16)
    assert np.array_equal(gotb, O.round_to_bf16(got))
    refb = O.round_to_bf16(ref)
    assert np.linalg.norm(gotb - refb) / np.linalg.norm(refb) <= 1e-3


def test_gemm_exact_integer_regime_and_one_hot_rows():
    """Equal scales: fp32 accumulation is exact in any order and through the split, so the result is the
    oracle's bit for bit.  One-hot activation rows return single dequantized weight columns: a mix-up of
    row <-> scale or K-block <-> scale on either (swapped) side would show exactly."""
    M, N, K = 48, 400, 1536
    ac, _ = _rand_operand(M, K, 3)
    wc, _ = _rand_operand(N, K, 4)
    asb = np.full((M, K // 32), 127, np.uint8)
    wsb = np.full((N, K // 32), 127, np.uint8)
    assert (_gpu_gemm(ac, asb, wc, wsb, torch.float32) == O.gemm_dequant(ac, asb, wc, wsb)).all()
    g = np.random.default_rng(9)
    wc, wsb = _rand_operand(N, K, 5)
    ac = np.zeros((M, K), np.uint8)
    asb = g.integers(120, 131, size=(M, K // 32), dtype=np.uint8)
    hot = g.integers(0, K, size=M)
    ac[np.arange(M), hot] = 2                              # codeword 1.0
    ref = O.gemm_dequant(ac, asb, wc, wsb)
    assert (_gpu_gemm(ac, asb, wc, wsb, torch.float32) == ref).all()


def test_gemm_leaves_the_neighbours_of_its_output_alone():
    M, N, K = 20, 72, 256
    ac, asb = _rand_operand(M, K, 11)
    wc, wsb = _rand_operand(N, K, 12)
    buf = torch.full((M + 2, N), 777.0, dtype=torch.float32, device="cuda")
    Y = buf[1:M + 1]
    torq.torq_mxfp4_gemm(dev_u8(O.pack_codes(ac)), dev_u8(O.swizzle_scales(asb, K, fill=0)), dev_u8(O.pack_codes(wc)),
                         dev_u8(O.swizzle_scales(wsb, K, fill=0)), Y=Y)
    torch.cuda.synchronize()
    assert bool((buf[0] == 777.0).all()) and bool((buf[M + 1] == 777.0).all())
    ref = O.gemm_dequant(ac, asb, wc, wsb)
    assert np.linalg.norm(Y.cpu().numpy() - ref) / np.linalg.norm(ref) <= 1e-5
