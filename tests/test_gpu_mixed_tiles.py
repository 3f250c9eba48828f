"""GPU parity of the CTA-pair kernels on shapes whose tile list mixes 256- and 192-column tiles (the
last wave is dealt as narrower tiles where 256-column tiles would leave it partly empty).  A narrow
tile starts on a multiple of 64 columns, so half of them start in the middle of a 4-byte group of scale
bytes (rotation) or 64 rows into a 128-row scale chunk of W (GEMM): the shapes below contain both
kinds, and every case first checks that its tile list really has narrow tiles on this device.
Bounds as in every other parity test."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import dev_bf16, dev_u8, gpu_quantized_to_numpy, mismatch_report
from paper_2605_19561_b200 import inputs as I
from paper_2605_19561_b200 import torq
import test_gpu_mxint4 as TI
import test_gpu_nvfp4 as TN

pytestmark = pytest.mark.gpu


def _pairs():
    return torch.cuda.get_device_properties(0).multi_processor_count // 2


def _narrow_starts(rows, cols):
    tl = torq.torq_pair_tile_list(rows, cols, _pairs())
    return sorted({c0 % 128 for _, c0, w in tl if w == 192})


# (rows, cols) with both kinds of narrow tiles on 74 pairs: 3840 x 1280 -> 72 wide + 4 narrow (columns 512, 704,
# 896, 1088), 4864 x 1024 -> 73 + 4 (one row tile: 256, 448, 640, 832), 2500 x 2048 -> 74 + 8 with a ragged last
# row tile; 6400 x 768 -> 72 + 4, where the one row tile that trades has no 256-column tile left at all
SHAPES = [(3840, 1280), (4864, 1024), (2500, 2048), (6400, 768)]


def _rand_rotation(d, seed):
    g = np.random.default_rng(seed)
    return I.to_bf16_bits(I.orthogonal(d, g)) if d <= 1024 else I.to_bf16_bits(g.standard_normal((d, d)) / np.sqrt(d))


@pytest.mark.parametrize("M,d", SHAPES)
def test_rotation_mxfp4(M, d):
    if _pairs() == 74:
        assert _narrow_starts(M, d) == [0, 64]
    g = np.random.default_rng(M + d)
    xb = I.to_bf16_bits(g.standard_t(3.0, size=(M, d)))
    rb = _rand_rotation(d, d)
    rib = I.to_bf16_bits(I.orthogonal(32, g, batch=d // 32))
    for intra in (rib, None):
        codes_t = torch.full((M, d // 2), 0xEE, dtype=torch.uint8, device="cuda")
        scales_t = torch.full((torq.torq_scales_bytes(M, d),), 0xEE, dtype=torch.uint8, device="cuda")
        torq.torq_rotate_quantize(dev_bf16(xb), dev_bf16(rb), None if intra is None else dev_bf16(intra),
                                  out_codes=codes_t, out_scales=scales_t)
        torch.cuda.synchronize()
        assert torq.torq_last_device_error() == 0
        g_codes, g_sb = gpu_quantized_to_numpy(codes_t, scales_t, M, d)
        o_codes, o_sb = O.quantize_mxfp4(O.round_to_f32(O.rotate(xb, rb, intra)))
        rep = mismatch_report(g_codes, g_sb, o_codes, o_sb)
        assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
        assert rep["elem_mismatch_frac"] <= 1e-4 and rep["block_scale_mismatch_frac"] <= 1e-4, rep
        # every byte of the scale buffer was written: real rows hold scales, padding rows zero
        raw = scales_t.cpu().numpy().copy()
        rr, cc = np.meshgrid(np.arange(M), np.arange(d // 32), indexing="ij")
        raw[O.scale_layout_offset(rr, cc, d)] = 0
        assert not raw.any()


def test_rotation_exact_case_is_bit_exact():
    """Permutations of small integers: every partial sum is exact, so codes and scales equal the oracle's
    bit for bit whichever tile computed them."""
    M, d = 3840, 1280
    g = np.random.default_rng(3)
    xb = I.to_bf16_bits(g.integers(-8, 9, size=(M, d)).astype(np.float64))
    P = np.zeros((d, d))
    P[np.arange(d), g.permutation(d)] = 1.0
    pin = np.stack([np.eye(32)[g.permutation(32)] for _ in range(d // 32)])
    for rib in (I.to_bf16_bits(pin), None):
        codes_t, scales_t = torq.torq_rotate_quantize(dev_bf16(xb), dev_bf16(I.to_bf16_bits(P)),
                                                      None if rib is None else dev_bf16(rib))
        torch.cuda.synchronize()
        g_codes, g_sb = gpu_quantized_to_numpy(codes_t, scales_t, M, d)
        o_codes, o_sb = O.quantize_mxfp4(O.round_to_f32(O.rotate(xb, I.to_bf16_bits(P), rib)))
        assert np.array_equal(g_sb, o_sb) and np.array_equal(g_codes, o_codes)
    assert torq.torq_last_device_error() == 0


def test_rotation_nvfp4_and_mxint4():
    M, d = 3840, 1280
    cfg = I.CONFIGS["tiny"]
    xb = I.activations(cfg, M=M, d=d)
    rb = _rand_rotation(d, 5)
    TN._rotate_case(xb, rb, I.intra_rotations16(cfg, d=d))
    TN._rotate_case(xb, rb, None)
    g = np.random.default_rng(6)
    TI._rotate_case(xb, rb, I.to_bf16_bits(I.orthogonal(32, g, batch=d // 32)))
    TI._rotate_case(xb, rb, None)


def test_weight_preparation_takes_narrow_tiles_with_the_float_output():
    """The offline weight side runs the same kernel with a float32 output and three bf16 terms per weight."""
    d, N = 1280, 3840
    cfg = I.CONFIGS["tiny"]
    if _pairs() == 74:
        assert _narrow_starts(N, d) == [0, 64]
    rb, rib, _, _ = I.rotations(cfg, d=d)
    w = I.weights(cfg, d=d, N=N)
    Wq, Ws = torq.torq_prepare_weights(dev_bf16(rb), dev_bf16(rib), torch.from_numpy(w).cuda())
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    g_codes, g_sb = gpu_quantized_to_numpy(Wq, Ws, N, d)
    o_codes, o_sb = O.prepare_weights(rb, rib, w)
    rep = mismatch_report(g_codes, g_sb, o_codes, o_sb)
    assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
    assert rep["elem_mismatch_frac"] <= 1e-4 and rep["block_scale_mismatch_frac"] <= 1e-4, rep


# ------------------------------------------------------------------------------------- GEMM
def _rand_operand(rows, k, seed, lo=118, hi=134):
    g = np.random.default_rng(seed)
    return g.integers(0, 16, size=(rows, k), dtype=np.uint8), g.integers(lo, hi, size=(rows, k // 32), dtype=np.uint8)


def _gpu_gemm(ac, asb, wc, wsb, out_dtype):
    K = ac.shape[1]
    y = torq.torq_mxfp4_gemm(dev_u8(O.pack_codes(ac)), dev_u8(O.swizzle_scales(asb, K, fill=0)),
                             dev_u8(O.pack_codes(wc)), dev_u8(O.swizzle_scales(wsb, K, fill=0)), out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    return y.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("M,N,K", [(3840, 1280, 512), (4864, 1024, 384), (2500, 2048, 256), (6400, 768, 256)])
def test_gemm_mxfp4(M, N, K):
    if _pairs() == 74:
        assert _narrow_starts(M, N) == [0, 64]
    ac, asb = _rand_operand(M, K, 1)
    wc, wsb = _rand_operand(N, K, 2)
    ref = O.gemm_dequant(ac, asb, wc, wsb)
    got = _gpu_gemm(ac, asb, wc, wsb, torch.float32)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5
    gotb = _gpu_gemm(ac, asb, wc, wsb, torch.bfloat16)
    assert np.array_equal(gotb, O.round_to_bf16(got))


def test_gemm_exact_regime_and_one_hot_rows():
    """Equal scales: bit-exact.  One-hot activation rows return single dequantized weight columns, so a weight
    row paired with another row's scale (the narrow tiles read their W scales at an offset) shows exactly."""
    M, N, K = 3840, 1280, 256
    ac, _ = _rand_operand(M, K, 3)
    wc, _ = _rand_operand(N, K, 4)
    asb = np.full((M, K // 32), 127, np.uint8)
    wsb = np.full((N, K // 32), 127, np.uint8)
    assert (_gpu_gemm(ac, asb, wc, wsb, torch.float32) == O.gemm_dequant(ac, asb, wc, wsb)).all()
    g = np.random.default_rng(9)
    wc, wsb = _rand_operand(N, K, 5)
    ac = np.zeros((M, K), np.uint8)
    asb = g.integers(120, 131, size=(M, K // 32), dtype=np.uint8)
    ac[np.arange(M), g.integers(0, K, size=M)] = 2           # codeword 1.0
    assert (_gpu_gemm(ac, asb, wc, wsb, torch.float32) == O.gemm_dequant(ac, asb, wc, wsb)).all()


def test_gemm_nvfp4_and_mxint4():
    M, N, K = 3840, 1280, 512
    ac, asb = TN._rand_operand(M, K, 1)
    wc, wsb = TN._rand_operand(N, K, 2)
    ats, wts = np.float32(0.013), np.float32(2.5e-4)
    ref = O.gemm_nvfp4(ac, asb, ats, wc, wsb, wts)
    got = TN._gpu_gemm(ac, asb, ats, wc, wsb, wts, torch.float32)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5
    aq, asb = TI._rand_operand(M, K, 3)
    wq, wsb = TI._rand_operand(N, K, 4)
    ref = O.gemm_mxint4(aq, asb, wq, wsb)
    got = TI._gpu_gemm(aq, asb, wq, wsb, torch.float32)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5
