"""GPU parity: rotate + quantize (Algorithm 3 steps 1-4) and the fused rotated linear layer
(steps 1-5) against the oracle.

Bounds (the fp32 tensor-core accumulation order differs from the oracle's fp64): at most 1e-4 of
the elements may differ, each by one step on the e2m1 lattice; at most 1e-4 of the blocks may
differ in scale, by one step; the GEMM result is compared, on the codes the GPU actually
produced, to 1e-3 relative Frobenius error."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import dev_bf16, dev_u8, gpu_quantized_to_numpy, mismatch_report
from paper_2605_19561_b200 import inputs as I
from paper_2605_19561_b200 import torq

pytestmark = pytest.mark.gpu


def _rotate_quantize_case(xb, rb, rib, check_exact=False):
    M, d = xb.shape
    codes_t, scales_t = torq.torq_rotate_quantize(dev_bf16(xb), None if rb is None else dev_bf16(rb),
                                                  None if rib is None else dev_bf16(rib))
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    g_codes, g_sb = gpu_quantized_to_numpy(codes_t, scales_t, M, d)
    o_codes, o_sb = O.quantize_mxfp4(O.round_to_f32(O.rotate(xb, rb, rib)))
    rep = mismatch_report(g_codes, g_sb, o_codes, o_sb)
    if check_exact:
        assert (g_sb == o_sb).all() and (g_codes == o_codes).all()
    assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
    assert rep["elem_mismatch_frac"] <= 1e-4, rep
    assert rep["block_scale_mismatch_frac"] <= 1e-4, rep
    return g_codes, g_sb, rep


def _hadamard(n):
    H = np.array([[1.0]])
    while H.shape[0] < n:
        H = np.block([[H, H], [H, -H]])
    return H


def test_exact_rotations_give_bit_exact_codes():
    """Permutation and Walsh-Hadamard rotations with small-integer activations: every partial
    sum is exact in fp32, so codes and scales must equal the oracle's bit for bit.  A non-symmetric
    permutation also pins the operand orientation of the tensor-core contraction."""
    d, M = 256, 150
    g = np.random.default_rng(0)
    x = g.integers(-8, 9, size=(M, d)).astype(np.float32)
    xb = I.to_bf16_bits(x)
    P = np.zeros((d, d), np.float32); P[np.arange(d), g.permutation(d)] = 1
    Q = np.zeros((d // 32, 32, 32), np.float32)
    for b in range(d // 32):
        Q[b, np.arange(32), g.permutation(32)] = 1
    _rotate_quantize_case(xb, I.to_bf16_bits(P), None, check_exact=True)
    _rotate_quantize_case(xb, I.to_bf16_bits(P), I.to_bf16_bits(Q), check_exact=True)
    _rotate_quantize_case(xb, None, I.to_bf16_bits(Q), check_exact=True)
    H = (_hadamard(d) / 16.0).astype(np.float32)
    H32 = (_hadamard(32) / 4.0).astype(np.float32)
    _rotate_quantize_case(xb, I.to_bf16_bits(H), I.to_bf16_bits(np.stack([H32] * (d // 32))), check_exact=True)


@pytest.mark.parametrize("M,d", [(64, 256), (1, 256), (130, 512), (257, 320), (100, 64), (33, 1024)])
def test_random_rotations_small_shapes(M, d):
    cfg = I.CONFIGS["tiny"]
    xb = I.activations(cfg, M=M, d=d)
    rb, rib, _, _ = I.rotations(cfg, d=d)
    _rotate_quantize_case(xb, rb, rib)
    _rotate_quantize_case(xb, rb, None)


def test_tiny_config_end_to_end():
    """Config 1: X 64x256 Student-t with 4 outlier channels, W 256x256, fp32 output."""
    cfg = I.CONFIGS["tiny"]
    xb = I.activations(cfg)
    rb, rib, _, _ = I.rotations(cfg)
    w = I.weights(cfg)
    w_codes, w_sb = O.prepare_weights(rb, rib, w)
    Wq, Ws = dev_u8(O.pack_codes(w_codes)), dev_u8(O.swizzle_scales(w_sb, cfg.d, fill=0))
    dbg_c = torch.empty((cfg.M, cfg.d // 2), dtype=torch.uint8, device="cuda")
    dbg_s = torch.empty(torq.torq_scales_bytes(cfg.M, cfg.d), dtype=torch.uint8, device="cuda")
    y = torq.torq_rotated_linear(dev_bf16(xb), dev_bf16(rb), dev_bf16(rib), Wq, Ws, out_dtype=torch.float32,
                                 dbg_codes=dbg_c, dbg_scales=dbg_s)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    g_codes, g_sb = gpu_quantized_to_numpy(dbg_c, dbg_s, cfg.M, cfg.d)
    o_out, o_codes, o_sb = O.rotated_linear(xb, rb, rib, w_codes, w_sb)
    rep = mismatch_report(g_codes, g_sb, o_codes, o_sb)
    assert rep["non_adjacent"] == 0 and rep["elem_mismatch_frac"] <= 1e-4, rep
    # GEMM parity on the operands actually fed
    ref = O.gemm_dequant(g_codes, g_sb, w_codes, w_sb)
    got = y.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-3
    # and the whole layer stays close to the all-oracle result (a few flipped codes at most)
    assert np.linalg.norm(got - o_out) / np.linalg.norm(o_out) <= 2e-2


def test_llama3_qkv_shape_sampled_rows():
    """Config 2 at full size (2048 x 4096 -> 6144): rotate+quantize checked on sampled rows that
    span several row tiles, the GEMM on the same rows, bf16 output."""
    cfg = I.CONFIGS["llama3_8b_qkv"]
    xb = I.activations(cfg)
    rb, rib, _, _ = I.rotations(cfg)
    Xd, Rd, Rid = dev_bf16(xb), dev_bf16(rb), dev_bf16(rib)
    w = I.weights(cfg)
    Wq, Ws = torq.prepare_weights(Rd, Rid, torch.from_numpy(w).cuda())
    dbg_c = torch.empty((cfg.M, cfg.d // 2), dtype=torch.uint8, device="cuda")
    dbg_s = torch.empty(torq.torq_scales_bytes(cfg.M, cfg.d), dtype=torch.uint8, device="cuda")
    y = torq.torq_rotated_linear(Xd, Rd, Rid, Wq, Ws, out_dtype=torch.bfloat16, dbg_codes=dbg_c, dbg_scales=dbg_s)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    rows = np.array([0, 1, 127, 128, 129, 640, 1023, 1024, 1777, 2046, 2047])
    g_codes = O.unpack_codes(dbg_c.cpu().numpy()[rows])
    g_sb = O.unswizzle_scales(dbg_s.cpu().numpy(), cfg.M, cfg.d)[rows]
    o_codes, o_sb = O.quantize_mxfp4(O.round_to_f32(O.rotate(xb[rows], rb, rib)))
    rep = mismatch_report(g_codes, g_sb, o_codes, o_sb)
    assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
    assert rep["elem_mismatch_frac"] <= 1e-4 and rep["block_scale_mismatch_frac"] <= 1e-4, rep
    w_codes, w_sb = gpu_quantized_to_numpy(Wq, Ws, cfg.N, cfg.d)
    ref = O.round_to_bf16(O.gemm_dequant(g_codes, g_sb, w_codes, w_sb))
    got = y.float().cpu().numpy()[rows].astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-3


@pytest.mark.parametrize("M,d", [(1, 256), (33, 256), (100, 512), (128, 1024), (64, 2048), (17, 4096),
                                 (200, 512), (384, 1024), (257, 256)])
def test_few_token_split_k_path_through_the_fused_call(M, d):
    """Few output tiles (fewer than half the SMs) through torq_rotated_linear, one or several row
    tiles: the rotation runs as split-K partial tiles plus the
    reduce/intra/quantize kernel (the workspace carries the partials).  Same bounds as the
    single-pass path, and the codes must also agree with the single-pass kernel to the same
    bounds (only the fp32 summation order differs)."""
    cfg = I.CONFIGS["tiny"]
    xb = I.activations(cfg, M=M, d=d)
    rb, rib, _, _ = I.rotations(cfg, d=d)
    N = 64
    wq, wsb = I.random_codes(N, d, seed=21)
    Wq, Ws = dev_u8(wq), dev_u8(O.swizzle_scales(wsb, d, fill=0))
    for intra in (rib, None):
        dbg_c = torch.empty((M, d // 2), dtype=torch.uint8, device="cuda")
        dbg_s = torch.empty(torq.torq_scales_bytes(M, d), dtype=torch.uint8, device="cuda")
        before = torq.torq_launch_count()
        y = torq.torq_rotated_linear(dev_bf16(xb), dev_bf16(rb), None if intra is None else dev_bf16(intra), Wq, Ws,
                                     out_dtype=torch.float32, dbg_codes=dbg_c, dbg_scales=dbg_s)
        torch.cuda.synchronize()
        # up to 256 tokens (d a multiple of 128): one rotation kernel that reduces its K splits on chip, then
        # the GEMM; above: split-K partial tiles, the reduce kernel, the GEMM
        assert torq.torq_launch_count() - before == (2 if M <= 256 and d % 128 == 0 else 3)
        assert torq.torq_last_device_error() == 0
        g_codes, g_sb = gpu_quantized_to_numpy(dbg_c, dbg_s, M, d)
        o_codes, o_sb = O.quantize_mxfp4(O.round_to_f32(O.rotate(xb, rb, intra)))
        rep = mismatch_report(g_codes, g_sb, o_codes, o_sb)
        assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
        assert rep["elem_mismatch_frac"] <= max(1e-4, 1.5 / g_codes.size), rep
        assert rep["block_scale_mismatch_frac"] <= max(1e-4, 1.5 / g_sb.size), rep
        # padding rows of the scale tiles are zero
        raw = dbg_s.cpu().numpy()
        for r in range(M, (M + 127) // 128 * 128):
            assert raw[torq.torq_scale_offset(r, 0, d)] == 0
        ref = O.gemm_dequant(g_codes, g_sb, O.unpack_codes(wq), wsb)
        got = y.cpu().numpy().astype(np.float64)
        assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-3


@pytest.mark.parametrize("M,d", [(129, 256), (255, 512), (257, 320), (300, 1024), (511, 5120), (640, 96)])
def test_ragged_shapes_on_the_cta_pair_rotation(M, d):
    """M > 128 (CTA pairs, last-tile tensor-core epilogue and fp32-FMA epilogue both exercised when a
    pair works more than one tile), d that ends inside a 256-column tile (320, 96) and M that leaves
    the pair's second row tile partial or absent."""
    cfg = I.CONFIGS["tiny"]
    xb = I.activations(cfg, M=M, d=d)
    rb, rib, _, _ = I.rotations(cfg, d=d)
    _rotate_quantize_case(xb, rb, rib)
    _rotate_quantize_case(xb, rb, None)


@pytest.mark.parametrize("M,out_dtype", [(3072, torch.bfloat16), (3001, torch.float32)])
def test_many_tokens_through_the_whole_call_equal_the_two_calls(M, out_dtype):
    """Several waves of tiles per kernel (3072 x 5120 -> 5120): the whole-layer call is the two kernels back to
    back on the workspace, so its codes, scales and output equal those of the separate calls bit for bit, also
    when called twice in a row."""
    cfg = I.CONFIGS["qwen3_32b_sweep"]
    d, N = cfg.d, 5120
    xb = I.activations(cfg, M=M)
    rb, rib, _, _ = I.rotations(cfg, device="cuda")
    X, R, Ri = dev_bf16(xb), dev_bf16(rb), dev_bf16(rib)
    g = np.random.default_rng(12)
    Wq = dev_u8(g.integers(0, 256, (N, d // 2), dtype=np.uint8))
    Ws = dev_u8(O.swizzle_scales(g.integers(120, 131, (N, d // 32), dtype=np.uint8), d, fill=0))
    dbg_c = torch.empty((M, d // 2), dtype=torch.uint8, device="cuda")
    dbg_s = torch.empty(torq.torq_scales_bytes(M, d), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    before = torq.torq_launch_count()
    y1 = torq.torq_rotated_linear(X, R, Ri, Wq, Ws, out_dtype=out_dtype, dbg_codes=dbg_c, dbg_scales=dbg_s)
    torch.cuda.synchronize()
    assert torq.torq_launch_count() - before == 2
    assert torq.torq_last_device_error() == 0
    c2, s2 = torq.torq_rotate_quantize(X, R, Ri)
    y2 = torq.torq_mxfp4_gemm(c2, s2, Wq, Ws, out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert torch.equal(dbg_c, c2) and torch.equal(dbg_s, s2) and torch.equal(y1, y2)
    y3 = torq.torq_rotated_linear(X, R, Ri, Wq, Ws, out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert torch.equal(y1, y3)
