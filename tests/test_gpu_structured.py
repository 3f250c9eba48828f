"""GPU parity of the structured rotation (one B x B inter-block matrix R_B, one shared 32 x 32
R_intra: the form Section 5 / Algorithm 3 / App. A.7 of the paper describe) against the oracle's
rotate_structured followed by the oracle quantizer.  Bounds as for the dense path: at most 1e-4 of
the elements differ, each by one lattice step; scale bytes likewise; exact operands must reproduce
the oracle bit for bit."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import dev_bf16, gpu_quantized_to_numpy, mismatch_report
from paper_2605_19561_b200 import inputs as I
from paper_2605_19561_b200 import torq

pytestmark = pytest.mark.gpu


def _run(xb, rb, ri, rows=None, exact=False):
    M, d = xb.shape
    codes_t, scales_t = torq.torq_rotate_quantize_structured(dev_bf16(xb), dev_bf16(rb), None if ri is None else dev_bf16(ri))
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    g_codes, g_sb = gpu_quantized_to_numpy(codes_t, scales_t, M, d)
    rows = np.arange(M) if rows is None else np.asarray(rows)
    o_codes, o_sb = O.quantize_mxfp4(O.round_to_f32(O.rotate_structured(xb[rows], rb, ri)))
    rep = mismatch_report(g_codes[rows], g_sb[rows], o_codes, o_sb)
    if exact:
        assert (g_sb[rows] == o_sb).all() and (g_codes[rows] == o_codes).all()
    assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
    assert rep["elem_mismatch_frac"] <= max(1e-4, 1.5 / o_codes.size), rep
    assert rep["block_scale_mismatch_frac"] <= max(1e-4, 1.5 / o_sb.size), rep
    # padding rows of the scale tiles are zero
    raw = scales_t.cpu().numpy()
    for r in range(M, (M + 127) // 128 * 128, 7):
        assert raw[torq.torq_scale_offset(r, 0, d)] == 0 and raw[torq.torq_scale_offset(r, d // 32 - 1, d)] == 0
    return rep


def test_block_and_position_permutations_are_bit_exact():
    """A non-symmetric block permutation pins which side R_B multiplies from and that positions
    are untouched by it; a position permutation pins the orientation of R_intra."""
    g = np.random.default_rng(0)
    for M, nb in [(37, 8), (150, 16), (9, 160)]:
        x = g.integers(-8, 9, size=(M, nb * 32)).astype(np.float32)
        PB = np.zeros((nb, nb), np.float32); PB[np.arange(nb), g.permutation(nb)] = 1
        PK = np.zeros((32, 32), np.float32); PK[g.permutation(32), np.arange(32)] = 1
        xb = I.to_bf16_bits(x)
        _run(xb, I.to_bf16_bits(PB), I.to_bf16_bits(PK), exact=True)
        _run(xb, I.to_bf16_bits(PB), None, exact=True)
        _run(xb, I.to_bf16_bits(np.eye(nb, dtype=np.float32)), I.to_bf16_bits(PK), exact=True)


@pytest.mark.parametrize("M,d", [(1, 256), (9, 256), (64, 512), (130, 1024), (100, 4096), (33, 5120), (257, 2048)])
def test_random_orthogonal_factors(M, d):
    g = np.random.default_rng(1000 + M + d)
    cfg = I.CONFIGS["tiny"]
    xb = I.activations(cfg, M=M, d=d)
    rb = I.to_bf16_bits(I.orthogonal(d // 32, g))
    ri = I.to_bf16_bits(I.orthogonal(32, g))
    _run(xb, rb, ri)
    _run(xb, rb, None)


def test_agrees_with_the_dense_kernel_on_kronecker_operands():
    """The dense entry point fed kron(R_B^T, I_32) and the repeated R_intra computes the same
    rotation; the two GPU paths may differ only by accumulation order."""
    g = np.random.default_rng(5)
    M, nb = 200, 16
    d = nb * 32
    xb = I.activations(I.CONFIGS["tiny"], M=M, d=d)
    RB, RI = I.orthogonal(nb, g), I.orthogonal(32, g)
    rb, ri = I.to_bf16_bits(RB), I.to_bf16_bits(RI)
    dense = I.to_bf16_bits(np.kron(O.decode_bf16(rb).T, np.eye(32)))
    c1, s1 = torq.torq_rotate_quantize_structured(dev_bf16(xb), dev_bf16(rb), dev_bf16(ri))
    c2, s2 = torq.torq_rotate_quantize(dev_bf16(xb), dev_bf16(dense), dev_bf16(np.stack([ri] * nb)))
    torch.cuda.synchronize()
    a_codes, a_sb = gpu_quantized_to_numpy(c1, s1, M, d)
    b_codes, b_sb = gpu_quantized_to_numpy(c2, s2, M, d)
    rep = mismatch_report(a_codes, a_sb, b_codes, b_sb)
    assert rep["non_adjacent"] == 0 and rep["elem_mismatch_frac"] <= 2e-4, rep


def test_llama3_qkv_shape_sampled_rows():
    """M = 2048, d = 4096 (B = 128): the benchmark configuration of the structured path."""
    cfg = I.CONFIGS["llama3_8b_qkv"]
    g = np.random.default_rng(77)
    xb = I.activations(cfg)
    rb = I.to_bf16_bits(I.orthogonal(cfg.d // 32, g))
    ri = I.to_bf16_bits(I.orthogonal(32, g))
    _run(xb, rb, ri, rows=[0, 1, 7, 8, 9, 127, 128, 1023, 1024, 2040, 2046, 2047])


def test_argument_errors():
    L = torq.lib()
    import ctypes
    one = ctypes.c_void_p(16)
    assert L.torq_rotate_quantize_structured(one, None, None, 4, 256, one, one, None) == 1     # R_B required
    assert L.torq_rotate_quantize_structured(one, one, None, 4, 128, one, one, None) == 2      # d % 256 != 0
    assert L.torq_rotate_quantize_structured(one, one, None, 0, 256, one, one, None) == 2


def test_whole_layer_with_the_structured_rotation():
    """Steps 1-5 in one call.  Weights are rotated by the same operator offline (oracle, dense form
    kron(R_B^T, I) . blockdiag(R_intra)) and quantized; the GEMM is checked on the codes the GPU
    produced, and the layer output against the all-oracle result."""
    g = np.random.default_rng(11)
    M, nb, N = 200, 8, 136
    d = nb * 32
    cfg = I.CONFIGS["tiny"]
    xb = I.activations(cfg, M=M, d=d)
    rb = I.to_bf16_bits(I.orthogonal(nb, g))
    ri = I.to_bf16_bits(I.orthogonal(32, g))
    dense = I.to_bf16_bits(np.kron(O.decode_bf16(rb).T, np.eye(32)))
    w = (g.standard_normal(size=(d, N)) * 0.02).astype(np.float32)
    w_codes, w_sb = O.prepare_weights(dense, np.stack([ri] * nb), w)
    dev_u8 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint8)).cuda()
    Wq, Ws = dev_u8(O.pack_codes(w_codes)), dev_u8(O.swizzle_scales(w_sb, d, fill=0))
    dbg_c = torch.empty((M, d // 2), dtype=torch.uint8, device="cuda")
    dbg_s = torch.empty(torq.torq_scales_bytes(M, d), dtype=torch.uint8, device="cuda")
    y = torq.torq_rotated_linear_structured(dev_bf16(xb), dev_bf16(rb), dev_bf16(ri), Wq, Ws, out_dtype=torch.float32,
                                            dbg_codes=dbg_c, dbg_scales=dbg_s)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    g_codes, g_sb = gpu_quantized_to_numpy(dbg_c, dbg_s, M, d)
    o_codes, o_sb = O.quantize_mxfp4(O.round_to_f32(O.rotate_structured(xb, rb, ri)))
    rep = mismatch_report(g_codes, g_sb, o_codes, o_sb)
    assert rep["non_adjacent"] == 0 and rep["elem_mismatch_frac"] <= 1e-4, rep
    got = y.cpu().numpy().astype(np.float64)
    ref = O.gemm_dequant(g_codes, g_sb, w_codes, w_sb)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-3
    full = O.gemm_dequant(o_codes, o_sb, w_codes, w_sb)
    assert np.linalg.norm(got - full) / np.linalg.norm(full) <= 2e-2
    # and the rotated-quantized layer approximates the unrotated full-precision one (identity chain)
    exact = O.decode_bf16(xb) @ w.astype(np.float64)
    assert np.linalg.norm(got - exact) / np.linalg.norm(exact) <= 0.25
