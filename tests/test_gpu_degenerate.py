"""Degenerate inputs through every path of the library: all-zero activations (every block takes the
smallest scale and zero codes, the layer's output is exactly zero), a single non-zero element with
identity-like rotations (one code, one scale), and one token."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import dev_bf16, dev_u8, gpu_quantized_to_numpy
from paper_2605_19561_b200 import inputs as I
from paper_2605_19561_b200 import torq

pytestmark = pytest.mark.gpu


def _layer_operands(d, N, seed=1):
    cfg = I.CONFIGS["tiny"]
    rb, rib, _, _ = I.rotations(cfg, d=d)
    g = np.random.default_rng(seed)
    wc = g.integers(0, 16, (N, d), dtype=np.uint8)
    return rb, rib, wc, g


@pytest.mark.parametrize("M", [1, 64, 200, 300])
def test_all_zero_activations(M):
    d, N = 512, 256
    rb, rib, wc, g = _layer_operands(d, N)
    xb = np.zeros((M, d), np.uint16)
    # MXFP4, dense rotation
    wsb = g.integers(120, 131, (N, d // 32), dtype=np.uint8)
    dbg_c = torch.full((M, d // 2), 0xAA, dtype=torch.uint8, device="cuda")
    dbg_s = torch.full((torq.torq_scales_bytes(M, d),), 0xAA, dtype=torch.uint8, device="cuda")
    y = torq.torq_rotated_linear(dev_bf16(xb), dev_bf16(rb), dev_bf16(rib), dev_u8(O.pack_codes(wc)),
                                 dev_u8(O.swizzle_scales(wsb, d, fill=0)), out_dtype=torch.float32,
                                 dbg_codes=dbg_c, dbg_scales=dbg_s)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    assert not dbg_c.any() and not dbg_s.any() and not y.any()
    # NVFP4
    ri32 = torq.torq_expand_intra16(dev_bf16(I.intra_rotations16(I.CONFIGS["tiny"], d=d)))
    wsb16 = g.integers(0x30, 0x40, (N, d // 16), dtype=np.uint8)
    dbg_s2 = torch.full((torq.torq_nvfp4_scales_bytes(M, d),), 0xAA, dtype=torch.uint8, device="cuda")
    dbg_c.fill_(0xAA)
    torch.cuda.synchronize()
    y = torq.torq_rotated_linear_nvfp4(dev_bf16(xb), dev_bf16(rb), ri32, 1.0, dev_u8(O.pack_codes(wc)),
                                       dev_u8(O.nv_swizzle_scales(wsb16, d)), 0.5, out_dtype=torch.float32,
                                       dbg_codes=dbg_c, dbg_scales=dbg_s2)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    assert not dbg_c.any() and not dbg_s2.any() and not y.any()
    # structured rotation, both quantizers
    rbb = I.to_bf16_bits(I.orthogonal(d // 32, np.random.default_rng(2)))
    for fn, nbytes in ((lambda: torq.torq_rotate_quantize_structured(dev_bf16(xb), dev_bf16(rbb), dev_bf16(rib[0])),
                        torq.torq_scales_bytes(M, d)),
                       (lambda: torq.torq_rotate_quantize_structured_nvfp4(dev_bf16(xb), dev_bf16(rbb), dev_bf16(rib[0]), 1.0),
                        torq.torq_nvfp4_scales_bytes(M, d))):
        c, s = fn()
        torch.cuda.synchronize()
        assert torq.torq_last_device_error() == 0
        assert s.numel() == nbytes and not c.any() and not s.any()


def test_single_nonzero_element_with_permutation_rotations():
    """x = 3.0 at one position, a permutation matrix as the rotation: amax 3 gives e = floor(log2 3) - 2 = -1
    (scale byte 126), 3 / 2^-1 = 6 = the top codeword (index 7), at the permuted position; everything else zero."""
    M, d = 130, 256
    g = np.random.default_rng(9)
    x = np.zeros((M, d), np.float32)
    x[77, 100] = 3.0
    perm = g.permutation(d)
    P = np.zeros((d, d), np.float32); P[np.arange(d), perm] = 1
    codes_t, scales_t = torq.torq_rotate_quantize(dev_bf16(I.to_bf16_bits(x)), dev_bf16(I.to_bf16_bits(P)), None)
    torch.cuda.synchronize()
    codes, sb = gpu_quantized_to_numpy(codes_t, scales_t, M, d)
    o_codes, o_sb = O.quantize_mxfp4(O.round_to_f32(O.rotate(I.to_bf16_bits(x), I.to_bf16_bits(P), None)))
    assert np.array_equal(codes, o_codes) and np.array_equal(sb, o_sb)
    j = perm[100]
    assert codes[77, j] == 7 and sb[77, j // 32] == 126 and codes.sum() == 7 and sb.sum() == 126     # 3 = 6 * 2^-1


@pytest.mark.parametrize("M", [1, 64, 300])
def test_all_zero_activations_in_mxint4(M):
    """The MXINT4 paths on all-zero activations: zero operand bytes, zero scale bytes, zero output; through
    the dense rotation (single pass, or split for few tokens) and the structured one."""
    d, N = 512, 256
    rb, rib, _, g = _layer_operands(d, N)
    xb = np.zeros((M, d), np.uint16)
    wq = g.integers(-7, 8, (N, d)).astype(np.int8)
    wsb = g.integers(120, 131, (N, d // 32), dtype=np.uint8)
    dbg_b = torch.full((M, d), 0xAA, dtype=torch.uint8, device="cuda")
    dbg_s = torch.full((torq.torq_scales_bytes(M, d),), 0xAA, dtype=torch.uint8, device="cuda")
    y = torq.torq_rotated_linear_mxint4(dev_bf16(xb), dev_bf16(rb), dev_bf16(rib), dev_u8(O.int4_to_e4m3(wq)),
                                        dev_u8(O.swizzle_scales(wsb, d, fill=0)), out_dtype=torch.float32,
                                        dbg_bytes=dbg_b, dbg_scales=dbg_s)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    assert not (dbg_b & 0x7F).any() and not dbg_s.any() and not y.any()      # a zero may carry a sign bit
    rbb = I.to_bf16_bits(I.orthogonal(d // 32, np.random.default_rng(2)))
    c, s = torq.torq_rotate_quantize_structured_mxint4(dev_bf16(xb), dev_bf16(rbb), dev_bf16(rib[0]))
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    assert not (c & 0x7F).any() and not s.any()


def test_single_nonzero_element_in_mxint4():
    """x = 3.0 at one position through a permutation: amax 3 gives e = -1 (scale byte 126) and the code 6 at
    the permuted position (E4M3 byte 0x4C); everything else zero."""
    M, d = 130, 256
    g = np.random.default_rng(9)
    x = np.zeros((M, d), np.float32)
    x[77, 100] = 3.0
    perm = g.permutation(d)
    P = np.zeros((d, d), np.float32); P[np.arange(d), perm] = 1
    b_t, s_t = torq.torq_rotate_quantize_mxint4(dev_bf16(I.to_bf16_bits(x)), dev_bf16(I.to_bf16_bits(P)), None)
    torch.cuda.synchronize()
    b = b_t.cpu().numpy()
    sb = O.unswizzle_scales(s_t.cpu().numpy(), M, d)
    j = perm[100]
    assert b[77, j] == 0x4C and sb[77, j // 32] == 126
    b[77, j] = 0
    assert not (b & 0x7F).any() and sb.sum() == 126
