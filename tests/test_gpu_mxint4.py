"""GPU parity of the MXINT4 variant (format study of Section 6) against the oracle: quantizer and
nibble -> operand-byte expansion bit for bit; GEMM bit for bit where fp32 accumulation is exact and
to 1e-5 relative Frobenius error otherwise; rotate + quantize with at most 1e-4 of the elements one
integer step off and at most 1e-4 of the block scales one step off (the fp32 tensor-core
accumulation order differs from the oracle's fp64)."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import dev_bf16, dev_u8
from paper_2605_19561_b200 import inputs as I
from paper_2605_19561_b200 import torq

pytestmark = pytest.mark.gpu


def _operand_to_int(bytes_t):
    return O.e4m3_to_int4(bytes_t.cpu().numpy())


# ----------------------------------------------------------------------------- quantizer
@pytest.mark.parametrize("M,d", [(64, 256), (1, 32), (130, 96), (257, 1056), (128, 128), (300, 4096)])
def test_quantizer_fp32_input_is_bit_exact_in_both_forms(M, d):
    g = np.random.default_rng(M * 1000 + d)
    z = (g.standard_t(3, size=(M, d)) * np.exp(g.uniform(-30, 30, size=(M, 1)))).astype(np.float32)
    z[0, :32] = 0.0                                       # an all-zero block
    if M > 2:
        z[2, :32] = 1e-42                                 # subnormal block: the scale clamps at 2^-127
    zt = torch.from_numpy(z).cuda()
    nib_t, s1 = torq.torq_quantize_mxint4(zt, packed=True)
    byt_t, s2 = torq.torq_quantize_mxint4(zt, packed=False)
    torch.cuda.synchronize()
    o_q, o_sb = O.quantize_mxint4(z)
    assert np.array_equal(O.unswizzle_scales(s1.cpu().numpy(), M, d), o_sb)
    assert np.array_equal(s1.cpu().numpy(), s2.cpu().numpy())
    assert np.array_equal(nib_t.cpu().numpy(), O.pack_int4(o_q))
    assert np.array_equal(_operand_to_int(byt_t), o_q)
    # the operand bytes are the E4M3 bytes of the integers, up to the sign bit of a zero
    want = O.int4_to_e4m3(o_q)
    got = byt_t.cpu().numpy()
    assert np.array_equal(got & 0x7F, want & 0x7F) and np.array_equal(got[o_q != 0], want[o_q != 0])
    # padding bytes of the tiled scale buffer are zero
    buf = s1.cpu().numpy().copy()
    rr, cc = np.meshgrid(np.arange(M), np.arange(d // 32), indexing="ij")
    buf[O.scale_layout_offset(rr, cc, d)] = 0
    assert not buf.any()


def test_quantizer_ties_saturation_and_bf16_input():
    """Every half-integer and its float32 neighbours in units of the block scale, at several scales."""
    pts = np.arange(0.5, 8.0, 1.0, dtype=np.float32)
    near = np.concatenate([pts, np.nextafter(pts, np.float32(0)), np.nextafter(pts, np.float32(9))])
    vals = np.concatenate([near, -near, [7.75, 0.0]]).astype(np.float32)          # 7.75 fixes e = 0
    rows = []
    for sh in (-20, -3, 0, 5, 40):
        for start in range(0, vals.size, 31):
            blk = np.zeros(32, np.float32)
            part = vals[start:start + 31]
            blk[:part.size] = part
            blk[31] = 7.75
            rows.append(np.ldexp(blk, sh))
    z = np.stack(rows).astype(np.float32)
    byt_t, s = torq.torq_quantize_mxint4(torch.from_numpy(z).cuda())
    torch.cuda.synchronize()
    o_q, o_sb = O.quantize_mxint4(z)
    assert np.array_equal(_operand_to_int(byt_t), o_q)
    assert np.array_equal(O.unswizzle_scales(s.cpu().numpy(), z.shape[0], 32), o_sb)
    zb = I.to_bf16_bits(np.random.default_rng(5).standard_normal((96, 512)).astype(np.float32))
    byt_t, s = torq.torq_quantize_mxint4(dev_bf16(zb))
    torch.cuda.synchronize()
    o_q, o_sb = O.quantize_mxint4(O.decode_bf16(zb).astype(np.float32))
    assert np.array_equal(_operand_to_int(byt_t), o_q)
    assert np.array_equal(O.unswizzle_scales(s.cpu().numpy(), 96, 512), o_sb)


def test_expand_covers_every_nibble():
    g = np.random.default_rng(1)
    q = g.integers(-8, 8, size=(70, 160)).astype(np.int8)
    q[0, :16] = np.arange(-8, 8)
    got = torq.torq_mxint4_expand(dev_u8(O.pack_int4(q)))
    torch.cuda.synchronize()
    assert np.array_equal(got.cpu().numpy(), O.int4_to_e4m3(q))


# ---------------------------------------------------------------------------------- GEMM
def _rand_operand(rows, k, seed, lo=117, hi=137):
    g = np.random.default_rng(seed)
    q = g.integers(-7, 8, size=(rows, k)).astype(np.int8)
    sb = g.integers(lo, hi, size=(rows, k // 32), dtype=np.uint8)
    return q, sb


def _gpu_gemm(aq, asb, wq, wsb, out_dtype):
    K = aq.shape[1]
    y = torq.torq_mxint4_gemm(dev_u8(O.int4_to_e4m3(aq)), dev_u8(O.swizzle_scales(asb, K, fill=0)),
                              dev_u8(O.int4_to_e4m3(wq)), dev_u8(O.swizzle_scales(wsb, K, fill=0)), out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    return y.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("M,N,K", [(64, 256, 256), (128, 256, 128), (1, 8, 128), (33, 24, 384), (129, 264, 512),
                                   (200, 136, 1024), (256, 512, 4096), (130, 640, 640), (511, 1032, 896),
                                   (300, 520, 1152), (700, 1280, 2048)])
def test_gemm_random_operands_fp32_output(M, N, K):
    aq, asb = _rand_operand(M, K, 1)
    wq, wsb = _rand_operand(N, K, 2)
    ref = O.gemm_mxint4(aq, asb, wq, wsb)
    got = _gpu_gemm(aq, asb, wq, wsb, torch.float32)
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert rel <= 1e-5, rel


def test_gemm_exact_regime_is_bit_exact():
    """Scale bytes 126..128 on both sides: every product is an integer multiple of 2^-2 and the sums
    stay below 2^24 units, so fp32 accumulation is exact whatever its order."""
    for M, N, K in ((160, 272, 512), (384, 512, 1024)):       # one-CTA kernel and CTA-pair kernel
        aq, asb = _rand_operand(M, K, 3, 126, 129)
        wq, wsb = _rand_operand(N, K, 4, 126, 129)
        ref = O.gemm_mxint4(aq, asb, wq, wsb)
        got = _gpu_gemm(aq, asb, wq, wsb, torch.float32)
        assert (got == ref).all()


@pytest.mark.parametrize("M", [128, 256, 384])
def test_gemm_one_hot_rows_pin_the_scale_assignment(M):
    """A one-hot activation row returns one dequantized weight element times the row's own block scale:
    any mix-up of row <-> scale or K-block <-> scale byte on either side, in either kernel (one CTA:
    M <= 128 and M = 256 with this few column tiles; CTA pair: M = 384), shows up exactly."""
    N, K = 256, 1024
    g = np.random.default_rng(5 + M)
    wq = g.integers(-7, 8, (N, K)).astype(np.int8)
    wsb = g.integers(90, 165, (N, K // 32), dtype=np.uint8)
    aq = np.zeros((M, K), np.int8)
    hot = g.integers(0, K, size=M)
    aq[np.arange(M), hot] = g.choice(np.array([-7, -3, 1, 5], np.int8), size=M)
    asb = g.integers(90, 165, (M, K // 32), dtype=np.uint8)
    ref = O.gemm_mxint4(aq, asb, wq, wsb)
    got = _gpu_gemm(aq, asb, wq, wsb, torch.float32)
    assert (got == ref).all()


def test_gemm_bf16_output_and_untouched_neighbours():
    M, N, K = 300, 520, 768
    aq, asb = _rand_operand(M, K, 7)
    wq, wsb = _rand_operand(N, K, 8)
    buf = torch.full((M * N + 4096,), 3.0, dtype=torch.bfloat16, device="cuda")
    Y = buf[2048:2048 + M * N].view(M, N)
    torq.torq_mxint4_gemm(dev_u8(O.int4_to_e4m3(aq)), dev_u8(O.swizzle_scales(asb, K, fill=0)),
                          dev_u8(O.int4_to_e4m3(wq)), dev_u8(O.swizzle_scales(wsb, K, fill=0)), Y=Y)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    assert bool((buf[:2048] == 3.0).all()) and bool((buf[2048 + M * N:] == 3.0).all())
    want = O.round_to_bf16(O.gemm_mxint4(aq, asb, wq, wsb))
    got = Y.float().cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - want) / np.linalg.norm(want) <= 1e-3
    assert (got == want).mean() > 0.99


def test_gemm_full_size_sampled_outputs_llama3_qkv_shape():
    M, N, K = 2048, 6144, 4096
    aq, asb = _rand_operand(M, K, 9, 120, 134)
    wq, wsb = _rand_operand(N, K, 10, 120, 134)
    y = torq.torq_mxint4_gemm(dev_u8(O.int4_to_e4m3(aq)), dev_u8(O.swizzle_scales(asb, K, fill=0)),
                              dev_u8(O.int4_to_e4m3(wq)), dev_u8(O.swizzle_scales(wsb, K, fill=0)),
                              out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    rows = np.array([0, 127, 128, 1000, 2047])
    cols = np.array([0, 255, 256, 3000, 6143])
    yn = y.cpu().numpy().astype(np.float64)
    ref = O.gemm_mxint4(aq[rows], asb[rows], wq, wsb)
    assert np.linalg.norm(yn[rows] - ref) / np.linalg.norm(ref) <= 1e-5
    ref2 = O.gemm_mxint4(aq, asb, wq[cols], wsb[cols])
    assert np.linalg.norm(yn[:, cols] - ref2) / np.linalg.norm(ref2) <= 1e-5


# ------------------------------------------------------------------ rotation + quantizer
def _mismatch(g_q, g_sb, o_q, o_sb):
    M, d = o_q.shape
    same = g_sb == o_sb
    same_e = np.repeat(same, 32, axis=1)
    diff = (g_q != o_q) & same_e
    bad = int((diff & (np.abs(g_q.astype(np.int64) - o_q) > 1)).sum())
    step = np.abs(g_sb.astype(np.int64) - o_sb.astype(np.int64))
    if (~same).any():                                     # neighbouring scales: values within one coarse step
        dg, do = O.dequantize_mxint4(g_q, g_sb), O.dequantize_mxint4(o_q, o_sb)
        coarse = np.ldexp(1.0, np.maximum(g_sb, o_sb).astype(np.int64) - 127)
        bad += int(((np.abs(dg - do) > np.repeat(coarse, 32, axis=1)) & ~same_e).sum())
    return {"elem": float(diff.sum()) / (M * d), "blocks": float((~same).sum()) / same.size,
            "non_adjacent": bad, "scale_off_by_more_than_one": int((step > 1).sum())}


def _rotate_case(xb, rb, rib, exact=False):
    M, d = xb.shape
    byt_t, s_t = torq.torq_rotate_quantize_mxint4(dev_bf16(xb), dev_bf16(rb), None if rib is None else dev_bf16(rib))
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    g_q, g_sb = _operand_to_int(byt_t), O.unswizzle_scales(s_t.cpu().numpy(), M, d)
    o_q, o_sb = O.quantize_mxint4(O.round_to_f32(O.rotate(xb, rb, rib)))
    if exact:
        assert np.array_equal(g_sb, o_sb) and np.array_equal(g_q, o_q)
    rep = _mismatch(g_q, g_sb, o_q, o_sb)
    assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
    assert rep["elem"] * M * d <= max(2, 1e-4 * M * d) and rep["blocks"] * M * (d // 32) <= max(1, 1e-4 * M * (d // 32)), rep
    # padding of the scale tiles is zero
    buf = s_t.cpu().numpy().copy()
    rr, cc = np.meshgrid(np.arange(M), np.arange(d // 32), indexing="ij")
    buf[O.scale_layout_offset(rr, cc, d)] = 0
    assert not buf.any()
    return rep


def test_rotation_exact_cases_are_bit_exact():
    """Permutations (inter and intra) of small-integer activations: every partial sum is exact in fp32."""
    g = np.random.default_rng(0)
    for M, d in ((150, 256), (300, 512), (520, 768)):     # one-CTA kernel, CTA-pair kernel (both epilogue forms)
        x = g.integers(-9, 10, size=(M, d)).astype(np.float32) * 0.5
        P = np.zeros((d, d), np.float32); P[np.arange(d), g.permutation(d)] = 1
        Q = np.zeros((d // 32, 32, 32), np.float32)
        for b in range(d // 32):
            Q[b, np.arange(32), g.permutation(32)] = 1
        _rotate_case(I.to_bf16_bits(x), I.to_bf16_bits(P), None, exact=True)
        _rotate_case(I.to_bf16_bits(x), I.to_bf16_bits(P), I.to_bf16_bits(Q), exact=True)


@pytest.mark.parametrize("M,d", [(64, 256), (1, 256), (130, 512), (257, 320), (100, 64), (400, 1024), (1000, 768)])
def test_rotation_random_small_shapes(M, d):
    cfg = I.CONFIGS["tiny"]
    xb = I.activations(cfg, M=M, d=d)
    rb, rib, _, _ = I.rotations(cfg, d=d)
    _rotate_case(xb, rb, rib)
    _rotate_case(xb, rb, None)


@pytest.mark.parametrize("M", [64, 600])
def test_rotated_linear_end_to_end(M):
    cfg = I.CONFIGS["tiny"]
    d, N = 512, 384
    xb = I.activations(cfg, M=M, d=d)
    rb, rib, _, _ = I.rotations(cfg, d=d)
    w = I.weights(cfg, d=d, N=N)
    w_q, w_sb = O.prepare_weights_mxint4(rb, rib, w)
    dbg_b = torch.empty((M, d), dtype=torch.uint8, device="cuda")
    dbg_s = torch.empty(torq.torq_scales_bytes(M, d), dtype=torch.uint8, device="cuda")
    n0 = torq.torq_launch_count()
    y = torq.torq_rotated_linear_mxint4(dev_bf16(xb), dev_bf16(rb), dev_bf16(rib), dev_u8(O.int4_to_e4m3(w_q)),
                                        dev_u8(O.swizzle_scales(w_sb, d, fill=0)), out_dtype=torch.float32,
                                        dbg_bytes=dbg_b, dbg_scales=dbg_s)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    assert torq.torq_launch_count() - n0 == (2 if M <= 256 else 3)   # few tiles: the rotation is split along its contraction
    g_q, g_sb = _operand_to_int(dbg_b), O.unswizzle_scales(dbg_s.cpu().numpy(), M, d)
    o_out, o_q, o_sb = O.rotated_linear_mxint4(xb, rb, rib, w_q, w_sb)
    rep = _mismatch(g_q, g_sb, o_q, o_sb)
    assert rep["non_adjacent"] == 0 and rep["elem"] <= 1e-4 and rep["blocks"] <= 1e-4, rep
    ref = O.gemm_mxint4(g_q, g_sb, w_q, w_sb)             # the GEMM on the codes the GPU produced
    got = y.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5
    assert np.linalg.norm(got - o_out) / np.linalg.norm(o_out) <= 2e-2
    exact = O.decode_bf16(xb) @ w                         # the layer approximates x W (two 4-bit operands)
    assert np.linalg.norm(got - exact) / np.linalg.norm(exact) < 0.25


@pytest.mark.parametrize("M,intra", [(1, True), (33, True), (128, True), (40, False)])
def test_rotated_linear_few_tokens_takes_the_split_rotation(M, intra):
    """Few tokens: the rotation is split along its contraction over the SMs.  Up to 64 tokens one kernel
    reduces the splits through distributed shared memory; above, the partial sums go through the workspace
    and a second kernel adds them, rotates inside the blocks and quantizes (three launches instead of two)."""
    cfg = I.CONFIGS["tiny"]
    d, N = 1024, 256
    xb = I.activations(cfg, M=M, d=d)
    rb, rib, _, _ = I.rotations(cfg, d=d)
    if not intra:
        rib = None
    g = np.random.default_rng(3)
    wq = g.integers(-7, 8, (N, d)).astype(np.int8)
    wsb = g.integers(120, 134, (N, d // 32), dtype=np.uint8)
    dbg_b = torch.empty((M, d), dtype=torch.uint8, device="cuda")
    dbg_s = torch.empty(torq.torq_scales_bytes(M, d), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    n0 = torq.torq_launch_count()
    y = torq.torq_rotated_linear_mxint4(dev_bf16(xb), dev_bf16(rb), None if rib is None else dev_bf16(rib),
                                        dev_u8(O.int4_to_e4m3(wq)), dev_u8(O.swizzle_scales(wsb, d, fill=0)),
                                        out_dtype=torch.float32, dbg_bytes=dbg_b, dbg_scales=dbg_s)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    assert torq.torq_launch_count() - n0 == (2 if M <= 256 else 3)   # up to 256 tokens: one rotation kernel, K splits reduced on chip
    g_q, g_sb = _operand_to_int(dbg_b), O.unswizzle_scales(dbg_s.cpu().numpy(), M, d)
    o_q, o_sb = O.quantize_mxint4(O.round_to_f32(O.rotate(xb, rb, rib)))
    rep = _mismatch(g_q, g_sb, o_q, o_sb)
    assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
    assert rep["elem"] * M * d <= max(2, 1e-4 * M * d) and rep["blocks"] * M * (d // 32) <= max(1, 1e-4 * M * (d // 32)), rep
    buf = dbg_s.cpu().numpy().copy()                      # padding of the scale tiles is zero
    rr, cc = np.meshgrid(np.arange(M), np.arange(d // 32), indexing="ij")
    buf[O.scale_layout_offset(rr, cc, d)] = 0
    assert not buf.any()
    ref = O.gemm_mxint4(g_q, g_sb, wq, wsb)
    got = y.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5


def test_llama3_qkv_shape_sampled_rows():
    """Benchmark shape (2048 x 4096 -> 6144): rotation and quantizer on sampled rows against the oracle
    (rows are independent), the GEMM on the GPU's own codes for the same rows."""
    cfg = I.CONFIGS["llama3_8b_qkv"]
    xb = I.activations(cfg)
    rb, rib, _, _ = I.rotations(cfg)
    rows = np.array([0, 1, 127, 128, 255, 256, 1000, 1023, 1024, 2047])
    g = np.random.default_rng(77)
    wq = g.integers(-7, 8, (cfg.N, cfg.d)).astype(np.int8)
    wsb = g.integers(120, 134, (cfg.N, cfg.d // 32), dtype=np.uint8)
    dbg_b = torch.empty((cfg.M, cfg.d), dtype=torch.uint8, device="cuda")
    dbg_s = torch.empty(torq.torq_scales_bytes(cfg.M, cfg.d), dtype=torch.uint8, device="cuda")
    y = torq.torq_rotated_linear_mxint4(dev_bf16(xb), dev_bf16(rb), dev_bf16(rib), dev_u8(O.int4_to_e4m3(wq)),
                                        dev_u8(O.swizzle_scales(wsb, cfg.d, fill=0)), out_dtype=torch.float32,
                                        dbg_bytes=dbg_b, dbg_scales=dbg_s)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    g_q = _operand_to_int(dbg_b[torch.from_numpy(rows).cuda()])
    g_sb = O.unswizzle_scales(dbg_s.cpu().numpy(), cfg.M, cfg.d)[rows]
    o_q, o_sb = O.quantize_mxint4(O.round_to_f32(O.rotate(xb[rows], rb, rib)))
    rep = _mismatch(g_q, g_sb, o_q, o_sb)
    assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
    assert rep["elem"] <= 1e-4 and rep["blocks"] <= 1e-4, rep
    ref = O.gemm_mxint4(g_q, g_sb, wq, wsb)
    got = y.cpu().numpy().astype(np.float64)[rows]
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5


@pytest.mark.parametrize("M,d", [(64, 256), (130, 512), (7, 1024), (2048, 4096)])
def test_structured_rotation_with_the_mxint4_quantizer(M, d):
    """The rotation in the paper's own structure (one matrix across blocks, one shared matrix inside them)
    followed by the MXINT4 quantizer."""
    cfg = I.CONFIGS["tiny"]
    xb = I.activations(cfg, M=M, d=d)
    g = np.random.Generator(np.random.PCG64(I.BASE_SEED + 78))
    rbb = I.to_bf16_bits(I.orthogonal(d // 32, g))
    ri = I.to_bf16_bits(I.orthogonal(32, g))
    rows = np.arange(M) if M <= 256 else np.array([0, 1, 3, 4, 127, 128, 1000, 2046, 2047])
    byt_t, s_t = torq.torq_rotate_quantize_structured_mxint4(dev_bf16(xb), dev_bf16(rbb), dev_bf16(ri))
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    g_q = _operand_to_int(byt_t[torch.from_numpy(rows).cuda()])
    g_sb = O.unswizzle_scales(s_t.cpu().numpy(), M, d)[rows]
    o_q, o_sb = O.quantize_mxint4(O.round_to_f32(O.rotate_structured(xb[rows], rbb, ri)))
    rep = _mismatch(g_q, g_sb, o_q, o_sb)
    assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
    n = rows.size * d
    assert rep["elem"] * n <= max(2, 2e-4 * n) and rep["blocks"] * (n // 32) <= max(1, 2e-4 * (n // 32)), rep
    buf = s_t.cpu().numpy().copy()                                       # padding of the scale tiles is zero
    rr, cc = np.meshgrid(np.arange(M), np.arange(d // 32), indexing="ij")
    buf[O.scale_layout_offset(rr, cc, d)] = 0
    assert not buf.any()
