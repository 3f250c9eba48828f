"""GPU parity of the NVFP4 variant (format study of Section 6) against the oracle: quantizer bit for
bit; GEMM to 1e-3 relative Frobenius error (fp32 accumulation; far better in practice) and bit for
bit where fp32 accumulation is exact; rotate + quantize with at most 1e-4 of the elements one
lattice step off and at most 1e-4 of the block scales one E4M3 step off (the fp32 tensor-core
accumulation order differs from the oracle's fp64)."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import dev_bf16, dev_u8, lattice
from paper_2605_19561_b200 import inputs as I
from paper_2605_19561_b200 import torq

pytestmark = pytest.mark.gpu


def _to_numpy(codes_t, scales_t, M, d):
    return O.unpack_codes(codes_t.cpu().numpy()), O.nv_unswizzle_scales(scales_t.cpu().numpy(), M, d)


# ----------------------------------------------------------------------------- quantizer
@pytest.mark.parametrize("M,d", [(64, 256), (1, 16), (130, 48), (257, 1040), (128, 64), (300, 4096)])
def test_quantizer_fp32_input_is_bit_exact(M, d):
    g = np.random.default_rng(M * 1000 + d)
    z = (g.standard_t(3, size=(M, d)) * np.exp(g.uniform(-4, 4, size=(M, 1)))).astype(np.float32)
    if d > 16:
        z[0, :16] = 0.0                                   # an all-zero block
    if M > 2:
        z[2, :16] = 1e-30                                 # a block far below the tensor scale
    ts = float(O.tensor_scale_from_amax(np.abs(z).max()))
    codes_t, scales_t = torq.torq_quantize_nvfp4(torch.from_numpy(z).cuda(), ts)
    torch.cuda.synchronize()
    g_codes, g_sb = _to_numpy(codes_t, scales_t, M, d)
    o_codes, o_sb = O.quantize_nvfp4(z, ts)
    assert np.array_equal(g_sb, o_sb)
    assert np.array_equal(g_codes, o_codes)
    # padding bytes of the tiled scale buffer are zero
    buf = scales_t.cpu().numpy().copy()
    rr, cc = np.meshgrid(np.arange(M), np.arange(d // 16), indexing="ij")
    buf[O.nv_scale_layout_offset(rr, cc, d)] = 0
    assert not buf.any()


@pytest.mark.parametrize("ts", [1.0, 0.37, 3.1e-4, 250.0])
def test_quantizer_tensor_scales_and_bf16_input(ts):
    """Arbitrary (not power-of-two) tensor scales exercise every float32 rounding of the recipe."""
    g = np.random.default_rng(11)
    M, d = 96, 512
    zb = I.to_bf16_bits((g.standard_normal((M, d)) * ts * 300).astype(np.float32))
    z = O.decode_bf16(zb).astype(np.float32)
    codes_t, scales_t = torq.torq_quantize_nvfp4(dev_bf16(zb), ts)
    torch.cuda.synchronize()
    g_codes, g_sb = _to_numpy(codes_t, scales_t, M, d)
    o_codes, o_sb = O.quantize_nvfp4(z, np.float32(ts))
    assert np.array_equal(g_sb, o_sb) and np.array_equal(g_codes, o_codes)


def test_quantizer_thresholds_of_both_roundings():
    """Blocks whose scaled maximum sits on and next to every E4M3 rounding threshold, and elements on
    and next to every e2m1 threshold (tensor scale 1, so the thresholds are known exactly)."""
    vals = O.e4m3_value(np.arange(1, 0x7F, dtype=np.uint8))
    mids = (0.5 * (vals[1:] + vals[:-1])).astype(np.float32)
    am = np.concatenate([mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(1e9))]) * np.float32(6)
    z = np.zeros((am.size, 16), np.float32)
    z[:, 0] = am
    thr = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], np.float32)
    for j, t in enumerate(thr):                           # elements near thresholds, in units of amax / 6
        z[:, 1 + 2 * j] = am / 6 * t
        z[:, 2 + 2 * j] = -np.nextafter(am / 6 * t, np.float32(1e9))
    codes_t, scales_t = torq.torq_quantize_nvfp4(torch.from_numpy(z).cuda(), 1.0)
    torch.cuda.synchronize()
    g_codes, g_sb = _to_numpy(codes_t, scales_t, z.shape[0], 16)
    o_codes, o_sb = O.quantize_nvfp4(z, 1.0)
    assert np.array_equal(g_sb, o_sb) and np.array_equal(g_codes, o_codes)


def test_quantizer_against_the_exact_definition_of_the_format():
    """The kernel against the format's definition in float64 (no float32 reciprocal anywhere), on
    heavy-tailed blocks with tensor scales that are not powers of two: at most 1e-5 of the block
    scales differ, each by one E4M3 step; outside those blocks at most 1e-5 of the elements differ;
    every differing element is one lattice step away; sign bits never differ.  (The same bound the
    CPU pin puts on the float32 recipe: the kernel is that recipe bit for bit.)"""
    g = np.random.default_rng(5)
    n_blocks = n_elems = d_blocks = d_elems = 0
    for mul in (1.0, 0.37, 3.1e-4, 250.0, 1.0 / 3.0, 0.7071):
        z = (g.standard_t(3, size=(1024, 1024)) * np.exp(g.uniform(-4, 4, size=(1024, 1)))).astype(np.float32)
        ts = np.float32(np.abs(z).max() / (6 * 448) * mul * 1.2345)
        codes_t, scales_t = torq.torq_quantize_nvfp4(torch.from_numpy(z).cuda(), float(ts))
        torch.cuda.synchronize()
        g_codes, g_sb = _to_numpy(codes_t, scales_t, *z.shape)
        cex, sex = O.quantize_nvfp4_exact(z, ts)
        step = np.abs(g_sb.astype(np.int64) - sex.astype(np.int64))
        lat = np.abs(lattice(g_codes) - lattice(cex))
        assert step.max() <= 1 and lat.max() <= 1
        assert np.array_equal(g_codes >> 3, cex >> 3)
        same = np.repeat(step == 0, 16, axis=1)
        n_blocks += step.size
        n_elems += lat.size
        d_blocks += int((step != 0).sum())
        d_elems += int(((lat != 0) & same).sum())
    assert d_blocks <= 1e-5 * n_blocks and d_elems <= 1e-5 * n_elems, (d_blocks, n_blocks, d_elems, n_elems)


def test_expand_intra16_matches_the_oracle_form():
    ri16 = I.intra_rotations16(I.CONFIGS["tiny"], d=256)
    got = torq.torq_expand_intra16(dev_bf16(ri16))
    torch.cuda.synchronize()
    assert np.array_equal(got.view(torch.int16).cpu().numpy().view(np.uint16), O.expand_intra16(ri16))


# ---------------------------------------------------------------------------------- GEMM
def _rand_operand(rows, k, seed, lo=0x28, hi=0x48):
    g = np.random.default_rng(seed)
    codes = g.integers(0, 16, size=(rows, k), dtype=np.uint8)
    sb = g.integers(lo, hi, size=(rows, k // 16), dtype=np.uint8)
    return codes, sb


def _gpu_gemm(ac, asb, ats, wc, wsb, wts, out_dtype):
    K = ac.shape[1]
    y = torq.torq_nvfp4_gemm(dev_u8(O.pack_codes(ac)), dev_u8(O.nv_swizzle_scales(asb, K)), float(ats),
                             dev_u8(O.pack_codes(wc)), dev_u8(O.nv_swizzle_scales(wsb, K)), float(wts),
                             out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    return y.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("M,N,K", [(64, 256, 256), (128, 256, 128), (1, 8, 128), (33, 24, 384), (129, 264, 512),
                                   (200, 136, 1024), (256, 512, 4096), (130, 640, 640), (511, 1032, 896),
                                   (300, 520, 1152)])
def test_gemm_random_operands_fp32_output(M, N, K):
    ac, asb = _rand_operand(M, K, 1)
    wc, wsb = _rand_operand(N, K, 2)
    ats, wts = np.float32(0.013), np.float32(2.5e-4)
    ref = O.gemm_nvfp4(ac, asb, ats, wc, wsb, wts)
    got = _gpu_gemm(ac, asb, ats, wc, wsb, wts, torch.float32)
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert rel <= 1e-3, rel
    assert rel <= 1e-5, rel          # fp32 accumulation should do far better than the bound


def test_gemm_exact_regime_is_bit_exact():
    """Power-of-two scales (bytes 0x30, 0x38, 0x40 = 0.5, 1, 2) and tensor scales: every product is
    a multiple of 2^-4 below 2^24 units, so fp32 accumulation is exact whatever its order."""
    M, N, K = 160, 272, 512
    g = np.random.default_rng(3)
    ac = g.integers(0, 16, (M, K), dtype=np.uint8)
    wc = g.integers(0, 16, (N, K), dtype=np.uint8)
    asb = g.choice(np.array([0x30, 0x38, 0x40], np.uint8), size=(M, K // 16))
    wsb = g.choice(np.array([0x30, 0x38, 0x40], np.uint8), size=(N, K // 16))
    ref = O.gemm_nvfp4(ac, asb, 0.25, wc, wsb, 2.0)
    got = _gpu_gemm(ac, asb, 0.25, wc, wsb, 2.0, torch.float32)
    assert (got == ref).all()


@pytest.mark.parametrize("M", [128, 256, 384])
def test_gemm_one_hot_rows_pin_the_scale_assignment(M):
    """A one-hot activation row with value 1.0 returns one dequantized weight element times the row's
    own block scale: any mix-up of row <-> scale or 16-block <-> scale byte on either side, in either
    kernel (one CTA: M <= 128, and M = 256 with this few column tiles; CTA pair: M = 384), shows up exactly.  Scales over the whole E4M3 range,
    subnormals and zero included."""
    N, K = 256, 1024
    g = np.random.default_rng(5 + M)
    wc = g.integers(0, 16, (N, K), dtype=np.uint8)
    wsb = g.integers(0x00, 0x7F, (N, K // 16), dtype=np.uint8)
    ac = np.zeros((M, K), np.uint8)
    hot = g.integers(0, K, size=M)
    ac[np.arange(M), hot] = 2
    asb = g.integers(0x00, 0x7F, (M, K // 16), dtype=np.uint8)
    ref = O.gemm_nvfp4(ac, asb, 1.0, wc, wsb, 1.0)
    got = _gpu_gemm(ac, asb, 1.0, wc, wsb, 1.0, torch.float32)
    assert (got == ref).all()


def test_gemm_bf16_output_and_untouched_neighbours():
    M, N, K = 300, 520, 768
    ac, asb = _rand_operand(M, K, 7)
    wc, wsb = _rand_operand(N, K, 8)
    ats, wts = np.float32(0.02), np.float32(0.004)
    buf = torch.full((M * N + 4096,), 3.0, dtype=torch.bfloat16, device="cuda")
    Y = buf[2048:2048 + M * N].view(M, N)
    torq.torq_nvfp4_gemm(dev_u8(O.pack_codes(ac)), dev_u8(O.nv_swizzle_scales(asb, K)), float(ats),
                         dev_u8(O.pack_codes(wc)), dev_u8(O.nv_swizzle_scales(wsb, K)), float(wts), Y=Y)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    assert bool((buf[:2048] == 3.0).all()) and bool((buf[2048 + M * N:] == 3.0).all())
    want = O.round_to_bf16(O.gemm_nvfp4(ac, asb, ats, wc, wsb, wts))
    got = Y.float().cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - want) / np.linalg.norm(want) <= 1e-3
    assert (got == want).mean() > 0.99


def test_gemm_full_size_sampled_outputs_llama3_qkv_shape():
    M, N, K = 2048, 6144, 4096
    ac, asb = _rand_operand(M, K, 9, 0x30, 0x40)
    wc, wsb = _rand_operand(N, K, 10, 0x30, 0x40)
    y = torq.torq_nvfp4_gemm(dev_u8(O.pack_codes(ac)), dev_u8(O.nv_swizzle_scales(asb, K)), 0.5,
                             dev_u8(O.pack_codes(wc)), dev_u8(O.nv_swizzle_scales(wsb, K)), 0.125,
                             out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    rows = np.array([0, 127, 128, 1000, 2047])
    cols = np.array([0, 255, 256, 3000, 6143])
    yn = y.cpu().numpy().astype(np.float64)
    ref = O.gemm_nvfp4(ac[rows], asb[rows], 0.5, wc, wsb, 0.125)
    assert np.linalg.norm(yn[rows] - ref) / np.linalg.norm(ref) <= 1e-5
    ref2 = O.gemm_nvfp4(ac, asb, 0.5, wc[cols], wsb[cols], 0.125)
    assert np.linalg.norm(yn[:, cols] - ref2) / np.linalg.norm(ref2) <= 1e-5


# ------------------------------------------------------------------ rotation + quantizer
def _mismatch(g_codes, g_sb, o_codes, o_sb, ts):
    M, d = o_codes.shape
    same = g_sb == o_sb
    same_e = np.repeat(same, 16, axis=1)
    lg, lo = lattice(g_codes), lattice(o_codes)
    diff = (lg != lo) & same_e
    bad = int((diff & (np.abs(lg - lo) > 1)).sum())
    step = np.abs(g_sb.astype(np.int64) - o_sb.astype(np.int64))
    bad_blocks = int((step > 1).sum())
    if (~same).any():                                     # neighbouring scales: values within one coarse step
        dg, do = O.dequantize_nvfp4(g_codes, g_sb, ts), O.dequantize_nvfp4(o_codes, o_sb, ts)
        coarse = O.e4m3_value(np.maximum(g_sb, o_sb)) * float(ts)
        bad += int(((np.abs(dg - do) > 2.0 * np.repeat(coarse, 16, axis=1)) & ~same_e).sum())
    return {"elem": float(diff.sum()) / (M * d), "blocks": float((~same).sum()) / same.size,
            "non_adjacent": bad, "scale_off_by_more_than_one": bad_blocks}


def _rotate_case(xb, rb, ri16, exact=False):
    M, d = xb.shape
    z = O.rotate_blocks(xb, rb, ri16)
    ts = O.tensor_scale_from_amax(np.abs(z).max())
    ri32 = None if ri16 is None else torq.torq_expand_intra16(dev_bf16(ri16))
    torch.cuda.synchronize()
    codes_t, scales_t = torq.torq_rotate_quantize_nvfp4(dev_bf16(xb), dev_bf16(rb), ri32, float(ts))
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    g_codes, g_sb = _to_numpy(codes_t, scales_t, M, d)
    o_codes, o_sb = O.quantize_nvfp4(z.astype(np.float32), ts)
    if exact:
        assert np.array_equal(g_sb, o_sb) and np.array_equal(g_codes, o_codes)
    rep = _mismatch(g_codes, g_sb, o_codes, o_sb, ts)
    assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
    assert rep["elem"] <= 1e-4 and rep["blocks"] <= 1e-4, rep
    return rep


def test_rotation_exact_cases_are_bit_exact():
    """Permutations (inter and intra) of small-integer activations: every partial sum is exact in fp32."""
    g = np.random.default_rng(0)
    for M, d in ((150, 256), (300, 512)):                 # one-CTA kernel and CTA-pair kernel
        x = g.integers(-8, 9, size=(M, d)).astype(np.float32)
        P = np.zeros((d, d), np.float32); P[np.arange(d), g.permutation(d)] = 1
        Q = np.zeros((d // 16, 16, 16), np.float32)
        for b in range(d // 16):
            Q[b, np.arange(16), g.permutation(16)] = 1
        _rotate_case(I.to_bf16_bits(x), I.to_bf16_bits(P), None, exact=True)
        _rotate_case(I.to_bf16_bits(x), I.to_bf16_bits(P), I.to_bf16_bits(Q), exact=True)


@pytest.mark.parametrize("M,d", [(64, 256), (1, 256), (130, 512), (257, 320), (100, 64), (400, 1024)])
def test_rotation_random_small_shapes(M, d):
    cfg = I.CONFIGS["tiny"]
    xb = I.activations(cfg, M=M, d=d)
    rb, _, _, _ = I.rotations(cfg, d=d)
    _rotate_case(xb, rb, I.intra_rotations16(cfg, d=d))
    _rotate_case(xb, rb, None)


def test_rotated_linear_end_to_end_tiny_config():
    cfg = I.CONFIGS["tiny"]
    xb = I.activations(cfg)
    rb, _, _, _ = I.rotations(cfg)
    ri16 = I.intra_rotations16(cfg)
    w = I.weights(cfg)
    w_codes, w_sb, w_ts = O.prepare_weights_nvfp4(rb, ri16, w)
    x_ts = O.tensor_scale_from_amax(np.abs(O.rotate_blocks(xb, rb, ri16)).max())
    ri32 = torq.torq_expand_intra16(dev_bf16(ri16))
    dbg_c = torch.empty((cfg.M, cfg.d // 2), dtype=torch.uint8, device="cuda")
    dbg_s = torch.empty(torq.torq_nvfp4_scales_bytes(cfg.M, cfg.d), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    y = torq.torq_rotated_linear_nvfp4(dev_bf16(xb), dev_bf16(rb), ri32, float(x_ts), dev_u8(O.pack_codes(w_codes)),
                                       dev_u8(O.nv_swizzle_scales(w_sb, cfg.d)), float(w_ts),
                                       out_dtype=torch.float32, dbg_codes=dbg_c, dbg_scales=dbg_s)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    g_codes, g_sb = _to_numpy(dbg_c, dbg_s, cfg.M, cfg.d)
    o_out, o_codes, o_sb = O.rotated_linear_nvfp4(xb, rb, ri16, x_ts, w_codes, w_sb, w_ts)
    rep = _mismatch(g_codes, g_sb, o_codes, o_sb, x_ts)
    assert rep["non_adjacent"] == 0 and rep["elem"] <= 1e-4 and rep["blocks"] <= 1e-4, rep
    # the GEMM on the codes the GPU produced
    ref = O.gemm_nvfp4(g_codes, g_sb, x_ts, w_codes, w_sb, w_ts)
    got = y.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5
    assert np.linalg.norm(got - o_out) / np.linalg.norm(o_out) <= 2e-2
    # the layer approximates x W (two 4-bit operands)
    exact = O.decode_bf16(xb) @ w
    assert np.linalg.norm(got - exact) / np.linalg.norm(exact) < 0.25


@pytest.mark.parametrize("M", [1, 33, 128])
def test_rotated_linear_few_tokens_takes_the_split_rotation(M):
    """Few tokens: the rotation is split along its contraction over the SMs.  Up to 64 tokens one kernel
    reduces the splits through distributed shared memory; above, the partial sums go through the workspace
    and a second kernel adds them, rotates inside the blocks and quantizes (three launches instead of two)."""
    cfg = I.CONFIGS["tiny"]
    d, N = 1024, 256
    xb = I.activations(cfg, M=M, d=d)
    rb, _, _, _ = I.rotations(cfg, d=d)
    ri16 = I.intra_rotations16(cfg, d=d)
    z = O.rotate_blocks(xb, rb, ri16)
    x_ts = O.tensor_scale_from_amax(np.abs(z).max())
    g = np.random.default_rng(3)
    wc = g.integers(0, 16, (N, d), dtype=np.uint8)
    wsb = g.integers(0x30, 0x40, (N, d // 16), dtype=np.uint8)
    ri32 = torq.torq_expand_intra16(dev_bf16(ri16))
    dbg_c = torch.empty((M, d // 2), dtype=torch.uint8, device="cuda")
    dbg_s = torch.empty(torq.torq_nvfp4_scales_bytes(M, d), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    n0 = torq.torq_launch_count()
    y = torq.torq_rotated_linear_nvfp4(dev_bf16(xb), dev_bf16(rb), ri32, float(x_ts), dev_u8(O.pack_codes(wc)),
                                       dev_u8(O.nv_swizzle_scales(wsb, d)), 0.01, out_dtype=torch.float32,
                                       dbg_codes=dbg_c, dbg_scales=dbg_s)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    assert torq.torq_launch_count() - n0 == (2 if M <= 256 else 3)   # up to 256 tokens: one rotation kernel, K splits reduced on chip
    g_codes, g_sb = _to_numpy(dbg_c, dbg_s, M, d)
    o_codes, o_sb = O.quantize_nvfp4(z.astype(np.float32), x_ts)
    rep = _mismatch(g_codes, g_sb, o_codes, o_sb, x_ts)
    assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
    assert rep["elem"] * M * d <= max(2, 1e-4 * M * d) and rep["blocks"] * M * (d // 16) <= max(1, 1e-4 * M * (d // 16)), rep
    # padding of the scale tiles is zero
    buf = dbg_s.cpu().numpy().copy()
    rr, cc = np.meshgrid(np.arange(M), np.arange(d // 16), indexing="ij")
    buf[O.nv_scale_layout_offset(rr, cc, d)] = 0
    assert not buf.any()
    ref = O.gemm_nvfp4(g_codes, g_sb, x_ts, wc, wsb, np.float32(0.01))
    got = y.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5


def test_llama3_qkv_shape_sampled_rows():
    """Benchmark shape (2048 x 4096 -> 6144): rotation and quantizer on sampled rows against the oracle
    (rows are independent), the GEMM on the GPU's own codes for the same rows."""
    cfg = I.CONFIGS["llama3_8b_qkv"]
    xb = I.activations(cfg)
    rb, _, _, _ = I.rotations(cfg)
    ri16 = I.intra_rotations16(cfg)
    rows = np.array([0, 1, 127, 128, 255, 256, 1000, 1023, 1024, 2047])
    z = O.rotate_blocks(xb[rows], rb, ri16)
    x_ts = np.float32(np.abs(z).max() / (6 * 448) * 4)          # a calibrated-style scale, not this sample's own
    g = np.random.default_rng(77)
    wc = g.integers(0, 16, (cfg.N, cfg.d), dtype=np.uint8)
    wsb = g.integers(0x30, 0x40, (cfg.N, cfg.d // 16), dtype=np.uint8)
    w_ts = np.float32(3e-4)
    ri32 = torq.torq_expand_intra16(dev_bf16(ri16))
    dbg_c = torch.empty((cfg.M, cfg.d // 2), dtype=torch.uint8, device="cuda")
    dbg_s = torch.empty(torq.torq_nvfp4_scales_bytes(cfg.M, cfg.d), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    y = torq.torq_rotated_linear_nvfp4(dev_bf16(xb), dev_bf16(rb), ri32, float(x_ts), dev_u8(O.pack_codes(wc)),
                                       dev_u8(O.nv_swizzle_scales(wsb, cfg.d)), float(w_ts), out_dtype=torch.float32,
                                       dbg_codes=dbg_c, dbg_scales=dbg_s)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    g_codes, g_sb = _to_numpy(dbg_c, dbg_s, cfg.M, cfg.d)
    o_codes, o_sb = O.quantize_nvfp4(z.astype(np.float32), x_ts)
    rep = _mismatch(g_codes[rows], g_sb[rows], o_codes, o_sb, x_ts)
    assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
    assert rep["elem"] <= 2e-4 and rep["blocks"] <= 2e-4, rep      # 40960 elements sampled: a handful may differ
    ref = O.gemm_nvfp4(g_codes[rows], g_sb[rows], x_ts, wc, wsb, w_ts)
    got = y.cpu().numpy()[rows].astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5


@pytest.mark.parametrize("M,d", [(64, 256), (130, 512), (2048, 4096)])
def test_structured_rotation_with_the_nvfp4_quantizer(M, d):
    """The rotation in the paper's own structure (one matrix across blocks, one shared matrix inside them,
    here two 16 x 16 blocks on the diagonal of a 32 x 32) followed by the NVFP4 quantizer."""
    cfg = I.CONFIGS["tiny"]
    xb = I.activations(cfg, M=M, d=d)
    g = np.random.Generator(np.random.PCG64(I.BASE_SEED + 77))
    rbb = I.to_bf16_bits(I.orthogonal(d // 32, g))
    ri32 = O.expand_intra16(I.intra_rotations16(cfg, d=32))[0]           # [32, 32] bit patterns
    rows = np.arange(M) if M <= 256 else np.array([0, 1, 3, 4, 127, 128, 1000, 2046, 2047])
    z = O.rotate_structured(xb[rows], rbb, ri32)
    ts = np.float32(np.abs(z).max() / (6 * 448) * (1 if M <= 256 else 2))
    codes_t, scales_t = torq.torq_rotate_quantize_structured_nvfp4(dev_bf16(xb), dev_bf16(rbb), dev_bf16(ri32), float(ts))
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    g_codes, g_sb = _to_numpy(codes_t, scales_t, M, d)
    o_codes, o_sb = O.quantize_nvfp4(z.astype(np.float32), ts)
    rep = _mismatch(g_codes[rows], g_sb[rows], o_codes, o_sb, ts)
    assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
    assert rep["elem"] <= 2e-4 and rep["blocks"] <= 2e-4, rep
    buf = scales_t.cpu().numpy().copy()                                  # padding of the scale tiles is zero
    rr, cc = np.meshgrid(np.arange(M), np.arange(d // 16), indexing="ij")
    buf[O.nv_scale_layout_offset(rr, cc, d)] = 0
    assert not buf.any()
