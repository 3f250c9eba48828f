"""GPU parity at the full sizes of the remaining workloads, in the launch configuration the
benchmark uses (one torq_rotated_linear call, bf16 output): LLaMA3-8B down-projection
(2048 x 14336 -> 4096, Laplace activations), Qwen3-32B gate/up at long prefill
(8192 x 5120 -> 51200) and the token sweep at hidden 5120 (M = 1 ... 16384).

The oracle cannot afford the whole problem, but every step is independent per row (token), so it
computes sampled rows one by one: rows at tile edges (0, 127, 128, 255, 256 ...), the last rows,
and a few in the middle.  Bounds as in the small-shape tests: at most 1e-4 of the sampled elements
differ from the oracle's codes, each by one lattice step; scale bytes likewise; the GEMM on the
codes the GPU produced is within 1e-3 relative Frobenius error of the oracle's rounded result."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import dev_bf16, gpu_quantized_to_numpy, mismatch_report
from paper_2605_19561_b200 import inputs as I
from paper_2605_19561_b200 import torq

pytestmark = pytest.mark.gpu


def _layer_operands(cfg):
    """Rotations (QR on the device: LAPACK on a few host cores is slow at d = 14336) and the
    device-prepared weights of one workload."""
    rb, rib, _, _ = I.rotations(cfg, device="cuda")
    Rd, Rid = dev_bf16(rb), dev_bf16(rib)
    Wq, Ws = torq.prepare_weights(Rd, Rid, torch.from_numpy(I.weights(cfg)).cuda())
    torch.cuda.synchronize()
    return rb, rib, Rd, Rid, Wq, Ws


def _check_layer(cfg, M, rb, rib, Rd, Rid, Wq, Ws, rows, cols):
    xb = I.activations(cfg, M=M)
    d, N = cfg.d, Wq.shape[0]
    dbg_c = torch.empty((M, d // 2), dtype=torch.uint8, device="cuda")
    dbg_s = torch.empty(torq.torq_scales_bytes(M, d), dtype=torch.uint8, device="cuda")
    y = torq.torq_rotated_linear(dev_bf16(xb), Rd, Rid, Wq, Ws, out_dtype=torch.bfloat16,
                                 dbg_codes=dbg_c, dbg_scales=dbg_s)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    rows = np.unique(np.clip(np.asarray(rows), 0, M - 1))
    g_codes = O.unpack_codes(dbg_c[torch.from_numpy(rows).cuda()].cpu().numpy())
    g_sb = O.unswizzle_scales(dbg_s.cpu().numpy(), M, d)[rows]
    o_codes, o_sb = O.quantize_mxfp4(O.round_to_f32(O.rotate(xb[rows], rb, rib)))
    rep = mismatch_report(g_codes, g_sb, o_codes, o_sb)
    assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
    # with few sampled elements one benign flip can exceed a pure fraction: allow one element
    allowed = max(1e-4, 1.5 / g_codes.size)
    assert rep["elem_mismatch_frac"] <= allowed, rep
    assert rep["block_scale_mismatch_frac"] <= max(1e-4, 1.5 / g_sb.size), rep
    cols = np.unique(np.clip(np.asarray(cols), 0, N - 1))
    tc = torch.from_numpy(cols).cuda()
    w_codes = O.unpack_codes(Wq[tc].cpu().numpy())
    w_sb = O.unswizzle_scales(Ws.cpu().numpy(), N, d)[cols]
    want = O.round_to_bf16(O.gemm_dequant(g_codes, g_sb, w_codes, w_sb))
    got = y[torch.from_numpy(rows).cuda()][:, tc].float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert np.linalg.norm(got - want) / np.linalg.norm(want) <= 1e-3
    ulp = np.ldexp(1.0, np.frexp(np.maximum(np.abs(want), 1e-30))[1] - 8)
    assert (np.abs(got - want) <= ulp).all()
    return rep


def _edge_rows(M):
    base = [0, 1, 31, 127, 128, 129, 255, 256, 257, 383, 511, 512, M // 2, M - 257, M - 129, M - 128, M - 2, M - 1]
    return [r for r in base if 0 <= r < M]


def _edge_cols(N, n_random=500, seed=5):
    g = np.random.default_rng(seed)
    base = [0, 1, 127, 128, 255, 256, 257, 511, 512, N // 2, N - 257, N - 256, N - 255, N - 129, N - 1]
    return np.concatenate([np.array([c for c in base if 0 <= c < N]), g.integers(0, N, size=n_random)])


def test_llama3_down_projection_shape_sampled_rows():
    cfg = I.CONFIGS["llama3_8b_down"]
    ops = _layer_operands(cfg)
    _check_layer(cfg, cfg.M, *ops, rows=_edge_rows(cfg.M), cols=np.arange(cfg.N))


def test_qwen3_gate_up_shape_sampled_rows_and_columns():
    cfg = I.CONFIGS["qwen3_32b_gateup"]
    ops = _layer_operands(cfg)
    _check_layer(cfg, cfg.M, *ops, rows=_edge_rows(cfg.M), cols=_edge_cols(cfg.N, n_random=1500))


def test_token_sweep_at_hidden_5120():
    cfg = I.CONFIGS["qwen3_32b_sweep"]
    ops = _layer_operands(cfg)
    for M in I.SWEEP_M:
        rows = np.arange(M) if M <= 64 else _edge_rows(M)
        _check_layer(cfg, M, *ops, rows=rows, cols=np.arange(cfg.N))


def test_llama3_down_projection_shape_in_mxint4_sampled_rows():
    """The MXINT4 variant at the down-projection shape (2048 x 14336 -> 4096: 224 K steps in the rotation, 112 in
    the FP8-rate GEMM): sampled rows of the quantized activations against the oracle, the GEMM on the GPU's own
    codes for those rows, all columns."""
    cfg = I.CONFIGS["llama3_8b_down"]
    rb, rib, _, _ = I.rotations(cfg, device="cuda")
    Rd, Rid = dev_bf16(rb), dev_bf16(rib)
    Wn, W8, Ws = torq.prepare_weights_mxint4(Rd, Rid, torch.from_numpy(I.weights(cfg)).cuda())
    xb = I.activations(cfg)
    M, d, N = cfg.M, cfg.d, cfg.N
    dbg_b = torch.empty((M, d), dtype=torch.uint8, device="cuda")
    dbg_s = torch.empty(torq.torq_scales_bytes(M, d), dtype=torch.uint8, device="cuda")
    y = torq.torq_rotated_linear_mxint4(dev_bf16(xb), Rd, Rid, W8, Ws, out_dtype=torch.bfloat16, dbg_bytes=dbg_b,
                                        dbg_scales=dbg_s)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    rows = np.unique(np.array(_edge_rows(M)))
    tr = torch.from_numpy(rows).cuda()
    g_q = O.e4m3_to_int4(dbg_b[tr].cpu().numpy())
    g_sb = O.unswizzle_scales(dbg_s.cpu().numpy(), M, d)[rows]
    o_q, o_sb = O.quantize_mxint4(O.round_to_f32(O.rotate(xb[rows], rb, rib)))
    same = g_sb == o_sb
    diff = (g_q != o_q) & np.repeat(same, 32, axis=1)
    assert (np.abs(g_q.astype(np.int64) - o_q)[diff] <= 1).all()
    assert (np.abs(g_sb.astype(np.int64) - o_sb.astype(np.int64)) <= 1).all()
    assert diff.sum() <= max(1e-4 * g_q.size, 1.5) and (~same).sum() <= max(1e-4 * same.size, 1.5)
    w_q = O.unpack_int4(Wn.cpu().numpy())
    assert np.array_equal(O.e4m3_to_int4(W8.cpu().numpy()), w_q)
    w_sb = O.unswizzle_scales(Ws.cpu().numpy(), N, d)
    want = O.round_to_bf16(O.gemm_mxint4(g_q, g_sb, w_q, w_sb))
    got = y[tr].float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert np.linalg.norm(got - want) / np.linalg.norm(want) <= 1e-3
    ulp = np.ldexp(1.0, np.frexp(np.maximum(np.abs(want), 1e-30))[1] - 8)
    assert (np.abs(got - want) <= ulp).all()


def test_llama3_down_projection_shape_in_nvfp4_sampled_rows():
    """The NVFP4 variant at the down-projection shape (2048 x 14336 -> 4096): sampled rows of the quantized
    activations against the oracle (at most 1e-4 of the elements one lattice step off, at most 1.23e-3 of the block
    scales one E4M3 step off: the bound derived below from the depth of the accumulation), the GEMM on the GPU's own codes for those rows, all columns."""
    cfg = I.CONFIGS["llama3_8b_down"]
    rb, _, _, _ = I.rotations(cfg, device="cuda")
    ri16 = I.intra_rotations16(cfg)
    Rd = dev_bf16(rb)
    Ri32 = torq.torq_expand_intra16(dev_bf16(ri16))
    torch.cuda.synchronize()
    Wq, Ws, w_ts = torq.prepare_weights_nvfp4(Rd, Ri32, torch.from_numpy(I.weights(cfg)).cuda())
    xb = I.activations(cfg)
    M, d, N = cfg.M, cfg.d, cfg.N
    rows = np.unique(np.array(_edge_rows(M)))
    z = O.rotate_blocks(xb[rows], rb, ri16)
    x_ts = np.float32(np.abs(z).max() / (6 * 448) * 2)          # a calibrated-style scale, not this sample's own
    dbg_c = torch.empty((M, d // 2), dtype=torch.uint8, device="cuda")
    dbg_s = torch.empty(torq.torq_nvfp4_scales_bytes(M, d), dtype=torch.uint8, device="cuda")
    y = torq.torq_rotated_linear_nvfp4(dev_bf16(xb), Rd, Ri32, float(x_ts), Wq, Ws, float(w_ts),
                                       out_dtype=torch.bfloat16, dbg_codes=dbg_c, dbg_scales=dbg_s)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    tr = torch.from_numpy(rows).cuda()
    g_codes = O.unpack_codes(dbg_c[tr].cpu().numpy())
    g_sb = O.nv_unswizzle_scales(dbg_s.cpu().numpy(), M, d)[rows]
    o_codes, o_sb = O.quantize_nvfp4(z.astype(np.float32), x_ts)
    same = g_sb == o_sb
    lat = lambda c: np.where(c & 8, -(c & 7).astype(np.int64), (c & 7).astype(np.int64))
    diff = (lat(g_codes) != lat(o_codes)) & np.repeat(same, 16, axis=1)
    assert (np.abs(lat(g_codes) - lat(o_codes))[diff] <= 1).all()
    assert (np.abs(g_sb.astype(np.int64) - o_sb.astype(np.int64)) <= 1).all()
    # Bound on the block scales, derived: the inter-block sum runs over d terms as d/16 tensor-core accumulation
    # steps in fp32, each of which may lose up to one unit in the last place of the accumulator (2^-23 relative;
    # nothing documents that step as round-to-nearest), so a block maximum can sit up to delta = (d/16) 2^-23 =
    # 1.07e-4 relative away from the oracle's fp64 value.  E4M3 has eight rounding thresholds per octave of the
    # block maximum, i.e. a density of 8 / ln 2 per unit of ln(amax), so at most (8 / ln 2) delta = 1.23e-3 of the
    # blocks can land on the neighbouring scale byte (observed: 2e-4, the drift of a typical sum is a fraction of
    # the worst case).  Elements in blocks with equal scales keep the 1e-4 bound of the other shapes.
    scale_bound = 8.0 / np.log(2.0) * (d / 16) * 2.0 ** -23
    assert 1.2e-3 < scale_bound < 1.3e-3
    assert diff.sum() <= max(1e-4 * g_codes.size, 1.5) and (~same).sum() <= max(scale_bound * same.size, 1.5)
    w_codes = O.unpack_codes(Wq.cpu().numpy())
    w_sb = O.nv_unswizzle_scales(Ws.cpu().numpy(), N, d)
    want = O.round_to_bf16(O.gemm_nvfp4(g_codes, g_sb, x_ts, w_codes, w_sb, np.float32(w_ts)))
    got = y[tr].float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert np.linalg.norm(got - want) / np.linalg.norm(want) <= 1e-3
    ulp = np.ldexp(1.0, np.frexp(np.maximum(np.abs(want), 1e-30))[1] - 8)
    assert (np.abs(got - want) <= ulp).all()
