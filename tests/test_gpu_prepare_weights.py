"""The offline weight side (Algorithm 3 step 5, option B: W' = R~^T W, then quantization along K) on
the device, through torq_prepare_weights{,_nvfp4,_mxint4}, against the oracle's fp64 product.

The device contracts W^T (split exactly into three bfloat16 terms) with R_inter on the tensor cores
in fp32 and applies the intra-block step in fp32, so a value within ~1e-6 relative of a decision
threshold may land on the other side: the bound is the activation side's -- at most 1e-4 of the
elements differ, each to an adjacent codeword, at most 1e-4 of the block scales differ, each by one
step, nothing differs by more."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import dev_bf16, gpu_quantized_to_numpy, lattice, mismatch_report
from paper_2605_19561_b200 import inputs as I
from paper_2605_19561_b200 import torq

pytestmark = pytest.mark.gpu


def _rows_of_w_prime(rb, rib, w, cols, block=32):
    """Rows `cols` of W'^T = (R~^T W)^T in float64: W[:, n]^T R~ with R~ merged from the bf16 values."""
    r = O.decode_bf16(rb)
    ri = O.decode_bf16(rib)
    y = np.asarray(w, dtype=np.float64)[:, cols].T @ r
    z = np.empty_like(y)
    for b in range(ri.shape[0]):
        z[:, b * block:(b + 1) * block] = y[:, b * block:(b + 1) * block] @ ri[b]
    return z


def test_tiny_config_all_three_formats():
    cfg = I.CONFIGS["tiny"]
    rb, rib, _, _ = I.rotations(cfg)
    ri16 = I.intra_rotations16(cfg)
    w = I.weights(cfg)
    Wd, Rd, Rid = torch.from_numpy(w).cuda(), dev_bf16(rb), dev_bf16(rib)
    torch.cuda.synchronize()
    size = cfg.N * cfg.d
    one_block = 33.0 / size                     # at this size 1e-4 is six elements: allow one block with the other scale
    before = torq.torq_launch_count()
    Wq, Ws = torq.torq_prepare_weights(Rd, Rid, Wd)
    torch.cuda.synchronize()
    assert torq.torq_launch_count() - before == 3            # split/transpose, rotation, quantizer
    assert torq.torq_last_device_error() == 0
    g_codes, g_sb = gpu_quantized_to_numpy(Wq, Ws, cfg.N, cfg.d)
    o_codes, o_sb = O.prepare_weights(rb, rib, w)
    rep = mismatch_report(g_codes, g_sb, o_codes, o_sb)
    assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
    assert rep["elem_mismatch_frac"] <= max(1e-4, one_block) and rep["block_scale_mismatch_frac"] <= max(1e-4, 1.5 * 32 / size), rep
    # NVFP4
    ri32 = torq.torq_expand_intra16(dev_bf16(ri16))
    torch.cuda.synchronize()
    Nq, Ns, ts = torq.torq_prepare_weights_nvfp4(Rd, ri32, Wd)
    torch.cuda.synchronize()
    n_codes, n_sb, n_ts = O.prepare_weights_nvfp4(rb, ri16, w)
    # the maximum is itself an fp32 tensor-core sum over 3 d terms: up to one unit in the last place (2^-23) lost
    # in each of its 3 d / 16 accumulation steps, plus the intra-block step and the division
    assert abs(ts - float(n_ts)) <= (3 * cfg.d / 16 + 34) * 2.0 ** -23 * float(n_ts)
    gc = O.unpack_codes(Nq.cpu().numpy())
    gs = O.nv_unswizzle_scales(Ns.cpu().numpy(), cfg.N, cfg.d)
    if ts == float(n_ts):
        step = np.abs(gs.astype(np.int64) - n_sb.astype(np.int64))
        lat = np.abs(lattice(gc) - lattice(n_codes))
        assert step.max() <= 1 and lat.max() <= 1
        assert (step != 0).sum() <= max(1e-4 * step.size, 1.5) and (lat != 0).sum() <= max(1e-4 * lat.size, 17)
    else:                                                      # another tensor scale moves every threshold: compare values
        dg, do = O.dequantize_nvfp4(gc, gs, ts), O.dequantize_nvfp4(n_codes, n_sb, n_ts)
        assert np.linalg.norm(dg - do) / np.linalg.norm(do) <= 1e-3
    # MXINT4
    Wn, W8, Wsi = torq.torq_prepare_weights_mxint4(Rd, Rid, Wd)
    torch.cuda.synchronize()
    i_q, i_sb = O.prepare_weights_mxint4(rb, rib, w)
    g_q = O.unpack_int4(Wn.cpu().numpy())
    assert np.array_equal(O.e4m3_to_int4(W8.cpu().numpy()), g_q)
    g_isb = O.unswizzle_scales(Wsi.cpu().numpy(), cfg.N, cfg.d)
    same = np.repeat(g_isb == i_sb, 32, axis=1)
    assert np.abs(g_isb.astype(np.int64) - i_sb.astype(np.int64)).max() <= 1
    assert np.abs(g_q.astype(np.int64) - i_q.astype(np.int64))[same].max() <= 1
    assert (g_q != i_q)[same].sum() <= max(1e-4 * size, 1.5) and (g_isb != i_sb).sum() <= max(1e-4 * i_sb.size, 1.5)
    assert torq.torq_last_device_error() == 0


def test_narrow_weight_takes_the_single_cta_rotation_and_ragged_sizes():
    """N <= 128 output features (one row tile: the single-CTA rotation kernel) and sizes that are no
    multiple of a tile."""
    cfg = I.CONFIGS["tiny"]
    for d, N in ((256, 72), (320, 200)):
        rb, rib, _, _ = I.rotations(cfg, d=d)
        w = I.weights(cfg, d=d, N=N)
        Wq, Ws = torq.torq_prepare_weights(dev_bf16(rb), dev_bf16(rib), torch.from_numpy(w).cuda())
        torch.cuda.synchronize()
        g_codes, g_sb = gpu_quantized_to_numpy(Wq, Ws, N, d)
        o_codes, o_sb = O.prepare_weights(rb, rib, w)
        rep = mismatch_report(g_codes, g_sb, o_codes, o_sb)
        assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
        assert rep["elem_mismatch_frac"] <= max(1e-4, 33.0 / (N * d)), rep
    assert torq.torq_last_device_error() == 0


def test_llama3_qkv_weight_sampled_rows_and_the_nvfp4_tensor_scale():
    """The 4096 x 6144 weight of the QKV shape prepared on the device; 96 sampled output features (rows
    of the stored matrix, including the edges of 128- and 256-row tiles) against the oracle."""
    cfg = I.CONFIGS["llama3_8b_qkv"]
    rb, rib, _, _ = I.rotations(cfg)
    w = I.weights(cfg)
    d, N = cfg.d, cfg.N
    Wd, Rd, Rid = torch.from_numpy(w).cuda(), dev_bf16(rb), dev_bf16(rib)
    ws = torch.empty(torq.torq_prepare_weights_workspace_bytes(d, N), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    Wq, Ws = torq.torq_prepare_weights(Rd, Rid, Wd, workspace=ws)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    g = np.random.default_rng(5)
    cols = np.unique(np.concatenate([[0, 1, 127, 128, 255, 256, 257, 511, 512, N - 257, N - 256, N - 129, N - 128, N - 1],
                                     g.integers(0, N, 82)]))
    z32 = O.round_to_f32(_rows_of_w_prime(rb, rib, w, cols))
    o_codes, o_sb = O.quantize_mxfp4(z32)
    g_codes = O.unpack_codes(Wq[torch.from_numpy(cols).cuda()].cpu().numpy())
    g_sb = O.unswizzle_scales(Ws.cpu().numpy(), N, d)[cols]
    rep = mismatch_report(g_codes, g_sb, o_codes, o_sb)
    assert rep["non_adjacent"] == 0 and rep["scale_off_by_more_than_one"] == 0, rep
    assert rep["elem_mismatch_frac"] <= 1e-4 and rep["block_scale_mismatch_frac"] <= 1e-4, rep
    # NVFP4: the tensor scale needs the maximum over the whole of W' (float64 product on the host cores)
    ri16 = I.intra_rotations16(cfg)
    ri32 = torq.torq_expand_intra16(dev_bf16(ri16))
    torch.cuda.synchronize()
    Nq, Ns, ts = torq.torq_prepare_weights_nvfp4(Rd, ri32, Wd, workspace=ws)
    torch.cuda.synchronize()
    r = O.decode_bf16(rb)
    ri = O.decode_bf16(ri16)
    rt = np.empty_like(r)
    for b in range(ri.shape[0]):
        rt[:, 16 * b:16 * b + 16] = r[:, 16 * b:16 * b + 16] @ ri[b]
    amax = 0.0
    for n0 in range(0, N, 1024):
        amax = max(amax, float(np.abs(w[:, n0:n0 + 1024].astype(np.float64).T @ rt).max()))
    o_ts = O.tensor_scale_from_amax(np.float32(amax))
    assert abs(ts - float(o_ts)) <= (3 * d / 16 + 34) * 2.0 ** -23 * float(o_ts)       # see the tiny case
    z16 = _rows_of_w_prime(rb, ri16, w, cols, block=16).astype(np.float32)
    n_codes, n_sb = O.quantize_nvfp4(z16, np.float32(ts))       # the scale the device used, so thresholds coincide
    gc = O.unpack_codes(Nq[torch.from_numpy(cols).cuda()].cpu().numpy())
    gs = O.nv_unswizzle_scales(Ns.cpu().numpy(), N, d)[cols]
    step = np.abs(gs.astype(np.int64) - n_sb.astype(np.int64))
    lat = np.abs(lattice(gc) - lattice(n_codes))
    assert step.max() <= 1 and lat.max() <= 1
    same = np.repeat(step == 0, 16, axis=1)
    # Block scales: E4M3 has eight rounding thresholds per octave of the block maximum (density 8 / ln 2 per unit of
    # ln amax), and a block maximum is an fp32 tensor-core sum over 3 d terms, 3 d / 16 accumulation steps that may
    # each lose one unit in the last place: delta = (3 d / 16) 2^-23 = 9.2e-5, so at most (8 / ln 2) delta = 1.06e-3
    # of the blocks can carry the neighbouring scale byte (observed 3e-4).  Elements of equal-scale blocks: 1e-4.
    scale_bound = 8.0 / np.log(2.0) * (3 * d / 16) * 2.0 ** -23
    assert (step != 0).sum() <= scale_bound * step.size and ((lat != 0) & same).sum() <= 1e-4 * lat.size
    assert torq.torq_last_device_error() == 0


def test_argument_errors():
    W = torch.zeros((256, 64), dtype=torch.float32, device="cuda")
    R = torch.zeros((256, 256), dtype=torch.bfloat16, device="cuda")
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    before = torq.torq_launch_count()
    with pytest.raises(torq.TorqError) as e:
        torq.torq_prepare_weights(R, None, W, workspace=small)
    assert e.value.code == 7                                   # TORQ_ERR_WORKSPACE
    with pytest.raises(torq.TorqError) as e:
        torq.torq_prepare_weights(None, None, W)
    assert e.value.code == 1                                   # R_inter is required
    W96 = torch.zeros((96, 64), dtype=torch.float32, device="cuda")
    R96 = torch.zeros((96, 96), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(torq.TorqError) as e:
        torq.torq_prepare_weights(R96, None, W96)
    assert e.value.code == 2                                   # d % 64 != 0
    assert torq.torq_launch_count() == before
