"""GPU parity: the stand-alone MXFP4 quantizer against the oracle, bit for bit (Eq. 1)."""
import numpy as np
import pytest
import torch

import oracle as O
from helpers import dev_bf16, gpu_quantized_to_numpy
from paper_2605_19561_b200 import inputs as I
from paper_2605_19561_b200 import torq

pytestmark = pytest.mark.gpu


def _run_f32(z):
    zt = torch.from_numpy(z).cuda()
    codes_t, scales_t = torq.torq_quantize_mxfp4(zt)
    torch.cuda.synchronize()
    assert torq.torq_last_device_error() == 0
    return codes_t, scales_t


def _assert_bit_exact(z):
    M, d = z.shape
    codes_t, scales_t = _run_f32(z)
    g_codes, g_sb = gpu_quantized_to_numpy(codes_t, scales_t, M, d)
    o_codes, o_sb = O.quantize_mxfp4(z)
    assert (g_sb == o_sb).all()
    assert (g_codes == o_codes).all()
    assert (codes_t.cpu().numpy() == O.pack_codes(o_codes)).all()
    return scales_t


def test_every_bf16_value_in_every_position_class():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    with np.errstate(invalid="ignore"):
        v = O.decode_bf16(bits).astype(np.float32)
    v = v[np.isfinite(v)]
    # each value once as the block maximum (scale rule) ...
    z = np.zeros((v.size, 32), np.float32)
    z[:, 5] = v
    _assert_bit_exact(z)
    # ... and once next to a fixed maximum of 6 (bare e2m1 rounding incl. sign of zero)
    w = v[np.abs(v) < 8]
    z = np.zeros((w.size, 32), np.float32)
    z[:, 0] = 6.0
    z[:, 31] = w
    _assert_bit_exact(z)


def test_threshold_neighbourhoods_at_many_scales():
    thr = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], np.float32)
    rows = []
    for k in (-100, -20, -1, 0, 7, 60, 120):
        for t in thr:
            lo = t
            for _ in range(8):
                lo = np.nextafter(lo, np.float32(0))
            cur = lo
            for _ in range(17):
                for sgn in (1.0, -1.0):
                    r = np.zeros(32, np.float32)
                    r[3] = np.ldexp(np.float32(6.0), k)
                    r[17] = sgn * np.ldexp(cur, k)
                    rows.append(r)
                cur = np.nextafter(cur, np.float32(np.inf))
    _assert_bit_exact(np.stack(rows))


def test_extremes_zero_blocks_and_subnormals():
    z = np.zeros((6, 64), np.float32)
    z[0, :] = 0.0
    z[1, 3] = -0.0
    z[2, 0] = np.float32(1e-45); z[2, 40] = np.float32(-1e-40)
    z[3, 1] = np.float32(3.0e38); z[3, 2] = np.float32(-1.0e38); z[3, 33] = np.float32(2 ** -126)
    z[4, :] = np.float32(2 ** -126)
    z[5, :] = np.float32(-3.4e38)
    _assert_bit_exact(z)


@pytest.mark.parametrize("M,d", [(1, 32), (31, 64), (33, 96), (127, 256), (129, 160), (64, 256), (300, 4096)])
def test_heavy_tailed_blocks_ragged_shapes(M, d):
    g = np.random.default_rng(M * 1000 + d)
    z = (g.standard_t(3, size=(M, d)) * np.exp(g.normal(0, 4, size=(M, 1)))).astype(np.float32)
    scales_t = _assert_bit_exact(z)
    # padding rows / K-blocks of the tiled scale buffer are written as 0
    buf = scales_t.cpu().numpy()
    mask = np.ones(buf.size, bool)
    rr, cc = np.meshgrid(np.arange(M), np.arange(d // 32), indexing="ij")
    mask[O.scale_layout_offset(rr, cc, d)] = False
    assert (buf[mask] == 0).all()


def test_bf16_input_path_matches_the_same_values_in_f32():
    cfg = I.CONFIGS["tiny"]
    xb = I.activations(cfg)
    codes_t, scales_t = torq.torq_quantize_mxfp4(dev_bf16(xb))
    torch.cuda.synchronize()
    g_codes, g_sb = gpu_quantized_to_numpy(codes_t, scales_t, cfg.M, cfg.d)
    o_codes, o_sb = O.quantize_mxfp4(O.decode_bf16(xb).astype(np.float32))
    assert (g_sb == o_sb).all() and (g_codes == o_codes).all()


def test_swizzle_scales_helper():
    g = np.random.default_rng(9)
    sb = g.integers(0, 255, size=(200, 24), dtype=np.uint8)
    out = torq.torq_swizzle_scales(torch.from_numpy(sb).cuda(), 24 * 32)
    torch.cuda.synchronize()
    assert (out.cpu().numpy() == O.swizzle_scales(sb, 24 * 32, fill=0)).all()


def test_full_size_sampled_rows_llama3_qkv_shape():
    """At the benchmark's size (2048 x 4096, float32 input) check sampled rows one by one."""
    g = np.random.default_rng(77)
    z = (g.standard_t(3, size=(2048, 4096))).astype(np.float32)
    z[:, [7, 1000, 2222, 4000]] *= 100
    codes_t, scales_t = _run_f32(z)
    rows = np.array([0, 1, 127, 128, 1023, 1500, 2047])
    g_codes = O.unpack_codes(codes_t.cpu().numpy()[rows])
    g_sb = O.unswizzle_scales(scales_t.cpu().numpy(), 2048, 4096)[rows]
    o_codes, o_sb = O.quantize_mxfp4(z[rows])
    assert (g_sb == o_sb).all() and (g_codes == o_codes).all()
