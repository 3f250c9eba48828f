"""Pins for the oracle's NVFP4 functions (format study of Section 6; the format is defined by its
public specification: e2m1 elements, 16-element blocks, E4M3 block scale, float32 tensor scale).

Each check restates the format by a route the oracle does not use: ml_dtypes' float8_e4m3fn and
float4_e2m1fn casts, hand-worked blocks whose float32 arithmetic is exact, bounds that follow from
the format, and exact rational arithmetic in pure Python."""
from fractions import Fraction

import ml_dtypes
import numpy as np
import pytest

import oracle as O


def test_e4m3_table_matches_ml_dtypes_for_every_bit_pattern():
    b = np.arange(256, dtype=np.uint8)
    want = b.view(ml_dtypes.float8_e4m3fn).astype(np.float64)
    got = O.e4m3_value(b)
    assert np.array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok], want[ok])
    assert np.array_equal(np.signbit(got[ok]), np.signbit(want[ok]))
    assert O.e4m3_value(0x7E) == 448.0 and O.e4m3_value(0x01) == 2.0 ** -9 and O.e4m3_value(0x38) == 1.0


def test_e4m3_encoder_matches_ml_dtypes_on_values_midpoints_and_neighbours():
    vals = O.e4m3_value(np.arange(0x7F, dtype=np.uint8))                 # 0 .. 448
    mids = 0.5 * (vals[1:] + vals[:-1])
    m32 = mids.astype(np.float32)                                         # midpoints are exact in float32
    pts = np.concatenate([vals, mids, np.nextafter(m32, np.float32(0)), np.nextafter(m32, np.float32(1e9)),
                          np.random.default_rng(0).uniform(0, 448, 20000),
                          np.exp(np.random.default_rng(1).uniform(np.log(1e-4), np.log(448), 20000))])
    # float32 points, as the quantizer feeds them (ml_dtypes rounds float64 input to float32 first,
    # so a float64 neighbour of a midpoint would reach it as the midpoint itself)
    pts = pts.astype(np.float32)
    want = pts.astype(ml_dtypes.float8_e4m3fn).view(np.uint8)
    assert np.array_equal(O.encode_e4m3(pts.astype(np.float64)), want)
    # every representable value encodes to itself, and the byte order is the value order
    assert np.array_equal(O.encode_e4m3(vals), np.arange(0x7F))
    assert (np.diff(vals) > 0).all()


def test_e4m3_encoder_saturates_above_448():
    assert O.encode_e4m3(np.array([448.0, 460.0, 464.0, 480.0, 1e6])).tolist() == [0x7E] * 5


def test_e2m1_step_matches_ml_dtypes():
    a = np.random.default_rng(2).uniform(-7, 7, 4096).astype(np.float32).reshape(-1, 16)
    a[:, 0] = 6.0                                        # block maximum 6 with tensor scale 1: scale byte = 1.0
    codes, sb = O.quantize_nvfp4(np.clip(a, -6, 6), 1.0)
    assert (sb == 0x38).all()
    want = np.clip(a, -6, 6).astype(ml_dtypes.float4_e2m1fn).astype(np.float64)
    assert np.array_equal(O.dequantize_nvfp4(codes, sb, 1.0), want)


def _blk(vals):
    z = np.zeros((1, 16), dtype=np.float32)
    z[0, :len(vals)] = vals
    return z


@pytest.mark.parametrize("vals,ts,byte,codes", [
    # amax 6, tensor scale 1: 6 * fl(1/6) rounds to 1.0 -> scale 1.0; elements are codewords
    ([6, 3, -1.5, 0.5, -0.0], 1.0, 0x38, [7, 5, 8 | 3, 1, 8]),
    # amax 12: scale 2.0, elements halved; 5/2 = 2.5 is a tie between 2 and 3 -> 2, and -7/2 = -3.5 a
    # tie between 3 and 4 -> 4 (the neighbour with mantissa bit 0)
    ([12, 5, -7, 1], 1.0, 0x40, [7, 4, 8 | 6, 1]),
    # amax 7: 7/6 = 1.1667 lies between 1.125 and 1.25 -> 1.125 (0x39); 7/1.125 = 6.2 saturates
    ([7, 3.375, -1.6875], 1.0, 0x39, [7, 5, 8 | 3]),
    # tensor scale 2^-3: amax 0.75 -> 0.75/6/0.125 = 1.0 -> scale byte 1.0, dec = 0.125
    ([0.75, 0.25, -0.0625], 0.125, 0x38, [7, 4, 8 | 1]),
    # top of the range: amax = 6 * 448 with tensor scale 1 -> 0x7E
    ([2688, 1344, 2688 * 0.25], 1.0, 0x7E, [7, 5, 3]),
    # beyond the range of the scale: saturates at 448, elements saturate at 6
    ([5376, 2688], 1.0, 0x7E, [7, 7]),
    # far below the tensor scale: the block scale rounds to zero and the block encodes as zeros
    ([1e-4, -1e-4], 1.0, 0x00, [0, 8]),
])
def test_hand_worked_blocks(vals, ts, byte, codes):
    c, sb = O.quantize_nvfp4(_blk(vals), ts)
    assert sb[0, 0] == byte
    assert c[0, :len(codes)].tolist() == codes
    assert (c[0, len(codes):] == 0).all()


def test_subnormal_scale_bytes_are_used():
    # amax = 6 * 2^-9 (smallest positive E4M3) with tensor scale 1
    c, sb = O.quantize_nvfp4(_blk([6 * 2.0 ** -9, 3 * 2.0 ** -9]), 1.0)
    assert sb[0, 0] == 0x01 and c[0, :2].tolist() == [7, 5]


def test_error_bound_and_scale_range():
    """The block scale is within 2^-4 relative of amax/6 (3 mantissa bits), so the scaled block
    maximum lies in 6/(1+1/16) .. 6(1+1/16) and every element is within one code unit (the
    largest gap of the codebook is 2, half of it 1) of its codeword: |z - z^| <= dec."""
    g = np.random.default_rng(3)
    z = (g.standard_t(3, size=(64, 512)) * np.exp(g.uniform(-3, 3, size=(64, 1)))).astype(np.float32)
    ts = O.tensor_scale_from_amax(np.abs(z).max())
    codes, sb = O.quantize_nvfp4(z, ts)
    dec = O.e4m3_value(sb) * float(ts)
    amax = np.abs(z.astype(np.float64)).reshape(64, -1, 16).max(-1)
    normal = sb >= 0x08
    ratio = amax[normal] / dec[normal]
    assert ratio.min() >= 6 / (1 + 1 / 16) - 1e-6 and ratio.max() <= 6 * (1 + 1 / 16) + 1e-6
    err = np.abs(O.dequantize_nvfp4(codes, sb, ts) - z).reshape(64, -1, 16)
    assert (err[normal] <= dec[normal][:, None] * (1 + 1e-6)).all()
    assert sb.max() == 0x7E                              # the tensor maximum uses the top of E4M3
    # sign bits are the input's
    assert np.array_equal(codes >> 3, np.signbit(z).astype(np.uint8))


def test_idempotent_on_its_own_output():
    g = np.random.default_rng(4)
    z = g.standard_normal((32, 256)).astype(np.float32)
    ts = O.tensor_scale_from_amax(np.abs(z).max())
    codes, sb = O.quantize_nvfp4(z, ts)
    zq = O.dequantize_nvfp4(codes, sb, ts).astype(np.float32)
    codes2, sb2 = O.quantize_nvfp4(zq, ts)
    top = ((codes & 7).reshape(32, -1, 16).max(-1) == 7)          # blocks whose maximum sits on 6
    assert np.array_equal(sb2[top], sb[top])
    same = np.repeat(top, 16, axis=1)
    assert np.array_equal((codes2 & 7)[same], (codes & 7)[same])


def test_tiny_gemm_against_exact_rational_arithmetic():
    g = np.random.default_rng(5)
    M, N, K = 3, 4, 32
    ac = g.integers(0, 16, (M, K), dtype=np.uint8)
    wc = g.integers(0, 16, (N, K), dtype=np.uint8)
    asb = g.integers(0x20, 0x50, (M, K // 16), dtype=np.uint8)
    wsb = g.integers(0x20, 0x50, (N, K // 16), dtype=np.uint8)
    a_ts, w_ts = np.float32(0.37), np.float32(1.9e-3)
    book = [Fraction(0), Fraction(1, 2), Fraction(1), Fraction(3, 2), Fraction(2), Fraction(3), Fraction(4), Fraction(6)]

    def e4m3(b):                                         # from the format's definition
        ef, m = (int(b) >> 3) & 15, int(b) & 7
        return Fraction(m, 8) * Fraction(1, 64) if ef == 0 else (1 + Fraction(m, 8)) * Fraction(2) ** (ef - 7)

    def val(c, s, ts):
        v = book[int(c) & 7] * e4m3(s) * Fraction(float(ts))
        return -v if int(c) & 8 else v

    got = O.gemm_nvfp4(ac, asb, a_ts, wc, wsb, w_ts)
    for m in range(M):
        for n in range(N):
            acc = sum(val(ac[m, k], asb[m, k // 16], a_ts) * val(wc[n, k], wsb[n, k // 16], w_ts) for k in range(K))
            assert abs(got[m, n] - float(acc)) <= 1e-12 * max(1.0, abs(float(acc)))


def test_scale_layout_is_a_bijection_and_matches_the_32_wide_layout_rule():
    rows, k = 300, 16 * 13
    sb = np.random.default_rng(6).integers(1, 255, (rows, k // 16), dtype=np.uint8)
    buf = O.nv_swizzle_scales(sb, k)
    assert buf.size == O.nv_scale_layout_bytes(rows, k) == 3 * 4 * 512
    assert np.array_equal(O.nv_unswizzle_scales(buf, rows, k), sb)
    # same tiling rule as the MXFP4 scales: a K of 16*n here sits where a K of 32*n sits there
    rr, cc = np.meshgrid(np.arange(rows), np.arange(k // 16), indexing="ij")
    assert np.array_equal(O.nv_scale_layout_offset(rr, cc, k), O.scale_layout_offset(rr, cc, 2 * k))


def test_rotation_with_16_wide_blocks_and_its_32_wide_form_agree():
    g = np.random.default_rng(7)
    d = 64
    bits = lambda a: (np.asarray(a, np.float32).view(np.uint32) >> 16).astype(np.uint16)
    x = bits(g.standard_normal((5, d)))
    r = bits(g.standard_normal((d, d)) / 8)
    ri = bits(g.standard_normal((d // 16, 16, 16)) / 4)
    z16 = O.rotate_blocks(x, r, ri)
    z32 = O.rotate(x, r, O.expand_intra16(ri))
    assert np.allclose(z16, z32, rtol=0, atol=1e-12)
    # identity rotations leave x alone; energy is what the matrices make of it
    assert np.array_equal(O.rotate_blocks(x, None, None), O.decode_bf16(x))


def test_rotated_linear_identity_chain_recovers_the_product_up_to_quantization():
    g = np.random.default_rng(8)
    M, d, N = 8, 64, 16
    bits = lambda a: (np.asarray(a, np.float32).view(np.uint32) >> 16).astype(np.uint16)
    x = bits(g.standard_normal((M, d)))
    eye = bits(np.eye(d))
    eye16 = bits(np.broadcast_to(np.eye(16), (d // 16, 16, 16)))
    w = g.standard_normal((d, N)) * 0.05
    wc, wsb, wts = O.prepare_weights_nvfp4(eye, eye16, w)
    xts = O.tensor_scale_from_amax(np.abs(O.decode_bf16(x)).max())
    out, codes, sb = O.rotated_linear_nvfp4(x, eye, eye16, xts, wc, wsb, wts)
    ref = O.decode_bf16(x) @ w
    assert np.linalg.norm(out - ref) / np.linalg.norm(ref) < 0.2     # two 4-bit operands
    assert np.linalg.norm(O.dequantize_nvfp4(wc, wsb, wts) - w.T) / np.linalg.norm(w) < 0.12


def _lattice(codes):
    mag = (codes & 7).astype(np.int64)
    return np.where(codes & 8, -mag, mag)


def _exact_block_by_fractions(z_block, ts):
    """One 16-element block by the format's definition in exact rational arithmetic (pure Python)."""
    vals = [Fraction(float(v)) for v in O.e4m3_value(np.arange(0x7F, dtype=np.uint8))]
    book = [Fraction(float(c)) for c in O.CODEBOOK]

    def nearest_even(x, grid):
        best = min(range(len(grid)), key=lambda i: (abs(grid[i] - x), i % 2))
        return best

    zs = [Fraction(float(v)) for v in z_block]
    t = Fraction(float(np.float32(ts)))
    amax = max(abs(v) for v in zs)
    byte = nearest_even(min(amax / (6 * t), Fraction(448)), vals)
    if byte == 0:
        return byte, [(8 if np.signbit(v) else 0) for v in z_block]
    dec = vals[byte] * t
    codes = []
    for v, f in zip(z_block, zs):
        mag = nearest_even(min(abs(f) / dec, Fraction(6)), book)
        codes.append((8 if np.signbit(v) else 0) | mag)
    return byte, codes


def test_exact_definition_matches_rational_arithmetic_block_by_block():
    """quantize_nvfp4_exact (float64 divisions) against the definition in exact fractions, on blocks
    with tensor scales that are not powers of two, including a block on an E4M3 tie."""
    g = np.random.default_rng(21)
    for ts in (1.0, 0.37, 3.1e-4, 1.0 / 3.0, 250.0):
        z = (g.standard_t(3, size=(24, 16)) * float(ts) * np.exp(g.uniform(-2, 6, size=(24, 1)))).astype(np.float32)
        z[0] = 0.0
        z[1, 0] = np.float32(6.0 * 1.0625 * float(np.float32(ts)))       # amax / (6 ts) near the tie 1.0625
        codes, sb = O.quantize_nvfp4_exact(z, ts)
        for r in range(z.shape[0]):
            byte, want = _exact_block_by_fractions(z[r], ts)
            assert sb[r, 0] == byte, (ts, r)
            assert codes[r].tolist() == want, (ts, r)


def test_float32_recipe_is_the_exact_definition_up_to_its_roundings():
    """The float32 recipe (reciprocal multiplies, three roundings of 2^-24 per decision) against the
    exact definition on heavy-tailed blocks with tensor scales that are not powers of two.  A
    decision can move only for a value within ~2^-22 relative of a threshold: E4M3 has 8 thresholds
    per octave and e2m1 7 over [0, 6], so the expected rate is of order 1e-6 per block or element.
    Bound asserted: at most 1e-5 of the block scales differ, each by one E4M3 step; outside those
    blocks at most 1e-5 of the elements differ; every differing element, inside those blocks too
    (one E4M3 step moves a scaled value by at most 12.5 %, less than one codebook gap), is one
    lattice step away."""
    g = np.random.default_rng(5)
    n_blocks = n_elems = d_blocks = d_elems = 0
    for mul in (1.0, 0.37, 3.1e-4, 250.0, 1.0 / 3.0, 0.7071):
        z = (g.standard_t(3, size=(1024, 1024)) * np.exp(g.uniform(-4, 4, size=(1024, 1)))).astype(np.float32)
        ts = np.float32(np.abs(z).max() / (6 * 448) * mul * 1.2345)
        c32, s32 = O.quantize_nvfp4(z, ts)
        cex, sex = O.quantize_nvfp4_exact(z, ts)
        step = np.abs(s32.astype(np.int64) - sex.astype(np.int64))
        assert step.max() <= 1
        lat = np.abs(_lattice(c32) - _lattice(cex))
        assert lat.max() <= 1
        same = np.repeat(step == 0, 16, axis=1)
        n_blocks += step.size
        n_elems += lat.size
        d_blocks += int((step != 0).sum())
        d_elems += int(((lat != 0) & same).sum())
        assert np.array_equal(c32 >> 3, cex >> 3)                      # sign bits never differ
    assert d_blocks <= 1e-5 * n_blocks and d_elems <= 1e-5 * n_elems, (d_blocks, n_blocks, d_elems, n_elems)
