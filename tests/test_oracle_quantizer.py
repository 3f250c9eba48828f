"""Pins for the oracle's MXFP4 quantizer (Eq. 1; Algorithm 3 step 4).

Each check restates the format by a route the oracle does not use: an explicit
decision-threshold table, ml_dtypes' float4_e2m1fn cast, the float32 exponent field,
hand-derived worked values, and invariants of the encoding.
"""
import os

import ml_dtypes
import numpy as np
import pytest

import oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _block(first, second=0.0):
    n = max(np.size(first), np.size(second))
    z = np.zeros((n, 32), dtype=np.float32)
    z[:, 0] = first
    z[:, 1] = second
    return z


def _threshold_code(a):
    """e2m1 magnitude index by the midpoint table, ties to the even index, saturating."""
    a = abs(float(a))
    if a <= 0.25: return 0
    if a < 0.75: return 1
    if a <= 1.25: return 2
    if a < 1.75: return 3
    if a <= 2.5: return 4
    if a < 3.5: return 5
    if a <= 5.0: return 6
    return 7


def test_codebook_matches_paper():
    rows = [l.split() for l in open(os.path.join(GOLD, "e2m1_codebook.txt")) if l[0] != "#"]
    for idx, val in rows:
        assert O.CODEBOOK[int(idx)] == float(val)
    # the codebook is the e2m1 value set: sign, 2 exponent bits, 1 mantissa bit
    vals = [float(np.array([i], dtype=np.uint8).view(ml_dtypes.float4_e2m1fn).astype(np.float32)[0]) for i in range(8)]
    assert vals == list(O.CODEBOOK)


def _all_bf16_values():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    with np.errstate(invalid="ignore"):
        v = O.decode_bf16(bits).astype(np.float32)
    return v[np.isfinite(v)]


def test_every_bf16_input_at_unit_scale():
    """Block [6, v, 0...] has e = 0, so v is projected on the bare codebook."""
    v = _all_bf16_values()
    v = v[np.abs(v) < 8.0]
    codes, sb = O.quantize_mxfp4(_block(6.0, v))
    assert (sb[:, 0] == 127).all()
    want_mag = np.array([_threshold_code(x) for x in v], dtype=np.uint8)
    want = want_mag | (np.signbit(v).astype(np.uint8) << 3)
    assert (codes[:, 1] == want).all()
    # second opinion: the library cast (round to nearest even, saturating, sign kept)
    lib = v.astype(ml_dtypes.float4_e2m1fn).view(np.uint8) & 0xF
    assert (codes[:, 1] == lib).all()
    assert (codes[:, 0] == 7).all() and (codes[:, 2:] == 0).all()


@pytest.mark.parametrize("k", [-20, -3, 0, 5, 40])
def test_float32_neighbourhood_of_each_threshold(k):
    """+-8 ulps around each decision boundary, at several scales 2^k."""
    thr = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], dtype=np.float32)
    pts = []
    for t in thr:
        x = np.float32(t)
        lo = x
        for _ in range(8):
            lo = np.nextafter(lo, np.float32(0))
        cur = lo
        for _ in range(17):
            pts.append(cur)
            cur = np.nextafter(cur, np.float32(np.inf))
    a = np.array(pts, dtype=np.float32)
    for sign in (1.0, -1.0):
        v = (sign * np.ldexp(a, k)).astype(np.float32)
        codes, sb = O.quantize_mxfp4(_block(np.float32(np.ldexp(6.0, k)), v))
        assert (sb[:, 0] == 127 + k).all()
        want = np.array([_threshold_code(x) for x in a], dtype=np.uint8) | (8 if sign < 0 else 0)
        assert (codes[:, 1] == want).all()
        lib = (sign * a).astype(np.float32).astype(ml_dtypes.float4_e2m1fn).view(np.uint8) & 0xF
        assert (codes[:, 1] == lib).all()


def test_projection_is_nearest_and_monotone():
    g = np.random.default_rng(1)
    a = g.uniform(-7.9, 7.9, size=4096).astype(np.float32)
    codes, _ = O.quantize_mxfp4(_block(6.0, a))
    deq = O.CODEBOOK[codes[:, 1] & 7]
    # no other codeword is strictly closer
    d_all = np.abs(np.abs(a.astype(np.float64))[:, None] - O.CODEBOOK[None, :])
    assert (np.abs(np.abs(a.astype(np.float64)) - deq) <= d_all.min(1)).all()
    order = np.argsort(a)
    signed = np.where(codes[:, 1] & 8, -deq, deq)
    assert (np.diff(signed[order]) >= 0).all()


def test_scale_rule_worked_values():
    for line in open(os.path.join(GOLD, "scale_worked_values.txt")):
        if line.startswith("#") or not line.strip():
            continue
        amax, byte, code = line.split()
        codes, sb = O.quantize_mxfp4(_block(np.float32(amax)))
        assert sb[0, 0] == int(byte), line
        assert (codes[0, 0] & 7) == int(code), line


def test_scale_rule_every_bf16_amax():
    v = _all_bf16_values()
    v = v[v > 0]
    codes, sb = O.quantize_mxfp4(_block(v))
    # exponent field of the float32 value, minus the element format's emax (2)
    field = (v.view(np.uint32) >> 23) & 0xFF
    normal = field > 0
    want = np.clip(field.astype(np.int64) - 2, 0, 254)
    assert (sb[normal, 0] == want[normal]).all()
    e = sb[:, 0].astype(np.int64) - 127
    ratio = np.ldexp(v.astype(np.float64), -e)
    unclamped = (e > -127) & (e < 127)
    assert ((ratio >= 4) & (ratio < 8))[unclamped].all()
    assert np.isin(codes[unclamped, 0], [6, 7]).all()
    assert sb.max() <= 254
    # python's own floor(log2) as a third route
    import math
    for x, b in zip(v[::97], sb[::97, 0]):
        assert b == min(max(math.floor(math.log2(float(x))) - 2, -127), 127) + 127


def test_subnormal_and_extreme_scales():
    tiny = np.float32(1e-45)            # smallest subnormal, 2^-149
    codes, sb = O.quantize_mxfp4(_block(tiny))
    assert sb[0, 0] == 0 and codes[0, 0] == 0     # e clamps to -127; 2^-149 * 2^127 = 2^-22 -> 0
    big = np.float32(3.0e38)            # 2^127 <= big < 2^128
    codes, sb = O.quantize_mxfp4(_block(big))
    assert sb[0, 0] == 127 + 125
    zero = np.zeros((1, 32), np.float32)
    zero[0, 3] = -0.0
    codes, sb = O.quantize_mxfp4(zero)
    assert sb[0, 0] == 0 and codes[0, 3] == 8 and codes[0, 0] == 0


def test_sign_kept_when_magnitude_rounds_to_zero():
    codes, _ = O.quantize_mxfp4(_block(6.0, np.array([-0.1, 0.1, -0.25, -0.2500001], np.float32)))
    assert list(codes[:, 1]) == [8, 0, 8, 9]


def test_dequantized_set_and_idempotence():
    g = np.random.default_rng(2)
    z = (g.standard_t(3, size=(64, 256)) * np.exp(g.normal(0, 3, size=(64, 1)))).astype(np.float32)
    codes, sb = O.quantize_mxfp4(z)
    deq = O.dequantize(codes, sb)
    e = sb.astype(np.int64) - 127
    unit = np.abs(np.ldexp(deq.reshape(64, 8, 32), -e[..., None]))
    assert np.isin(unit, O.CODEBOOK).all()
    # relative error of a block is bounded by the grid: |z - z^| <= s_b for unsaturated, <= 2 s_b overall
    err = np.abs(deq - z).reshape(64, 8, 32)
    assert (err <= 2.0 * np.ldexp(1.0, e)[..., None]).all()
    # quantizing the dequantized values reproduces codes and scales
    codes2, sb2 = O.quantize_mxfp4(deq.astype(np.float32))
    assert (sb2 == sb).all()
    assert ((codes2 & 7) == (codes & 7)).all()


def test_pack_nibble_order_and_roundtrip():
    c = np.array([[1, 2, 0xF, 0, 7, 8]], dtype=np.uint8)
    assert list(O.pack_codes(c)[0]) == [0x21, 0x0F, 0x87]
    g = np.random.default_rng(3)
    c = g.integers(0, 16, size=(5, 64), dtype=np.uint8)
    assert (O.unpack_codes(O.pack_codes(c)) == c).all()


def test_scale_layout_is_the_128x4_tiling():
    k = 1024                       # 32 K-blocks -> 8 tiles per row-tile
    assert O.scale_layout_bytes(256, k) == 2 * 8 * 512
    assert O.scale_layout_offset(0, 0, k) == 0
    assert O.scale_layout_offset(0, 1, k) == 1
    assert O.scale_layout_offset(1, 0, k) == 16
    assert O.scale_layout_offset(32, 0, k) == 4
    assert O.scale_layout_offset(31, 3, k) == 31 * 16 + 3
    assert O.scale_layout_offset(127, 3, k) == 511
    assert O.scale_layout_offset(0, 4, k) == 512
    assert O.scale_layout_offset(128, 0, k) == 8 * 512
    rr, cc = np.meshgrid(np.arange(256), np.arange(32), indexing="ij")
    off = O.scale_layout_offset(rr, cc, k).ravel()
    assert sorted(off) == list(range(256 * 32))      # a bijection when nothing is padded
    sb = np.random.default_rng(4).integers(0, 255, size=(200, 24), dtype=np.uint8)
    buf = O.swizzle_scales(sb, 24 * 32)
    assert buf.size == O.scale_layout_bytes(200, 24 * 32)
    assert (O.unswizzle_scales(buf, 200, 24 * 32) == sb).all()
