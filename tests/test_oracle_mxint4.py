"""Pins for the oracle's MXINT4 functions (format study of Section 6).  The format is the
microscaling recipe with a signed integer element: 32-element blocks, E8M0 scale, q in [-7, 7].

Each check restates the definition by a route the oracle does not use: hand-worked blocks,
brute force over every candidate integer, bounds and symmetries that follow from the definition,
ml_dtypes' float8_e4m3fn for the operand bytes, exact rational arithmetic in pure Python."""
from fractions import Fraction

import ml_dtypes
import numpy as np

import oracle as O


def _blk(vals):
    z = np.zeros((1, 32), dtype=np.float32)
    z[0, :len(vals)] = vals
    return z


def test_hand_worked_block_with_ties_and_saturation():
    # amax = 7.75 -> floor(log2) = 2 -> e = 0, scale byte 127: the values are their own quotients
    z = _blk([7.75, -7.5, 7.49, 6.5, 5.5, -4.5, 3.5, 2.5, -1.5, 0.5, -0.5, 0.49, 1.0, -7.0, 0.0, 4.51])
    q, sb = O.quantize_mxint4(z)
    assert sb.tolist() == [[127]]
    # halves go to the even neighbour; 7.5 -> 8 and 7.75 -> 8 saturate to 7
    assert q[0, :16].tolist() == [7, -7, 7, 6, 6, -4, 4, 2, -2, 0, 0, 0, 1, -7, 0, 5]
    assert (q[0, 16:] == 0).all()


def test_hand_worked_block_with_scaled_maximum():
    # amax = 0.3 = 1.2 * 2^-2 -> e = -2 - 2 = -4, byte 123; quotients z * 16
    z = _blk([0.3, -0.1, 0.03125, 0.09375, -0.21875])
    q, sb = O.quantize_mxint4(z)
    assert sb.tolist() == [[123]]
    # 4.8 -> 5, -1.6 -> -2, 0.5 -> 0, 1.5 -> 2, -3.5 -> -4
    assert q[0, :5].tolist() == [5, -2, 0, 2, -4]
    assert np.array_equal(O.dequantize_mxint4(q, sb)[0, :5], np.array([5, -2, 0, 2, -4]) / 16.0)


def test_zero_block_and_scale_clamps():
    q, sb = O.quantize_mxint4(np.zeros((2, 64), dtype=np.float32))
    assert (q == 0).all() and (sb == 0).all()
    tiny = _blk([1e-45, -3e-45])                        # float32 subnormals: e clamps at -127
    q, sb = O.quantize_mxint4(tiny)
    assert sb.tolist() == [[0]] and (q == 0).all()
    big = _blk([3.0e38, -1.0e38])                       # floor(log2) = 127 -> e = 125
    q, sb = O.quantize_mxint4(big)
    assert sb.tolist() == [[252]]
    assert q[0, :2].tolist() == [7, -2]                 # 3e38 / 2^125 = 7.05 -> 7, 1e38 / 2^125 = 2.35 -> -2


def test_scale_bytes_equal_the_mxfp4_scale_bytes():
    z = (np.random.default_rng(0).standard_normal((64, 256)) * np.exp(np.random.default_rng(1).uniform(-20, 20, (64, 1)))
         ).astype(np.float32)
    _, sb_int = O.quantize_mxint4(z)
    _, sb_fp = O.quantize_mxfp4(z)
    assert np.array_equal(sb_int, sb_fp)


def test_nearest_integer_by_brute_force_and_error_bound():
    rng = np.random.default_rng(2)
    z = (rng.standard_normal((32, 128)) * np.exp(rng.uniform(-8, 8, (32, 1)))).astype(np.float32)
    q, sb = O.quantize_mxint4(z)
    e = sb.astype(np.int64) - 127
    a = (z.astype(np.float64).reshape(32, 4, 32) / np.exp2(e)[..., None]).reshape(32, 128)
    # the block maximum lands in [4, 8)
    amax = np.abs(a).reshape(32, 4, 32).max(axis=-1)
    assert ((amax >= 4) & (amax < 8)).all()
    cands = np.arange(-7, 8)
    dist = np.abs(a[..., None] - cands)
    assert np.array_equal(dist.min(axis=-1), np.abs(a - q))          # q is a nearest candidate
    below = np.abs(a) <= 7.5
    assert (np.abs(a - q)[below] <= 0.5).all()
    assert (np.abs(q[~below]) == 7).all()
    # exact halves went to the even integer
    half = (np.abs(a) % 1.0) == 0.5
    assert (q[half & below] % 2 == 0).all()


def test_every_half_integer_rounds_to_even():
    pts = np.arange(-7.5, 8.0, 1.0)                      # -7.5 .. 7.5
    z = np.zeros((1, 32), dtype=np.float32)
    z[0, :pts.size] = pts
    z[0, 31] = 7.75                                      # fixes e = 0
    q, sb = O.quantize_mxint4(z)
    assert sb[0, 0] == 127
    want = [-7, -6, -6, -4, -4, -2, -2, 0, 0, 2, 2, 4, 4, 6, 6, 7]
    assert q[0, :pts.size].tolist() == want


def test_negation_symmetry_idempotence_and_scaling_by_powers_of_two():
    rng = np.random.default_rng(3)
    z = rng.standard_normal((16, 96)).astype(np.float32)
    q, sb = O.quantize_mxint4(z)
    qn, sbn = O.quantize_mxint4(-z)
    assert np.array_equal(qn, -q) and np.array_equal(sbn, sb)
    zh = O.dequantize_mxint4(q, sb).astype(np.float32)
    q2, sb2 = O.quantize_mxint4(zh)
    assert np.array_equal(O.dequantize_mxint4(q2, sb2), zh.astype(np.float64))
    q8, sb8 = O.quantize_mxint4(z * np.float32(8.0))
    assert np.array_equal(q8, q) and np.array_equal(sb8.astype(int), sb.astype(int) + 3)


def test_pack_and_unpack_nibbles():
    q = np.array([[-8, -7, -1, 0, 1, 7, 3, -4]], dtype=np.int8)
    p = O.pack_int4(q)
    # two's complement: -8 = 0x8, -7 = 0x9, -1 = 0xF, -4 = 0xC; even element in the low nibble
    assert p.tolist() == [[0x98, 0x0F, 0x71, 0xC3]]
    assert np.array_equal(O.unpack_int4(p), q)
    allq = np.arange(-8, 8, dtype=np.int8).reshape(1, 16)
    assert np.array_equal(O.unpack_int4(O.pack_int4(allq)), allq)


def test_e4m3_operand_bytes_match_ml_dtypes():
    q = np.arange(-8, 9)
    b = O.int4_to_e4m3(q)
    assert np.array_equal(b.view(ml_dtypes.float8_e4m3fn).astype(np.float64), q.astype(np.float64))
    want = q.astype(np.float32).astype(ml_dtypes.float8_e4m3fn).view(np.uint8)
    assert np.array_equal(b, want)
    assert b[8] == 0 and b[9] == 0x38 and b[15] == 0x4E and b[1] == 0xCE     # 0, 1, 7, -7
    assert np.array_equal(O.e4m3_to_int4(b), q.astype(np.int8))


def test_tiny_gemm_in_exact_rational_arithmetic():
    rng = np.random.default_rng(4)
    a = (rng.standard_normal((3, 64)) * 3).astype(np.float32)
    w = (rng.standard_normal((5, 64)) * 0.02).astype(np.float32)
    aq, asb = O.quantize_mxint4(a)
    wq, wsb = O.quantize_mxint4(w)
    got = O.gemm_mxint4(aq, asb, wq, wsb)
    for m in range(3):
        for n in range(5):
            acc = Fraction(0)
            for k in range(64):
                sa = Fraction(2) ** (int(asb[m, k // 32]) - 127)
                sw = Fraction(2) ** (int(wsb[n, k // 32]) - 127)
                acc += int(aq[m, k]) * sa * int(wq[n, k]) * sw
            assert abs(Fraction(float(got[m, n])) - acc) <= abs(acc) * Fraction(1, 2 ** 48) + Fraction(1, 2 ** 200)


def test_rotated_linear_is_rotate_then_quantize_then_gemm_and_undoes_the_rotation():
    from paper_2605_19561_b200 import inputs as I
    cfg = I.CONFIGS["tiny"]
    d, n, m = 128, 32, 24
    x = I.activations(cfg, m, d)
    r_inter, r_intra, _, _ = I.rotations(cfg, d)
    w = I.weights(cfg, d, n)
    wq, ws = O.prepare_weights_mxint4(r_inter, r_intra, w)
    y, aq, asb = O.rotated_linear_mxint4(x, r_inter, r_intra, wq, ws)
    # the rotations cancel: the quantized product approximates x W (int4: coarse, hence the loose bound)
    ref = O.decode_bf16(x) @ np.asarray(w, dtype=np.float64)
    rel = np.linalg.norm(y - ref) / np.linalg.norm(ref)
    assert rel < 0.25
    # and it is exactly the GEMM of the quantized operands
    assert np.array_equal(y, O.dequantize_mxint4(aq, asb) @ O.dequantize_mxint4(wq, ws).T)
