"""Plain CPU oracle of the rotated linear layer in the MXINT4 format (the paper's format study,
Section 6 "Generalizability to Other Formats": the same rotations, an integer 4-bit block format).

TEST INFRASTRUCTURE, like the rest of this package: never on the product path, shares no code
with it.

The paper names the format and prints accuracies, not its arithmetic.  The reading taken here is
the microscaling recipe with an integer element in place of e2m1:

  * blocks of 32 along K, one E8M0 scale byte per block (as in MXFP4, same tiled byte layout);
  * elements are signed integers q in [-7, 7] (symmetric: -8 is never produced, so negating a
    block negates its codes); decoding x^ = q * 2^e;
  * shared exponent by the microscaling rule, e = floor(log2 amax) - emax_elem with emax_elem =
    floor(log2 7) = 2: the same e as MXFP4, clamped to [-127, 127], amax = 0 -> -127.  amax / 2^e
    lies in [4, 8); what exceeds 7.5 saturates to 7;
  * encoding q = clamp(rint(z / 2^e), -7, 7), rint = round half to even; z / 2^e is exact;
  * stored form: two's-complement nibbles, even element in the low nibble of a byte (`pack_int4`);
  * operand form for a tensor core without an integer 4-bit path: the FP8 E4M3 byte whose value
    is q (every integer of [-8, 8] is an E4M3 number), `int4_to_e4m3`.

Pins (tests/test_oracle_mxint4.py): hand-worked blocks; ties and saturation; the error bound
|z / 2^e - q| <= 1/2 below saturation; negation symmetry; idempotence; agreement with MXFP4 on
the scale bytes; the E4M3 bytes against ml_dtypes; a tiny GEMM in exact rational arithmetic.
The paper prints no worked example for this format: "parity unpinned" by the paper, pinned by the
definition above.
"""
from __future__ import annotations

import numpy as np

from .torq_oracle import K_BLOCK, merged_rotation, rotate, round_to_f32, shared_exponent
from .nvfp4_oracle import e4m3_value

INT4_MAX = 7

__all__ = [
    "INT4_MAX", "quantize_mxint4", "dequantize_mxint4", "gemm_mxint4", "pack_int4", "unpack_int4",
    "int4_to_e4m3", "e4m3_to_int4", "prepare_weights_mxint4", "rotated_linear_mxint4",
]


def quantize_mxint4(z32: np.ndarray, rows_per_chunk: int = 256):
    """float32 [M,d] -> (q [M,d] int8 in [-7,7], scale bytes [M,d/32] uint8 = e + 127)."""
    z32 = np.asarray(z32)
    assert z32.dtype == np.float32 and z32.ndim == 2 and z32.shape[1] % K_BLOCK == 0
    m, d = z32.shape
    nb = d // K_BLOCK
    q = np.empty((m, d), dtype=np.int8)
    sbytes = np.empty((m, nb), dtype=np.uint8)
    for r0 in range(0, m, rows_per_chunk):
        blk = z32[r0:r0 + rows_per_chunk].astype(np.float64).reshape(-1, nb, K_BLOCK)
        e = shared_exponent(np.abs(blk).max(axis=-1))
        a = np.ldexp(blk, (-e)[..., None])                      # z / 2^e, exact
        q[r0:r0 + rows_per_chunk] = np.clip(np.rint(a), -INT4_MAX, INT4_MAX).astype(np.int8).reshape(-1, d)
        sbytes[r0:r0 + rows_per_chunk] = (e + 127).astype(np.uint8)
    return q, sbytes


def dequantize_mxint4(q: np.ndarray, scale_bytes: np.ndarray) -> np.ndarray:
    """x^ = q * 2^e, exact in float64."""
    q = np.asarray(q, dtype=np.int8)
    m, d = q.shape
    e = np.asarray(scale_bytes).astype(np.int64) - 127
    return np.ldexp(q.astype(np.float64).reshape(m, d // K_BLOCK, K_BLOCK), e[..., None]).reshape(m, d)


def gemm_mxint4(a_q, a_scales, w_q, w_scales) -> np.ndarray:
    """out[m,n] = sum_k a^[m,k] w^[n,k] in float64."""
    return dequantize_mxint4(a_q, a_scales) @ dequantize_mxint4(w_q, w_scales).T


def pack_int4(q: np.ndarray) -> np.ndarray:
    """[M,d] integers in [-8,7] -> [M,d/2] bytes of two's-complement nibbles, even element low."""
    n = (np.asarray(q, dtype=np.int8).astype(np.int16) & 0xF).astype(np.uint8)
    return (n[:, 0::2] | (n[:, 1::2] << 4)).astype(np.uint8)


def unpack_int4(packed: np.ndarray) -> np.ndarray:
    p = np.asarray(packed, dtype=np.uint8)
    n = np.empty((p.shape[0], p.shape[1] * 2), dtype=np.int16)
    n[:, 0::2] = p & 0xF
    n[:, 1::2] = p >> 4
    return np.where(n >= 8, n - 16, n).astype(np.int8)


_E4M3_ALL = e4m3_value(np.arange(256, dtype=np.uint8))


def int4_to_e4m3(q: np.ndarray) -> np.ndarray:
    """The E4M3 byte whose value is q, for integers in [-8, 8]; zero is 0x00 for either sign."""
    q = np.asarray(q, dtype=np.int64)
    assert np.all(np.abs(q) <= 8)
    out = np.zeros(q.shape, dtype=np.uint8)
    for v in range(-8, 9):
        if v == 0:
            continue
        (hit,) = np.nonzero(_E4M3_ALL == float(v))
        assert hit.size == 1
        out[q == v] = hit[0]
    return out


def e4m3_to_int4(b: np.ndarray) -> np.ndarray:
    """Inverse of `int4_to_e4m3`; asserts that every byte decodes to an integer of [-8, 8]."""
    v = _E4M3_ALL[np.asarray(b, dtype=np.uint8)]
    assert np.all(np.isfinite(v)) and np.all(v == np.rint(v)) and np.all(np.abs(v) <= 8)
    return v.astype(np.int8)


def prepare_weights_mxint4(r_inter_bits, r_intra_bits, w: np.ndarray):
    """W' = R~^T W for W [d,N] (Algorithm 3, offline part), stored [N,d], rounded once to
    float32, quantized along K.  Returns (q [N,d] int8, scale bytes [N,d/32])."""
    rt = merged_rotation(r_inter_bits, r_intra_bits)
    wp = np.ascontiguousarray((rt.T @ np.asarray(w, dtype=np.float64)).T)
    return quantize_mxint4(round_to_f32(wp))


def rotated_linear_mxint4(x_bits, r_inter_bits, r_intra_bits, w_q, w_scales):
    """Algorithm 3 steps 1-5 with the MXINT4 quantizer.  Returns (Y float64, a_q, a_scales)."""
    z = round_to_f32(rotate(x_bits, r_inter_bits, r_intra_bits))
    a_q, a_s = quantize_mxint4(z)
    return gemm_mxint4(a_q, a_s, w_q, w_scales), a_q, a_s
