"""Plain CPU oracle of the rotated linear layer in the NVFP4 format (the paper's format study,
Section 6 "Generalizability to Other Formats": the same rotations, another 4-bit block format).

TEST INFRASTRUCTURE, like the rest of this package: never on the product path, shares no code
with it.

The paper names the format and prints accuracies, not its arithmetic; the format itself is public
(e2m1 elements, blocks of 16 along K, one FP8 E4M3 scale per block, one float32 scale per tensor).
What the paper leaves open is fixed here, each point a reading:

  * block size: the intra-block rotation acts inside a quantization block, so K = 16 here:
    R_intra is [d/16, 16, 16].
  * decoding:  x^ = codeword * e4m3(scale byte) * tensor_scale.
  * the tensor scale is an input (calibrated or computed beforehand); the usual choice,
    amax(tensor) / (6 * 448), maps the largest block's scale to the top of E4M3
    (`tensor_scale_from_amax`).
  * encoding, in float32 arithmetic (every operation below is one IEEE float32 operation,
    round to nearest even; this is the precision the kernel takes the decision in):
        c      = 1 / (6 * tensor_scale)
        byte   = E4M3(amax_block * c)      nearest, ties to even mantissa, saturating at 448
        dec    = e4m3(byte) * tensor_scale
        r      = 1 / dec                   (0 if byte == 0: the block encodes as zeros)
        a      = z * r
        code   = nearest e2m1 codeword to |a|, ties to even, saturating at 6; sign bit copied
  * scale bytes live in the same 128-row x 4-column tiled layout as the MXFP4 scales, with
    K/16 columns.

  * the format's plain definition, without any float32 step, is `quantize_nvfp4_exact`:
        byte = E4M3(amax_block / (6 * tensor_scale)),  code = e2m1(z / (e4m3(byte) * tensor_scale))
    in float64.  The float32 recipe above is that definition up to its own roundings (three per
    decision, each 2^-24 relative): a decision can differ only for a value within about 2^-22
    relative of a rounding threshold, and then by one step.  A test measures it.

Pins (tests/test_oracle_nvfp4.py): the E4M3 table and encoder against ml_dtypes' float8_e4m3fn
over every bit pattern and around every rounding threshold; hand-worked blocks whose arithmetic
is exact (tensor scale a power of two); error bound |a - Q(a)| <= 1 code unit; idempotence;
a tiny GEMM against exact rational arithmetic in pure Python; the float32 recipe against the
exact definition on heavy-tailed blocks with tensor scales that are not powers of two (every
difference one step, at most a stated fraction), and against exact rational arithmetic on single
blocks.  The paper prints no worked example for this format: "parity unpinned" by the paper,
pinned by the format's definition.
"""
from __future__ import annotations

import numpy as np

from .torq_oracle import CODEBOOK, decode_bf16, _nearest_codeword

NV_BLOCK = 16
E4M3_MAX = 448.0

__all__ = [
    "NV_BLOCK", "E4M3_MAX", "e4m3_value", "encode_e4m3", "tensor_scale_from_amax", "rotate_blocks",
    "quantize_nvfp4", "quantize_nvfp4_exact", "dequantize_nvfp4", "gemm_nvfp4", "nv_scale_layout_bytes", "nv_scale_layout_offset",
    "nv_swizzle_scales", "nv_unswizzle_scales", "expand_intra16", "prepare_weights_nvfp4",
    "rotated_linear_nvfp4",
]


# --------------------------------------------------------------------------- E4M3
def e4m3_value(byte) -> np.ndarray:
    """FP8 E4M3 (the "fn" variant: no infinities, one NaN pattern per sign) bit pattern -> float64.
    1 sign, 4 exponent bits (bias 7), 3 mantissa bits; exponent field 0 = subnormal m/8 * 2^-6;
    0x7F / 0xFF = NaN; largest finite 0x7E = 1.75 * 2^8 = 448."""
    b = np.asarray(byte, dtype=np.uint8).astype(np.int64)
    ef = (b >> 3) & 0xF
    m = b & 7
    mag = np.where(ef == 0, np.ldexp(m / 8.0, -6), np.ldexp(1.0 + m / 8.0, ef - 7))
    mag = np.where((b & 0x7F) == 0x7F, np.nan, mag)
    return np.where(b & 0x80, -mag, mag)


_E4M3_POS = e4m3_value(np.arange(0x7F, dtype=np.uint8))       # 0 .. 448, increasing with the byte


def encode_e4m3(v) -> np.ndarray:
    """Non-negative finite values -> E4M3 byte: nearest representable value, a tie goes to the
    even byte (mantissa bit 0), anything above 448 saturates to 448 (0x7E)."""
    v = np.asarray(v, dtype=np.float64)
    assert np.all(v >= 0) and np.all(np.isfinite(v))
    dist = np.abs(v[..., None] - _E4M3_POS)                    # [..., 127]
    best = dist.min(axis=-1, keepdims=True)
    hit = dist == best
    idx = np.arange(0x7F)
    even = hit & (idx % 2 == 0)
    return np.where(even.any(axis=-1), np.argmax(even, axis=-1), np.argmax(hit, axis=-1)).astype(np.uint8)


def tensor_scale_from_amax(amax) -> np.float32:
    """The usual per-tensor scale: the largest block scale amax/6 lands on 448."""
    return np.float32(np.float32(amax) / np.float32(6.0 * E4M3_MAX))


# ------------------------------------------------------------------------ rotation
def rotate_blocks(x_bits, r_inter_bits, r_intra_bits, block: int = NV_BLOCK) -> np.ndarray:
    """Algorithm 3 steps 1-3 with blocks of `block` features: y = x R_inter (dense d x d),
    z[:, block b] = y[:, block b] R_intra[b].  bfloat16 bit patterns in, float64 out;
    None = identity."""
    x = decode_bf16(x_bits)
    m, d = x.shape
    assert d % block == 0
    y = x if r_inter_bits is None else x @ decode_bf16(r_inter_bits)
    if r_intra_bits is None:
        return y.copy()
    ri = decode_bf16(r_intra_bits)
    assert ri.shape == (d // block, block, block)
    z = np.empty_like(y)
    for b in range(d // block):
        z[:, b * block:(b + 1) * block] = y[:, b * block:(b + 1) * block] @ ri[b]
    return z


def expand_intra16(r_intra_bits) -> np.ndarray:
    """[d/16,16,16] -> [d/32,32,32] bit patterns: blocks 2b and 2b+1 on the diagonal of 32 x 32
    block b, zeros elsewhere (the same linear map, written with 32-wide blocks)."""
    r = np.asarray(r_intra_bits, dtype=np.uint16)
    nb = r.shape[0]
    assert nb % 2 == 0 and r.shape[1:] == (16, 16)
    out = np.zeros((nb // 2, 32, 32), dtype=np.uint16)
    out[:, :16, :16] = r[0::2]
    out[:, 16:, 16:] = r[1::2]
    return out


# ----------------------------------------------------------------------- quantizer
def quantize_nvfp4(z32: np.ndarray, tensor_scale, rows_per_chunk: int = 256):
    """float32 [M,d] -> (codes [M,d] uint8 = sign<<3 | magnitude index, scale bytes [M,d/16]),
    by the float32 recipe in the module header."""
    z32 = np.asarray(z32)
    assert z32.dtype == np.float32 and z32.ndim == 2 and z32.shape[1] % NV_BLOCK == 0
    ts = np.float32(tensor_scale)
    assert ts > 0 and np.isfinite(ts)
    m, d = z32.shape
    nb = d // NV_BLOCK
    one = np.float32(1.0)
    c = one / (np.float32(6.0) * ts)
    codes = np.empty((m, d), dtype=np.uint8)
    sbytes = np.empty((m, nb), dtype=np.uint8)
    for r0 in range(0, m, rows_per_chunk):
        blk = z32[r0:r0 + rows_per_chunk].reshape(-1, nb, NV_BLOCK)
        amax = np.abs(blk).max(axis=-1)                           # float32, exact
        byte = encode_e4m3((amax * c).astype(np.float32))
        dec = (e4m3_value(byte).astype(np.float32) * ts).astype(np.float32)
        with np.errstate(divide="ignore"):
            r = np.where(byte == 0, np.float32(0.0), one / dec).astype(np.float32)
        a = (blk * r[..., None]).astype(np.float32)
        mag = _nearest_codeword(np.abs(a.astype(np.float64)))
        sign = np.signbit(blk).astype(np.uint8)
        codes[r0:r0 + rows_per_chunk] = ((sign << 3) | mag).reshape(-1, d)
        sbytes[r0:r0 + rows_per_chunk] = byte
    return codes, sbytes


def quantize_nvfp4_exact(z32: np.ndarray, tensor_scale, rows_per_chunk: int = 256):
    """The format's definition with no float32 step: per 16-element block
        byte = E4M3(amax / (6 ts))   nearest, ties to the even byte, saturating at 448
        code = e2m1(z / (e4m3(byte) ts))   nearest, ties to even, saturating at 6; sign of z
    (a block whose scale byte is 0 encodes as zeros), every quotient one float64 division of
    exactly represented operands (the tensor scale is the float32 value given).  Same outputs as
    quantize_nvfp4."""
    z32 = np.asarray(z32)
    assert z32.dtype == np.float32 and z32.ndim == 2 and z32.shape[1] % NV_BLOCK == 0
    ts = np.float64(np.float32(tensor_scale))
    assert ts > 0 and np.isfinite(ts)
    m, d = z32.shape
    nb = d // NV_BLOCK
    codes = np.empty((m, d), dtype=np.uint8)
    sbytes = np.empty((m, nb), dtype=np.uint8)
    for r0 in range(0, m, rows_per_chunk):
        blk = z32[r0:r0 + rows_per_chunk].astype(np.float64).reshape(-1, nb, NV_BLOCK)
        amax = np.abs(blk).max(axis=-1)
        byte = encode_e4m3(amax / (6.0 * ts))
        dec = e4m3_value(byte) * ts
        with np.errstate(divide="ignore", invalid="ignore"):
            a = np.where((byte == 0)[..., None], 0.0, np.abs(blk) / dec[..., None])
        mag = _nearest_codeword(a)
        sign = np.signbit(blk).astype(np.uint8)
        codes[r0:r0 + rows_per_chunk] = ((sign << 3) | mag).reshape(-1, d)
        sbytes[r0:r0 + rows_per_chunk] = byte
    return codes, sbytes


def dequantize_nvfp4(codes, scale_bytes, tensor_scale) -> np.ndarray:
    """x^ = codeword * e4m3(scale) * tensor_scale, exact in float64."""
    codes = np.asarray(codes, dtype=np.uint8)
    m, d = codes.shape
    val = CODEBOOK[codes & 7] * np.where(codes & 8, -1.0, 1.0)
    s = e4m3_value(scale_bytes) * np.float64(np.float32(tensor_scale))
    return (val.reshape(m, d // NV_BLOCK, NV_BLOCK) * s[..., None]).reshape(m, d)


def gemm_nvfp4(a_codes, a_scales, a_ts, w_codes, w_scales, w_ts) -> np.ndarray:
    """out[m,n] = sum_k a^[m,k] w^[n,k] in float64."""
    return dequantize_nvfp4(a_codes, a_scales, a_ts) @ dequantize_nvfp4(w_codes, w_scales, w_ts).T


# ------------------------------------------------------- scale-factor byte layout
def nv_scale_layout_bytes(rows: int, k: int) -> int:
    return ((rows + 127) // 128) * ((k // NV_BLOCK + 3) // 4) * 512


def nv_scale_layout_offset(r, c, k: int):
    """Byte offset of the scale of (row r, 16-element block c): 512-byte tiles of 128 rows x 4
    blocks, row-tile major; inside a tile byte = (r%32)*16 + ((r%128)//32)*4 + c%4."""
    kb4 = (k // NV_BLOCK + 3) // 4
    r = np.asarray(r)
    c = np.asarray(c)
    return ((r // 128) * kb4 + c // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + (c % 4)


def nv_swizzle_scales(scale_bytes: np.ndarray, k: int, fill: int = 0) -> np.ndarray:
    rows, kb = scale_bytes.shape
    out = np.full(nv_scale_layout_bytes(rows, k), fill, dtype=np.uint8)
    rr, cc = np.meshgrid(np.arange(rows), np.arange(kb), indexing="ij")
    out[nv_scale_layout_offset(rr, cc, k)] = scale_bytes
    return out


def nv_unswizzle_scales(buf: np.ndarray, rows: int, k: int) -> np.ndarray:
    rr, cc = np.meshgrid(np.arange(rows), np.arange(k // NV_BLOCK), indexing="ij")
    return np.asarray(buf, dtype=np.uint8)[nv_scale_layout_offset(rr, cc, k)]


# ------------------------------------------------------------------- whole path
def prepare_weights_nvfp4(r_inter_bits, r_intra_bits, w: np.ndarray):
    """W' = R~^T W for W [d,N], R~ = R_inter blockdiag(R_intra[b]) (16-wide blocks), stored [N,d],
    rounded once to float32, tensor scale from its amax, quantized along K.
    Returns (codes [N,d], scale bytes [N,d/16], tensor_scale)."""
    r = decode_bf16(r_inter_bits)
    ri = decode_bf16(r_intra_bits)
    rt = np.empty_like(r)
    for b in range(ri.shape[0]):
        rt[:, b * NV_BLOCK:(b + 1) * NV_BLOCK] = r[:, b * NV_BLOCK:(b + 1) * NV_BLOCK] @ ri[b]
    wp = np.ascontiguousarray((rt.T @ np.asarray(w, dtype=np.float64)).T).astype(np.float32)
    ts = tensor_scale_from_amax(np.abs(wp).max())
    codes, sb = quantize_nvfp4(wp, ts)
    return codes, sb, ts


def rotated_linear_nvfp4(x_bits, r_inter_bits, r_intra_bits, x_ts, w_codes, w_scales, w_ts):
    """Algorithm 3 end to end in NVFP4.  Returns (out float64 [M,N], codes, scale bytes)."""
    z32 = rotate_blocks(x_bits, r_inter_bits, r_intra_bits).astype(np.float32)
    codes, sb = quantize_nvfp4(z32, x_ts)
    return gemm_nvfp4(codes, sb, x_ts, w_codes, w_scales, w_ts), codes, sb
