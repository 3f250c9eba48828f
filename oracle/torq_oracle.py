"""Plain, slow, fp64 CPU oracle of TORQ's online inference path (Algorithm 3).

TEST INFRASTRUCTURE.  This module is the yardstick the CUDA kernels are compared
against; it is never on the product path, shares no code with it, and imports
nothing from the product package.  Everything is numpy in float64; matrix
products use numpy's matmul as a library step, everything else is written out.

The path (Algorithm 3 of the paper, with Eq. 1 for the quantizer):

  1. reshape : a token's d features are viewed as B = d/32 blocks of K = 32.
  2. inter   : Y = X . R_inter              (dense d x d orthogonal matrix)
  3. intra   : Z_b = Y_b . R_intra[b]       (one 32 x 32 matrix per block)
  4. quantize: per (token, block)  s = 2^e,  a = z / s,  code = Q(a),
               Q = nearest neighbour on the e2m1 codebook (Eq. 1)
  5. linear  : out = dequant(Z) . dequant(W')^T  with W' = R~^T W folded and
               quantized offline (step 5, option B: weight fusion)

Readings of points the paper leaves open (each is also listed in the design notes):
  * shared scale: Eq. 1 prints s = 2^floor(log2 amax); taken literally the block
    maximum would land in [1, 2) and the codewords 3, 4, 6 could never be used,
    which contradicts the S-step (Eq. 5), which maps the block maximum to the top
    codeword 6.  The OCP MX rule e = floor(log2 amax) - 2 is used: amax / 2^e
    lies in [4, 8) and values above 6 saturate.  e is clamped to [-127, 127]; an
    all-zero block takes e = -127.  The stored scale byte is E8M0: e + 127.
  * the scale is taken from the data at run time (per token and block), not from
    a stored matrix S.
  * ties of the nearest-neighbour projection go to the codeword whose mantissa
    bit is 0 (round to nearest even); magnitudes above 6 map to 6.
  * the sign bit is copied from the input even when the magnitude rounds to 0.
  * the quantizer is defined on float32 input: the fp64 rotation result is
    rounded once to float32 (nearest even) before step 4.
  * rotations and activations arrive as bfloat16 bit patterns and are used at
    exactly those values.
  * row-vector convention: tokens are rows, rotations multiply from the right.

Pins (tests/test_oracle_*.py): brute force over every bfloat16 input and around
every decision threshold, ml_dtypes' float4_e2m1fn / float8_e8m0fnu as a second
opinion, scale invariants, exact special-case rotations (identity, permutation,
Walsh-Hadamard), energy conservation, the unquantized identity chain, and tiny
GEMMs against pure Python loops.  The end-to-end chain has no printed worked
example in the paper: "parity unpinned" by the paper for the composition itself,
each stage is pinned separately.
"""
from __future__ import annotations

import numpy as np

K_BLOCK = 32
# Eq. 1: the positive half of the e2m1 codebook, index = 3-bit magnitude code.
CODEBOOK = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0], dtype=np.float64)
E2M1_EMAX = 2  # largest power of two in the codebook is 2^2

__all__ = [
    "K_BLOCK", "CODEBOOK", "decode_bf16", "rotate", "rotate_structured", "round_to_f32", "shared_exponent",
    "quantize_mxfp4", "pack_codes", "unpack_codes", "dequantize", "gemm_dequant",
    "round_to_bf16", "merged_rotation", "prepare_weights", "scale_layout_offset",
    "scale_layout_bytes", "swizzle_scales", "unswizzle_scales", "rotated_linear",
    "codeword_occupancy",
]


# --------------------------------------------------------------------------- inputs
def decode_bf16(bits: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> float64, exactly."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    f32 = (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return f32.astype(np.float64)


# ------------------------------------------------------------------------ rotation
def rotate(x_bits: np.ndarray, r_inter_bits, r_intra_bits) -> np.ndarray:
    """Algorithm 3 steps 1-3.  x_bits [M,d], r_inter_bits [d,d] or None (identity),
    r_intra_bits [d/32,32,32] or None (identity); all bfloat16 bit patterns.
    Returns Z [M,d] float64 with  y[m,j] = sum_i x[m,i] R_inter[i,j]  and
    z[m,32b+j] = sum_i y[m,32b+i] R_intra[b][i,j]."""
    x = decode_bf16(x_bits)
    m, d = x.shape
    assert d % K_BLOCK == 0
    if r_inter_bits is None:
        y = x
    else:
        r = decode_bf16(r_inter_bits)
        assert r.shape == (d, d)
        y = x @ r
    if r_intra_bits is None:
        return y.copy()
    ri = decode_bf16(r_intra_bits)
    nb = d // K_BLOCK
    assert ri.shape == (nb, K_BLOCK, K_BLOCK)
    z = np.empty_like(y)
    for b in range(nb):
        z[:, b * K_BLOCK:(b + 1) * K_BLOCK] = y[:, b * K_BLOCK:(b + 1) * K_BLOCK] @ ri[b]
    return z


def rotate_structured(x_bits: np.ndarray, r_b_bits, r_intra_bits) -> np.ndarray:
    """Algorithm 3 steps 1-3 in the paper's own structure: one B x B inter-block matrix acting
    across the blocks of a token (the same for every position inside a block) and one K x K
    intra-block matrix shared by all blocks (Section 5; App. A.7 counts B^2 + K^2 parameters and
    O(B^2 K) + O(B K^2) work per token).  Per token: reshape x to X [B, K] (step 1),
    Y = R_B X (step 2), Z = Y R_intra (step 3); returned flattened, Z [M, d] float64.
    r_b_bits [B, B] and r_intra_bits [K, K] are bfloat16 bit patterns; None = identity."""
    x = decode_bf16(x_bits)
    m, d = x.shape
    assert d % K_BLOCK == 0
    nb = d // K_BLOCK
    z = np.empty((m, d), dtype=np.float64)
    rb = None if r_b_bits is None else decode_bf16(r_b_bits)
    ri = None if r_intra_bits is None else decode_bf16(r_intra_bits)
    assert rb is None or rb.shape == (nb, nb)
    assert ri is None or ri.shape == (K_BLOCK, K_BLOCK)
    for t in range(m):
        xt = x[t].reshape(nb, K_BLOCK)                  # step 1: B blocks (rows) of K elements
        yt = xt if rb is None else rb @ xt               # step 2: Y = R_B X
        zt = yt if ri is None else yt @ ri               # step 3: Z = Y R_intra
        z[t] = zt.reshape(d)
    return z


def round_to_f32(z: np.ndarray) -> np.ndarray:
    """One rounding (nearest even) of the fp64 rotation result to float32."""
    return np.asarray(z, dtype=np.float64).astype(np.float32)


# ---------------------------------------------------------------------- quantizer
def shared_exponent(amax: np.ndarray) -> np.ndarray:
    """e with s_b = 2^e for block maxima `amax` (>= 0, finite):
    e = clamp(floor(log2 amax) - 2, -127, 127);  amax == 0 -> -127."""
    amax = np.asarray(amax, dtype=np.float64)
    _, ex = np.frexp(amax)            # amax = f * 2^ex with f in [0.5, 1)
    floor_log2 = ex.astype(np.int64) - 1
    e = np.clip(floor_log2 - E2M1_EMAX, -127, 127)
    return np.where(amax == 0.0, -127, e).astype(np.int64)


def _nearest_codeword(mag: np.ndarray) -> np.ndarray:
    """Index of the codebook entry nearest to each magnitude; a tie goes to the
    even index (mantissa bit 0).  Magnitudes above 6 are nearest to 6 anyway."""
    dist = np.abs(mag[..., None] - CODEBOOK)                  # [..., 8]
    best = dist.min(axis=-1, keepdims=True)
    is_best = dist == best
    idx = np.arange(8)
    # among the (one or two) nearest, prefer the even index
    even_hit = is_best & (idx % 2 == 0)
    any_even = even_hit.any(axis=-1)
    first_even = np.argmax(even_hit, axis=-1)
    first_any = np.argmax(is_best, axis=-1)
    return np.where(any_even, first_even, first_any).astype(np.uint8)


def quantize_mxfp4(z32: np.ndarray, rows_per_chunk: int = 256):
    """Eq. 1 / Algorithm 3 step 4 on float32 input z32 [M,d].
    Returns (codes [M,d] uint8, each 0..15 = sign<<3 | magnitude index;
             scale_bytes [M,d/32] uint8 = e + 127)."""
    z32 = np.asarray(z32)
    assert z32.dtype == np.float32 and z32.ndim == 2 and z32.shape[1] % K_BLOCK == 0
    m, d = z32.shape
    nb = d // K_BLOCK
    codes = np.empty((m, d), dtype=np.uint8)
    sbytes = np.empty((m, nb), dtype=np.uint8)
    for r0 in range(0, m, rows_per_chunk):
        blk = z32[r0:r0 + rows_per_chunk].astype(np.float64).reshape(-1, nb, K_BLOCK)
        amax = np.abs(blk).max(axis=-1)
        e = shared_exponent(amax)
        a = np.ldexp(blk, (-e)[..., None])                     # z / s_b, exact
        mag = _nearest_codeword(np.abs(a))
        sign = np.signbit(blk).astype(np.uint8)
        codes[r0:r0 + rows_per_chunk] = ((sign << 3) | mag).reshape(-1, d)
        sbytes[r0:r0 + rows_per_chunk] = (e + 127).astype(np.uint8)
    return codes, sbytes


def pack_codes(codes: np.ndarray) -> np.ndarray:
    """[M,d] 4-bit codes -> [M,d/2] bytes, even element in the low nibble."""
    codes = np.asarray(codes, dtype=np.uint8)
    return (codes[:, 0::2] | (codes[:, 1::2] << 4)).astype(np.uint8)


def unpack_codes(packed: np.ndarray) -> np.ndarray:
    packed = np.asarray(packed, dtype=np.uint8)
    out = np.empty((packed.shape[0], packed.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = packed & 0xF
    out[:, 1::2] = packed >> 4
    return out


def dequantize(codes: np.ndarray, scale_bytes: np.ndarray) -> np.ndarray:
    """z^ = s_b * codeword, exact in float64.  codes [M,d] (0..15), scale_bytes [M,d/32]."""
    codes = np.asarray(codes, dtype=np.uint8)
    m, d = codes.shape
    val = CODEBOOK[codes & 7] * np.where(codes & 8, -1.0, 1.0)
    e = scale_bytes.astype(np.int64) - 127
    return np.ldexp(val.reshape(m, d // K_BLOCK, K_BLOCK), e[..., None]).reshape(m, d)


# ---------------------------------------------------------------------------- GEMM
def gemm_dequant(a_codes, a_scales, w_codes, w_scales) -> np.ndarray:
    """Step 5, option B: out[m,n] = sum_k a^[m,k] w^[n,k] in float64.
    a_codes [M,K], a_scales [M,K/32]; w_codes [N,K], w_scales [N,K/32]."""
    a = dequantize(a_codes, a_scales)
    w = dequantize(w_codes, w_scales)
    return a @ w.T


def round_to_bf16(y: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of float64 values to the bfloat16 grid (8 significant
    bits), returned as float64.  Normal range only (no overflow/subnormal handling)."""
    y = np.asarray(y, dtype=np.float64)
    f, ex = np.frexp(y)                       # |f| in [0.5,1): 8 significant bits = f*256 integer
    return np.ldexp(np.rint(f * 256.0) / 256.0, ex)


# ------------------------------------------------------------- offline weight side
def merged_rotation(r_inter_bits, r_intra_bits) -> np.ndarray:
    """R~ = R_inter . blockdiag(R_intra[b]) in float64 from the bfloat16 values."""
    r = decode_bf16(r_inter_bits)
    ri = decode_bf16(r_intra_bits)
    out = np.empty_like(r)
    for b in range(ri.shape[0]):
        out[:, b * K_BLOCK:(b + 1) * K_BLOCK] = r[:, b * K_BLOCK:(b + 1) * K_BLOCK] @ ri[b]
    return out


def prepare_weights(r_inter_bits, r_intra_bits, w: np.ndarray):
    """Offline weight fusion: W' = R~^T W for W [d,N] (out = x W), stored as [N,d]
    so that K = d is contiguous, rounded once to float32 and MXFP4-quantized along K.
    Returns (codes [N,d], scale_bytes [N,d/32])."""
    rt = merged_rotation(r_inter_bits, r_intra_bits)
    wp = (rt.T @ np.asarray(w, dtype=np.float64)).T
    return quantize_mxfp4(round_to_f32(np.ascontiguousarray(wp)))


# ------------------------------------------------------- scale-factor byte layout
def scale_layout_bytes(rows: int, k: int) -> int:
    kb = k // K_BLOCK
    return ((rows + 127) // 128) * ((kb + 3) // 4) * 512


def scale_layout_offset(r, c, k: int):
    """Byte offset of the scale of (row r, K-block c) in the tiled layout the FP4
    tensor-core instruction consumes: 512-byte tiles of 128 rows x 4 K-blocks, tiles
    ordered row-tile major; inside a tile byte = (r%32)*16 + ((r%128)//32)*4 + c%4."""
    kb4 = (k // K_BLOCK + 3) // 4
    r = np.asarray(r)
    c = np.asarray(c)
    return ((r // 128) * kb4 + c // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + (c % 4)


def swizzle_scales(scale_bytes: np.ndarray, k: int, fill: int = 0x7F) -> np.ndarray:
    rows, kb = scale_bytes.shape
    out = np.full(scale_layout_bytes(rows, k), fill, dtype=np.uint8)
    rr, cc = np.meshgrid(np.arange(rows), np.arange(kb), indexing="ij")
    out[scale_layout_offset(rr, cc, k)] = scale_bytes
    return out


def unswizzle_scales(buf: np.ndarray, rows: int, k: int) -> np.ndarray:
    kb = k // K_BLOCK
    rr, cc = np.meshgrid(np.arange(rows), np.arange(kb), indexing="ij")
    return np.asarray(buf, dtype=np.uint8)[scale_layout_offset(rr, cc, k)]


# ------------------------------------------------------------------ whole path
def rotated_linear(x_bits, r_inter_bits, r_intra_bits, w_codes, w_scales):
    """Algorithm 3 end to end.  Returns (out float64 [M,N], codes, scale_bytes)."""
    z32 = round_to_f32(rotate(x_bits, r_inter_bits, r_intra_bits))
    codes, sb = quantize_mxfp4(z32)
    return gemm_dequant(codes, sb, w_codes, w_scales), codes, sb


def codeword_occupancy(codes: np.ndarray) -> np.ndarray:
    """Empirical occupancy p^_j of the 8 magnitude codewords (diagnostic only)."""
    return np.bincount((np.asarray(codes) & 7).ravel(), minlength=8) / codes.size
