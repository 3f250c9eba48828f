// MXFP4 block quantization (Eq. 1 of the paper with the OCP MX scale rule): device helpers shared
// by the rotation epilogue and the stand-alone kernels, plus the stand-alone kernels themselves
// (quantize-only, intra-rotation + quantize, scale re-tiling, rotation merge).
#pragma once
#include <cuda_bf16.h>
#include "sm100_ptx.cuh"

namespace torq {

// E8M0 byte and the exact reciprocal scale for a block maximum amax >= 0 (finite).
// With ef the float32 exponent field of amax: e = max(ef - 129, -127), byte = e + 127 =
// max(ef - 2, 0); subnormal and zero maxima (ef == 0) clamp to byte 0.  2^-e has exponent
// field 254 - byte, always a normal number.
__device__ __forceinline__ void block_scale(float amax, uint32_t& sbyte, float& inv_scale) {
  uint32_t ef = __float_as_uint(amax) >> 23;
  sbyte = ef > 2u ? ef - 2u : 0u;
  inv_scale = __uint_as_float((254u - sbyte) << 23);
}

// Eight scaled values -> eight e2m1 codes in one 32-bit word, element 0 in the lowest nibble.
// cvt.rn.satfinite rounds to nearest even on the e2m1 grid and saturates to +-6; the first
// source operand lands in the high nibble of the byte.
__device__ __forceinline__ uint32_t pack8_e2m1(float a0, float a1, float a2, float a3, float a4,
                                               float a5, float a6, float a7) {
  uint32_t out;
  asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
      "mov.b32 %0, {b0, b1, b2, b3};\n\t}"
      : "=r"(out)
      : "f"(a0), "f"(a1), "f"(a2), "f"(a3), "f"(a4), "f"(a5), "f"(a6), "f"(a7));
  return out;
}

// One whole block held by one thread: z[32] -> 16 code bytes + scale byte.
__device__ __forceinline__ void quantize_block32(const float (&z)[32], uint4& codes,
                                                 uint32_t& sbyte) {
  float amax = 0.f;
#pragma unroll
  for (int j = 0; j < 32; ++j) amax = fmaxf(amax, fabsf(z[j]));
  float inv;
  block_scale(amax, sbyte, inv);
  codes.x = pack8_e2m1(z[0] * inv, z[1] * inv, z[2] * inv, z[3] * inv, z[4] * inv, z[5] * inv,
                       z[6] * inv, z[7] * inv);
  codes.y = pack8_e2m1(z[8] * inv, z[9] * inv, z[10] * inv, z[11] * inv, z[12] * inv,
                       z[13] * inv, z[14] * inv, z[15] * inv);
  codes.z = pack8_e2m1(z[16] * inv, z[17] * inv, z[18] * inv, z[19] * inv, z[20] * inv,
                       z[21] * inv, z[22] * inv, z[23] * inv);
  codes.w = pack8_e2m1(z[24] * inv, z[25] * inv, z[26] * inv, z[27] * inv, z[28] * inv,
                       z[29] * inv, z[30] * inv, z[31] * inv);
}

// Intra-block rotation of one block held by one thread (Algorithm 3 step 3):
// z[j] = sum_i y[i] * R[i][j], fp32, i in index order, with R (fp32, row-major 32 x 32) read from
// shared memory at `r_saddr` -- every lane reads the same address, so each load is one broadcast.
// The FMAs are issued as packed pairs (fma.rn.f32x2: two independent IEEE fused multiply-adds per
// instruction, same results as 32 scalar chains).
__device__ __forceinline__ void intra_rotate32(const uint32_t (&y)[32], uint32_t r_saddr, float (&z)[32]) {
  uint64_t zp[16];
#pragma unroll
  for (int k = 0; k < 16; ++k) zp[k] = 0ull;
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    uint64_t yy;
    asm("mov.b64 %0, {%1, %1};" : "=l"(yy) : "r"(y[i]));
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      uint64_t r0, r1;
      asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(r0), "=l"(r1) : "r"(r_saddr + (uint32_t)((i * 8 + g) * 16)));
      asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(zp[2 * g]) : "l"(yy), "l"(r0));
      asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(zp[2 * g + 1]) : "l"(yy), "l"(r1));
    }
  }
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    uint32_t lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(zp[k]));
    z[2 * k] = __uint_as_float(lo);
    z[2 * k + 1] = __uint_as_float(hi);
  }
}

// ---- intra-block rotation on the warp-level tensor-core path -------------------------------------
// y (fp32) is split into three bfloat16 terms, y = hi + mid + lo up to 2^-24 relative; R_intra is
// bfloat16 already, so every product is exact in fp32 and the fp32-accumulating warp MMA
// (m16n8k16) reproduces the fp32 rotation to accumulation-order rounding.
// Two fp32 values -> packed pairs (element 0 in the low half) of the three terms.
__device__ __forceinline__ void split3_bf16x2(uint32_t x0, uint32_t x1, uint32_t& hi, uint32_t& mid,
                                              uint32_t& lo) {
  float f0 = __uint_as_float(x0), f1 = __uint_as_float(x1);
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(hi) : "f"(f1), "f"(f0));
  f0 -= __uint_as_float(hi << 16);                       // exact: hi is within half a bf16 ulp of f
  f1 -= __uint_as_float(hi & 0xFFFF0000u);
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(mid) : "f"(f1), "f"(f0));
  f0 -= __uint_as_float(mid << 16);
  f1 -= __uint_as_float(mid & 0xFFFF0000u);
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(lo) : "f"(f1), "f"(f0));
}
// The same split by truncation, with integer and add instructions only (no conversion unit): hi =
// the top 16 bits of y, mid = the top 16 bits of y - hi, lo = what is left, which has at most eight
// significant bits: y = hi + mid + lo exactly (subnormal leftovers aside).
__device__ __forceinline__ void split3_trunc_bf16x2(uint32_t x0, uint32_t x1, uint32_t& hi, uint32_t& mid,
                                                    uint32_t& lo) {
  const uint32_t h0 = x0 & 0xFFFF0000u, h1 = x1 & 0xFFFF0000u;
  const uint32_t r0 = __float_as_uint(__uint_as_float(x0) - __uint_as_float(h0));
  const uint32_t r1 = __float_as_uint(__uint_as_float(x1) - __uint_as_float(h1));
  const uint32_t m0 = r0 & 0xFFFF0000u, m1 = r1 & 0xFFFF0000u;
  const uint32_t l0 = __float_as_uint(__uint_as_float(r0) - __uint_as_float(m0));
  const uint32_t l1 = __float_as_uint(__uint_as_float(r1) - __uint_as_float(m1));
  hi = __byte_perm(x0, x1, 0x7632);                      // high halves: element 0 in the low half
  mid = __byte_perm(r0, r1, 0x7632);
  lo = __byte_perm(l0, l1, 0x7632);
}
// D[16x8] += A[16x16] . B[16x8], bf16 inputs, fp32 accumulate (fragment layouts of the PTX ISA).
__device__ __forceinline__ void mma_16816_bf16(float (&c)[4], const uint32_t* a, const uint32_t* b) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
// Four 8x8 bf16 matrices from shared memory, transposed on the way (B fragments of a row-major
// [k][n] matrix).  Lane l supplies the address of row l % 8 of matrix l / 8.
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t saddr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                                  uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(saddr));
}
// One row of a 32-block spread over the four lanes that share it in the accumulator layout: lane
// p = lane % 4 holds v[2 nt + e] = element 8 nt + 2 p + e.  Returns the scale byte and, in `word`,
// the four code bytes 4p .. 4p+3 of the block (so the four lanes together store 16 contiguous bytes).
__device__ __forceinline__ void quantize_row_fragment(const float (&v)[8], int p, uint32_t& word,
                                                      uint32_t& sbyte) {
  float amax = 0.f;
#pragma unroll
  for (int j = 0; j < 8; ++j) amax = fmaxf(amax, fabsf(v[j]));
  amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
  amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
  float inv;
  block_scale(amax, sbyte, inv);
  // byte nt of w = codes of elements 8 nt + 2 p, 8 nt + 2 p + 1 = byte 4 nt + p of the block
  const uint32_t w = pack8_e2m1(v[0] * inv, v[1] * inv, v[2] * inv, v[3] * inv, v[4] * inv, v[5] * inv,
                                v[6] * inv, v[7] * inv);
  // 4 x 4 byte transpose across the four lanes
  const uint32_t w1 = __shfl_xor_sync(0xFFFFFFFFu, w, 1);
  const uint32_t x = (p & 1) ? __byte_perm(w, w1, 0x3715) : __byte_perm(w, w1, 0x6240);
  const uint32_t x2 = __shfl_xor_sync(0xFFFFFFFFu, x, 2);
  word = (p & 2) ? __byte_perm(x, x2, 0x3276) : __byte_perm(x, x2, 0x5410);
}

__host__ __device__ __forceinline__ size_t scale_offset(int64_t row, int64_t kblock, int64_t kb4) {
  return (size_t)(((row >> 7) * kb4 + (kblock >> 2)) * 512 + (row & 31) * 16 +
                  ((row & 127) >> 5) * 4 + (kblock & 3));
}

__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
  float4 a = __ldg(reinterpret_cast<const float4*>(p));
  float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
  uint4 a = __ldg(reinterpret_cast<const uint4*>(p));
  uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}

// Quantize-only.  One warp handles 256 consecutive elements of a row (8 blocks): lane l owns
// elements 8l..8l+7, four lanes share a block.  Rows M..Mpad-1 and K-blocks beyond d only get
// their padding scale byte (0) written.
template <typename T>
__global__ void __launch_bounds__(256) quantize_kernel(const T* __restrict__ Z, int64_t M,
                                                       int64_t d, uint8_t* __restrict__ codes,
                                                       uint8_t* __restrict__ scales) {
  const int lane = threadIdx.x & 31;
  const int64_t kb4 = (d / 32 + 3) / 4;
  const int64_t dpad = kb4 * 128;
  const int64_t nseg = (dpad + 255) / 256;
  const int64_t mpad = (M + 127) / 128 * 128;
  const int64_t total = mpad * nseg;
  const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
  for (int64_t item = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); item < total;
       item += nwarps) {
    const int64_t row = item / nseg;
    const int64_t col = (item % nseg) * 256 + lane * 8;
    const bool has_data = row < M && col < d;
    float v[8];
    if (has_data) load8(Z + row * d + col, v);
    else {
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = 0.f;
    }
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(v[i]));
    amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
    amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
    uint32_t sbyte;
    float inv;
    block_scale(amax, sbyte, inv);
    if (has_data) {
      uint32_t w = pack8_e2m1(v[0] * inv, v[1] * inv, v[2] * inv, v[3] * inv, v[4] * inv,
                              v[5] * inv, v[6] * inv, v[7] * inv);
      *reinterpret_cast<uint32_t*>(codes + row * (d / 2) + col / 2) = w;
    }
    if ((lane & 3) == 0 && col < dpad) scales[scale_offset(row, col / 32, kb4)] = (uint8_t)sbyte;
  }
}

// Intra-block rotation (Algorithm 3 step 3) followed by quantization, without the inter-block
// step: one thread per (row, block).  Used when the caller passes no R_inter.
__global__ void __launch_bounds__(128) intra_quantize_kernel(
    const __nv_bfloat16* __restrict__ X, const __nv_bfloat16* __restrict__ R_intra, int64_t M,
    int64_t d, uint8_t* __restrict__ codes, uint8_t* __restrict__ scales) {
  const int64_t nb = d / 32;
  const int64_t kb4 = (nb + 3) / 4;
  const int64_t mpad = (M + 127) / 128 * 128;
  const int64_t total = mpad * kb4 * 4;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = t / (kb4 * 4), b = t % (kb4 * 4);
    if (row >= M || b >= nb) {
      scales[scale_offset(row, b, kb4)] = 0;
      continue;
    }
    float y[32], z[32];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float v[8];
      load8(X + row * d + b * 32 + q * 8, v);
#pragma unroll
      for (int i = 0; i < 8; ++i) y[q * 8 + i] = v[i];
    }
#pragma unroll
    for (int j = 0; j < 32; ++j) z[j] = 0.f;
    const __nv_bfloat16* r = R_intra + b * 1024;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float v[8];
        load8(r + i * 32 + q * 8, v);
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) z[q * 8 + jj] = fmaf(y[i], v[jj], z[q * 8 + jj]);
      }
    }
    uint4 c;
    uint32_t sbyte;
    quantize_block32(z, c, sbyte);
    *reinterpret_cast<uint4*>(codes + row * (d / 2) + b * 16) = c;
    scales[scale_offset(row, b, kb4)] = (uint8_t)sbyte;
  }
}

// Plain [rows, kb] scale bytes -> tiled layout; padding := 0.
__global__ void swizzle_scales_kernel(const uint8_t* __restrict__ lin, int64_t rows, int64_t kb,
                                      uint8_t* __restrict__ out) {
  const int64_t kb4 = (kb + 3) / 4;
  const int64_t mpad = (rows + 127) / 128 * 128;
  const int64_t total = mpad * kb4 * 4;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = t / (kb4 * 4), c = t % (kb4 * 4);
    out[scale_offset(row, c, kb4)] = (row < rows && c < kb) ? lin[row * kb + c] : (uint8_t)0;
  }
}

// R~[i, 32b+j] = sum_t R_inter[i, 32b+t] * R_intra[b][t][j], fp32 FMAs in index order; stored as
// float32, or rounded once (nearest even) to bfloat16.
template <typename OutT>
__global__ void merge_rotations_kernel(const __nv_bfloat16* __restrict__ R_inter,
                                       const __nv_bfloat16* __restrict__ R_intra, int64_t d,
                                       OutT* __restrict__ out) {
  const int64_t total = d * d;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = t / d, col = t % d, b = col / 32, j = col % 32;
    float acc = 0.f;
    for (int tt = 0; tt < 32; ++tt)
      acc = fmaf(__bfloat162float(R_inter[i * d + b * 32 + tt]),
                 __bfloat162float(R_intra[b * 1024 + tt * 32 + j]), acc);
    if constexpr (sizeof(OutT) == 2) out[t] = __float2bfloat16_rn(acc);
    else out[t] = acc;
  }
}

}  // namespace torq
