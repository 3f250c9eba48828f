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

// R~[i, 32b+j] = sum_t R_inter[i, 32b+t] * R_intra[b][t][j], fp32 (offline weight-side helper).
__global__ void merge_rotations_kernel(const __nv_bfloat16* __restrict__ R_inter,
                                       const __nv_bfloat16* __restrict__ R_intra, int64_t d,
                                       float* __restrict__ out) {
  const int64_t total = d * d;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (int64_t)gridDim.x * blockDim.x) {
    const int64_t i = t / d, col = t % d, b = col / 32, j = col % 32;
    float acc = 0.f;
    for (int tt = 0; tt < 32; ++tt)
      acc = fmaf(__bfloat162float(R_inter[i * d + b * 32 + tt]),
                 __bfloat162float(R_intra[b * 1024 + tt * 32 + j]), acc);
    out[t] = acc;
  }
}

}  // namespace torq
