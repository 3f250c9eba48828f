// MXINT4 block quantization (format study of Section 6: the rotations with an integer 4-bit block
// format): 32-element blocks, one E8M0 scale byte per block by the same rule as MXFP4, elements
// q = clamp(rint(z / 2^e), -7, 7).
//
// The tensor cores of this GPU have no 4-bit integer path, so the operand form of the layer is
// the FP8 E4M3 byte whose value is q (every integer of [-8, 8] is an E4M3 number; a zero may
// carry the sign of the value that rounded to it), consumed by kind::mxf8f6f4 with the same scale
// bytes.  The stored form, two's-complement nibbles with the even element in the low nibble,
// comes from the stand-alone quantizer and goes through `mxint4_expand_kernel` to become operands.
#pragma once
#include <cuda_bf16.h>
#include "quantize.cuh"

namespace torq {

// rint and clamp to [-7, 7]: the integer code as a float.
__device__ __forceinline__ float int4_round(float a) { return fminf(fmaxf(rintf(a), -7.0f), 7.0f); }

// Four integer-valued floats -> four E4M3 bytes, element 0 in the lowest byte (the conversion is
// exact on integers of [-8, 8]; its first source operand lands in the high byte).
__device__ __forceinline__ uint32_t pack4_e4m3(float r0, float r1, float r2, float r3) {
  uint32_t out;
  asm("{\n\t.reg .b16 lo, hi;\n\t"
      "cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1;\n\t"
      "cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3;\n\t"
      "mov.b32 %0, {lo, hi};\n\t}"
      : "=r"(out) : "f"(r0), "f"(r1), "f"(r2), "f"(r3));
  return out;
}

// Eight integer-valued floats -> eight two's-complement nibbles, element 0 in the lowest nibble.
__device__ __forceinline__ uint32_t pack8_int4(const float (&r)[8]) {
  uint32_t out = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) out |= ((uint32_t)__float2int_rn(r[j]) & 0xFu) << (4 * j);
  return out;
}

// One whole block held by one thread: z[32] -> 32 operand bytes (eight words) + scale byte.
__device__ __forceinline__ void mxint4_quantize_block32(const float (&z)[32], uint4& lo, uint4& hi,
                                                        uint32_t& sbyte) {
  float amax = 0.f;
#pragma unroll
  for (int j = 0; j < 32; ++j) amax = fmaxf(amax, fabsf(z[j]));
  float inv;
  block_scale(amax, sbyte, inv);
  uint32_t w[8];
#pragma unroll
  for (int g = 0; g < 8; ++g)
    w[g] = pack4_e4m3(int4_round(z[4 * g] * inv), int4_round(z[4 * g + 1] * inv), int4_round(z[4 * g + 2] * inv),
                      int4_round(z[4 * g + 3] * inv));
  lo = make_uint4(w[0], w[1], w[2], w[3]);
  hi = make_uint4(w[4], w[5], w[6], w[7]);
}

// One row of a 32-block spread over the four lanes that share it in the accumulator layout: lane
// p = lane % 4 holds v[2 nt + e] = element 8 nt + 2 p + e.  Returns the scale byte and, per nt, the
// two operand bytes of elements 8 nt + 2 p and 8 nt + 2 p + 1 in the low half of pair[nt].
__device__ __forceinline__ void mxint4_quantize_row_fragment(const float (&v)[8], uint32_t (&pair)[4],
                                                             uint32_t& sbyte) {
  float amax = 0.f;
#pragma unroll
  for (int j = 0; j < 8; ++j) amax = fmaxf(amax, fabsf(v[j]));
  amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
  amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
  float inv;
  block_scale(amax, sbyte, inv);
  const uint32_t w0 = pack4_e4m3(int4_round(v[0] * inv), int4_round(v[1] * inv), int4_round(v[2] * inv),
                                 int4_round(v[3] * inv));
  const uint32_t w1 = pack4_e4m3(int4_round(v[4] * inv), int4_round(v[5] * inv), int4_round(v[6] * inv),
                                 int4_round(v[7] * inv));
  pair[0] = w0 & 0xFFFFu; pair[1] = w0 >> 16; pair[2] = w1 & 0xFFFFu; pair[3] = w1 >> 16;
}

// Quantize-only.  One warp handles 256 consecutive elements of a row (8 blocks): lane l owns
// elements 8l..8l+7, four lanes share a block.  PACKED: codes [M, d/2] nibbles; otherwise codes
// [M, d] operand bytes.  Rows M..Mpad-1 and K-blocks beyond d only get their padding scale byte.
template <typename T, bool PACKED>
__global__ void __launch_bounds__(256) mxint4_quantize_kernel(const T* __restrict__ Z, int64_t M, int64_t d,
                                                              uint8_t* __restrict__ codes,
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
      float r[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) r[i] = int4_round(v[i] * inv);
      if constexpr (PACKED) {
        *reinterpret_cast<uint32_t*>(codes + row * (d / 2) + col / 2) = pack8_int4(r);
      } else {
        *reinterpret_cast<uint2*>(codes + row * d + col) =
            make_uint2(pack4_e4m3(r[0], r[1], r[2], r[3]), pack4_e4m3(r[4], r[5], r[6], r[7]));
      }
    }
    if ((lane & 3) == 0 && col < dpad) scales[scale_offset(row, col / 32, kb4)] = (uint8_t)sbyte;
  }
}

// Stored form -> operand form: `words` 32-bit words of eight nibbles each -> eight E4M3 bytes each.
__global__ void __launch_bounds__(256) mxint4_expand_kernel(const uint32_t* __restrict__ packed, int64_t words,
                                                            uint2* __restrict__ out) {
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < words;
       t += (int64_t)gridDim.x * blockDim.x) {
    const uint32_t w = __ldg(packed + t);
    float r[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) r[j] = (float)(((int32_t)(w << (28 - 4 * j))) >> 28);   // sign-extended nibble
    out[t] = make_uint2(pack4_e4m3(r[0], r[1], r[2], r[3]), pack4_e4m3(r[4], r[5], r[6], r[7]));
  }
}

}  // namespace torq
