// NVFP4 block quantization: e2m1 elements, blocks of 16 along K, one FP8 E4M3 scale per block and
// one float32 scale per tensor (the format study of Section 6 of the paper; the format itself is
// public).  The arithmetic is fixed operation by operation, each a single IEEE float32 operation
// rounded to nearest even, so that a host restatement in float32 reproduces every code:
//     c    = 1 / (6 * tensor_scale)
//     byte = E4M3(amax_block * c)          nearest even, saturating at 448
//     dec  = e4m3(byte) * tensor_scale
//     r    = 1 / dec                       (0 if byte == 0: the block encodes as zeros)
//     code = e2m1(z * r)                   nearest even, saturating at 6, sign of z kept
#pragma once
#include <cuda_fp16.h>
#include "quantize.cuh"

namespace torq {

// Per-tensor constants of the NVFP4 quantizer.
struct NvScale {
  float ts;   // tensor scale
  float c;    // 1 / (6 ts)
};
__device__ __forceinline__ NvScale nv_scale(float tensor_scale) {
  NvScale s;
  s.ts = tensor_scale;
  s.c = __fdiv_rn(1.0f, __fmul_rn(6.0f, tensor_scale));
  return s;
}

// v >= 0 -> E4M3 byte (round to nearest even, saturate to 448).
__device__ __forceinline__ uint32_t e4m3_byte(float v) {
  uint32_t out;
  asm("{\n\t.reg .b16 t;\n\tcvt.rn.satfinite.e4m3x2.f32 t, %1, %2;\n\tcvt.u32.u16 %0, t;\n\t}"
      : "=r"(out) : "f"(0.0f), "f"(v));                  // second source -> low byte
  return out & 0xFFu;
}
// E4M3 byte -> float, exact.
__device__ __forceinline__ float e4m3_to_float(uint32_t byte) {
  uint32_t h2;
  asm("{\n\t.reg .b16 t;\n\tcvt.u16.u32 t, %1;\n\tcvt.rn.f16x2.e4m3x2 %0, t;\n\t}" : "=r"(h2) : "r"(byte & 0xFFu));
  return __half2float(__ushort_as_half((unsigned short)(h2 & 0xFFFFu)));
}

// Block maximum -> scale byte and the multiplier applied to the block's elements.
__device__ __forceinline__ void nv_block_scale(float amax, const NvScale& s, uint32_t& sbyte, float& r) {
  sbyte = e4m3_byte(__fmul_rn(amax, s.c));
  const float dec = __fmul_rn(e4m3_to_float(sbyte), s.ts);
  r = sbyte ? __fdiv_rn(1.0f, dec) : 0.0f;
}

// Thirty-two consecutive values held by one thread = two blocks: 16 code bytes + two scale bytes
// (block 0 in the low byte of `sbytes`).
__device__ __forceinline__ void nv_quantize_2x16(const float (&z)[32], const NvScale& s, uint4& codes,
                                                 uint32_t& sbytes) {
  float a0 = 0.f, a1 = 0.f;
#pragma unroll
  for (int j = 0; j < 16; ++j) { a0 = fmaxf(a0, fabsf(z[j])); a1 = fmaxf(a1, fabsf(z[16 + j])); }
  uint32_t b0, b1;
  float r0, r1;
  nv_block_scale(a0, s, b0, r0);
  nv_block_scale(a1, s, b1, r1);
  auto m = [](float x, float r) { return __fmul_rn(x, r); };
  codes.x = pack8_e2m1(m(z[0], r0), m(z[1], r0), m(z[2], r0), m(z[3], r0), m(z[4], r0), m(z[5], r0), m(z[6], r0),
                       m(z[7], r0));
  codes.y = pack8_e2m1(m(z[8], r0), m(z[9], r0), m(z[10], r0), m(z[11], r0), m(z[12], r0), m(z[13], r0),
                       m(z[14], r0), m(z[15], r0));
  codes.z = pack8_e2m1(m(z[16], r1), m(z[17], r1), m(z[18], r1), m(z[19], r1), m(z[20], r1), m(z[21], r1),
                       m(z[22], r1), m(z[23], r1));
  codes.w = pack8_e2m1(m(z[24], r1), m(z[25], r1), m(z[26], r1), m(z[27], r1), m(z[28], r1), m(z[29], r1),
                       m(z[30], r1), m(z[31], r1));
  sbytes = b0 | (b1 << 8);
}

// One row of 32 columns spread over the four lanes that share it in the warp-MMA accumulator layout
// (lane p = lane % 4 holds v[2 nt + e] = element 8 nt + 2 p + e): the first block is nt 0..1, the
// second nt 2..3.  Returns both scale bytes (first block in the low byte) and, in `word`, the four
// code bytes 4p .. 4p+3 of the 32 columns.
__device__ __forceinline__ void nv_quantize_row_fragment(const float (&v)[8], int p, const NvScale& s,
                                                         uint32_t& word, uint32_t& sbytes) {
  float a0 = fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3])));
  float a1 = fmaxf(fmaxf(fabsf(v[4]), fabsf(v[5])), fmaxf(fabsf(v[6]), fabsf(v[7])));
  a0 = fmaxf(a0, __shfl_xor_sync(0xFFFFFFFFu, a0, 1));
  a1 = fmaxf(a1, __shfl_xor_sync(0xFFFFFFFFu, a1, 1));
  a0 = fmaxf(a0, __shfl_xor_sync(0xFFFFFFFFu, a0, 2));
  a1 = fmaxf(a1, __shfl_xor_sync(0xFFFFFFFFu, a1, 2));
  uint32_t b0, b1;
  float r0, r1;
  nv_block_scale(a0, s, b0, r0);
  nv_block_scale(a1, s, b1, r1);
  sbytes = b0 | (b1 << 8);
  const uint32_t w = pack8_e2m1(__fmul_rn(v[0], r0), __fmul_rn(v[1], r0), __fmul_rn(v[2], r0), __fmul_rn(v[3], r0),
                                __fmul_rn(v[4], r1), __fmul_rn(v[5], r1), __fmul_rn(v[6], r1), __fmul_rn(v[7], r1));
  const uint32_t w1 = __shfl_xor_sync(0xFFFFFFFFu, w, 1);                   // 4 x 4 byte transpose across the lanes
  const uint32_t x = (p & 1) ? __byte_perm(w, w1, 0x3715) : __byte_perm(w, w1, 0x6240);
  const uint32_t x2 = __shfl_xor_sync(0xFFFFFFFFu, x, 2);
  word = (p & 2) ? __byte_perm(x, x2, 0x3276) : __byte_perm(x, x2, 0x5410);
}

// Quantize-only.  One warp handles 256 consecutive elements of a row (16 blocks): lane l owns
// elements 8l..8l+7, two lanes share a block.  Rows M..Mpad-1 and blocks beyond d only get their
// padding scale byte (0, which decodes to 0.0) written.
template <typename T>
__global__ void __launch_bounds__(256) nv_quantize_kernel(const T* __restrict__ Z, int64_t M, int64_t d,
                                                          float tensor_scale, uint8_t* __restrict__ codes,
                                                          uint8_t* __restrict__ scales) {
  const int lane = threadIdx.x & 31;
  const NvScale s = nv_scale(tensor_scale);
  const int64_t kb4 = (d / 16 + 3) / 4;
  const int64_t dpad = kb4 * 64;
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
    uint32_t sbyte;
    float r;
    nv_block_scale(amax, s, sbyte, r);
    if (has_data) {
      uint32_t w = pack8_e2m1(__fmul_rn(v[0], r), __fmul_rn(v[1], r), __fmul_rn(v[2], r), __fmul_rn(v[3], r),
                              __fmul_rn(v[4], r), __fmul_rn(v[5], r), __fmul_rn(v[6], r), __fmul_rn(v[7], r));
      *reinterpret_cast<uint32_t*>(codes + row * (d / 2) + col / 2) = w;
    }
    if ((lane & 1) == 0 && col < dpad) scales[scale_offset(row, col / 16, kb4)] = (uint8_t)sbyte;
  }
}

// [d/16, 16, 16] intra-block rotations -> the same linear map written with 32-wide blocks
// [d/32, 32, 32]: blocks 2b and 2b+1 on the diagonal of block b, zeros elsewhere (what the rotation
// kernels, which work on 32 columns per thread, take).
__global__ void expand_intra16_kernel(const __nv_bfloat16* __restrict__ r16, int64_t nb32,
                                      __nv_bfloat16* __restrict__ r32) {
  const int64_t total = nb32 * 1024;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (int64_t)gridDim.x * blockDim.x) {
    const int64_t b = t >> 10;
    const int i = (int)(t & 1023) >> 5, j = (int)(t & 31);
    const bool on = (i >> 4) == (j >> 4);
    r32[t] = on ? r16[(2 * b + (i >> 4)) * 256 + (i & 15) * 16 + (j & 15)] : __float2bfloat16(0.0f);
  }
}

}  // namespace torq
