// Intra-block rotation + quantization of a 16-row x 32-column tile of rotated activations held in
// shared memory, by ONE warp on the warp-level tensor cores (Algorithm 3 steps 3-4 for one 32-block
// of 16 tokens): y is split into three bfloat16 terms (y = hi + mid + lo up to 2^-24 relative),
// R_intra is bfloat16 already, so every product is exact in fp32 and the fp32-accumulating
// mma.sync m16n8k16 reproduces the fp32 rotation up to the order of additions.  Then Eq. 1 (or the
// NVFP4 / MXINT4 quantizer) on the accumulator fragments: four lanes share a row.
#pragma once
#include <cuda_bf16.h>
#include "nvfp4_quantize.cuh"
#include "mxint4_quantize.cuh"
#include "quantize.cuh"
#include "sm100_ptx.cuh"

namespace torq {

// y_s: 16 rows of 33 floats (row stride 33).  r_saddr: shared-memory address of R_intra[blk] as 32 rows
// of 80 bytes (32 bf16 + padding: conflict-free ldmatrix); ignored when !has_intra.  Rows row0 ..
// row0 + 15 of the output; rows >= M get no codes and a zero scale byte.  blk: 32-block index along d.
// Scale bytes go to the single-byte positions of the tiled layout (16-blocks 2 blk, 2 blk + 1 for NVFP4).
// store == false: everything is computed and nothing is written (a dry pass over the same instructions).
template <int FMT>
__device__ __forceinline__ void intra_quantize_rows16(const float* y_s, uint32_t r_saddr, bool has_intra, int lane,
                                                      int row0, int M, int blk, int d, int nblocks,
                                                      float tensor_scale, uint8_t* __restrict__ codes,
                                                      uint8_t* __restrict__ scales, bool store = true) {
  const int p = lane & 3, r8 = lane >> 2;
  const int kb4 = FMT == FMT_NVFP4 ? (2 * nblocks + 3) / 4 : (nblocks + 3) / 4;
  float acc[4][4];
  if (has_intra) {
    uint32_t bfrag[2][4][2];                             // [k chunk][n tile][2]
    {
      // lane l: row l % 8 of matrix l / 8; matrices (k 0-7, n), (k 8-15, n), (k 0-7, n+8), (k 8-15, n+8)
      const uint32_t rb = r_saddr + (uint32_t)(((lane >> 3) & 1) * 8 + (lane & 7)) * 80 + (uint32_t)(lane >> 4) * 16;
#pragma unroll
      for (int kc = 0; kc < 2; ++kc)
#pragma unroll
        for (int np = 0; np < 2; ++np)
          ldmatrix_x4_trans(rb + kc * 16 * 80 + np * 32, bfrag[kc][2 * np][0], bfrag[kc][2 * np][1],
                            bfrag[kc][2 * np + 1][0], bfrag[kc][2 * np + 1][1]);
    }
    uint32_t ah[8], am[8], al[8];                        // A fragments: [k chunk * 4 + (n & 1) * 2 + row half]
#pragma unroll
    for (int n = 0; n < 4; ++n)
#pragma unroll
      for (int rh = 0; rh < 2; ++rh) {
        const float* yp = y_s + (r8 + 8 * rh) * 33 + 8 * n + 2 * p;
        const int ai = (n >> 1) * 4 + (n & 1) * 2 + rh;
        split3_bf16x2(__float_as_uint(yp[0]), __float_as_uint(yp[1]), ah[ai], am[ai], al[ai]);
      }
    // one accumulator per term, so that only two instructions depend on each other (a single chain of
    // six was a third of this function's time); the terms are added smallest first
    float accm[4][4], acch[4][4];
#pragma unroll
    for (int n = 0; n < 4; ++n)
#pragma unroll
      for (int e = 0; e < 4; ++e) { acc[n][e] = 0.f; accm[n][e] = 0.f; acch[n][e] = 0.f; }
#pragma unroll
    for (int kc = 0; kc < 2; ++kc)
#pragma unroll
      for (int n = 0; n < 4; ++n) {
        mma_16816_bf16(acc[n], al + 4 * kc, bfrag[kc][n]);
        mma_16816_bf16(accm[n], am + 4 * kc, bfrag[kc][n]);
        mma_16816_bf16(acch[n], ah + 4 * kc, bfrag[kc][n]);
      }
#pragma unroll
    for (int n = 0; n < 4; ++n)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[n][e] = (acc[n][e] + accm[n][e]) + acch[n][e];
  } else {
#pragma unroll
    for (int n = 0; n < 4; ++n)
#pragma unroll
      for (int rh = 0; rh < 2; ++rh) {
        const float* yp = y_s + (r8 + 8 * rh) * 33 + 8 * n + 2 * p;
        acc[n][2 * rh] = yp[0];
        acc[n][2 * rh + 1] = yp[1];
      }
  }
#pragma unroll
  for (int rh = 0; rh < 2; ++rh) {
    const float v[8] = {acc[0][2 * rh], acc[0][2 * rh + 1], acc[1][2 * rh], acc[1][2 * rh + 1],
                        acc[2][2 * rh], acc[2][2 * rh + 1], acc[3][2 * rh], acc[3][2 * rh + 1]};
    const int row = row0 + r8 + 8 * rh;
    const bool live = store && row < M;
    uint32_t word, sb;
    if constexpr (FMT == FMT_MXINT4) {
      uint32_t pr[4];
      mxint4_quantize_row_fragment(v, pr, sb);
      if (live) {
        uint8_t* dst = codes + (size_t)row * d + blk * 32 + 2 * p;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) *reinterpret_cast<uint16_t*>(dst + 8 * nt) = (uint16_t)pr[nt];
      }
    } else {
      if constexpr (FMT == FMT_NVFP4) nv_quantize_row_fragment(v, p, nv_scale(tensor_scale), word, sb);
      else quantize_row_fragment(v, p, word, sb);
      if (live) *reinterpret_cast<uint32_t*>(codes + (size_t)row * (d / 2) + blk * 16 + 4 * p) = word;
    }
    if (p == 0 && store) {
      if constexpr (FMT == FMT_NVFP4) {
        scales[scale_offset(row, 2 * blk, kb4)] = live ? (uint8_t)(sb & 0xFF) : (uint8_t)0;
        scales[scale_offset(row, 2 * blk + 1, kb4)] = live ? (uint8_t)(sb >> 8) : (uint8_t)0;
      } else {
        scales[scale_offset(row, blk, kb4)] = live ? (uint8_t)sb : (uint8_t)0;
      }
    }
  }
}

}  // namespace torq
