// Rotate + quantize for few tokens (fewer output tiles than half the SMs), where the work is
// streaming R_inter from HBM once: with one 128 x 256 tile per CTA only M/128 x d/256 CTAs would
// pull on the memory system (20 of 148 SMs at M <= 128, d = 5120).  Here the contraction is also split along K: CTA (n tile, k split) multiplies
// X[:, k range] by R_inter[k range, 256 columns] on the tensor cores and writes its fp32 partial
// tile to scratch; a second, small kernel adds the partials of each (token, 32-block) in split
// order, applies the intra-block rotation, and quantizes (Algorithm 3 steps 2-4; the quantizer
// needs the complete sum, so it cannot run per split).  Summation order is fixed: the result does
// not depend on timing.
//
// Scratch layout: P[split][rows padded to 128][d] fp32 (rows >= M of a 32-row group that holds a
// token are written as zeros; 32-row groups without any token are not written and not read).
#pragma once
#include <cuda_bf16.h>
#include "nvfp4_quantize.cuh"
#include "mxint4_quantize.cuh"
#include "sm100_ptx.cuh"

namespace torq {

struct RotSplitCfg {
  static constexpr int BM = 128, BN = 256, BK = 64;
  static constexpr int A_BYTES = BM * BK * 2;          // 16 KiB
  static constexpr int B_BOX_BYTES = 64 * BK * 2;      // 8 KiB
  static constexpr int B_BYTES = (BN / 64) * B_BOX_BYTES;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;   // 48 KiB
  static constexpr int STAGES = 4;
  static constexpr int OUT_WARP_BYTES = 32 * 128;      // staging for one [32 rows x 32 fp32] box
  static constexpr int OUT_BYTES = 4 * OUT_WARP_BYTES;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + OUT_BYTES + 256 + 1024;
  static constexpr int TMEM_COLS = 256;
  static constexpr int THREADS = 192;
  static constexpr int MAX_SPLITS = 8;
  static_assert(SMEM_BYTES <= 232448, "shared memory budget");
};

// grid = m_tiles * n_tiles * splits; CTA b works row tile b % m_tiles, n tile (b / m_tiles) % n_tiles,
// k split b / (m_tiles * n_tiles).  tmP: fp32 [splits * m_tiles * 128, d], box [32 rows x 32 columns],
// 128-byte swizzle.
__global__ void __launch_bounds__(192, 1)
rotate_splitk_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmR,
                     const __grid_constant__ CUtensorMap tmP, int M, int d, int splits, int* err_word) {
  using C = RotSplitCfg;
  constexpr int BN = C::BN;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t out_off = C::STAGES * C::STAGE_BYTES;
  const uint32_t bar_off = out_off + C::OUT_BYTES;
  const uint32_t bar_base = smem_base + bar_off;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (C::STAGES + s); };
  const uint32_t accf_bar = bar_base + 8u * (2 * C::STAGES);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + bar_off + 192);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(smem_gen + bar_off + 200);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tiles = (d + BN - 1) / BN;
  const int m_tiles = (M + C::BM - 1) / C::BM;
  const int mt = blockIdx.x % m_tiles, nt = (blockIdx.x / m_tiles) % n_tiles, ks = blockIdx.x / (m_tiles * n_tiles);
  const int k_tiles = (d + C::BK - 1) / C::BK;
  const int kt0 = (int)((long long)k_tiles * ks / splits);
  const int kt1 = (int)((long long)k_tiles * (ks + 1) / splits);

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(accf_bar, 1);
    *cta_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::TMEM_COLS); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // R_inter is a constant of the layer, never the output of the kernel that runs just before this
  // one: its loads for the first stages go out right away; everything else waits for that kernel.
  griddep_launch_dependents();
  const int pre = (kt1 - kt0) < C::STAGES ? (kt1 - kt0) : C::STAGES;
  if (warp == 0) {
    if (elect_one()) {
      tma_prefetch_desc(&tmX);
      tma_prefetch_desc(&tmR);
      for (int it = 0; it < pre; ++it) {
        const uint32_t st = smem_base + it * C::STAGE_BYTES;
        mbar_arrive_expect_tx(full_bar(it), C::STAGE_BYTES);
#pragma unroll
        for (int b = 0; b < BN / 64; ++b)
          tma_load_2d(st + C::A_BYTES + b * C::B_BOX_BYTES, &tmR, nt * BN + b * 64, (kt0 + it) * C::BK, full_bar(it));
      }
    }
    __syncwarp();
  }
  griddep_wait();

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    bool ok = true;
    for (int kt = kt0, it = 0; kt < kt1 && ok; ++kt, ++it) {
      const int s = it % C::STAGES;
      if (!mbar_wait_warp(empty_bar(s), ((it / C::STAGES) & 1) ^ 1, cta_abort, err_word,
                          SITE_PRODUCER_EMPTY)) { ok = false; break; }
      const uint32_t st = smem_base + s * C::STAGE_BYTES;
      if (elect_one()) {
        const bool r_issued = it < pre;                  // R side of this stage went out before the wait above
        if (!r_issued) mbar_arrive_expect_tx(full_bar(s), C::STAGE_BYTES);
        tma_load_2d(st, &tmX, kt * C::BK, mt * C::BM, full_bar(s));
        if (!r_issued) {
#pragma unroll
          for (int b = 0; b < BN / 64; ++b)
            tma_load_2d(st + C::A_BYTES + b * C::B_BOX_BYTES, &tmR, nt * BN + b * 64, kt * C::BK, full_bar(s));
        }
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    constexpr uint32_t idesc = idesc_bf16(128, BN, /*A MN-major*/ false, /*B MN-major*/ true);
    bool ok = true;
    for (int kt = kt0, it = 0; kt < kt1 && ok; ++kt, ++it) {
      const int s = it % C::STAGES;
      if (!mbar_wait_warp(full_bar(s), (it / C::STAGES) & 1, cta_abort, err_word, SITE_MMA_FULL)) {
        ok = false; break;
      }
      tc_fence_after_sync();
      const uint32_t st = smem_base + s * C::STAGE_BYTES;
      const uint64_t adesc = make_desc(st, 16, 1024, kSwizzle128);
      const uint64_t bdesc = make_desc(st + C::A_BYTES, C::B_BOX_BYTES, 1024, kSwizzle128);
      if (elect_one()) {
#pragma unroll
        for (int j = 0; j < C::BK / 16; ++j)
          mma_bf16(tmem_base, adesc + 2 * j, bdesc + 128 * j, idesc, (it | j) != 0);
        tc_commit(empty_bar(s));
      }
      __syncwarp();
    }
    if (ok && elect_one()) tc_commit(accf_bar);
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue: partial tile -> scratch
    const int q = warp & 3;
    bool ok = mbar_wait(accf_bar, 0, cta_abort, err_word, SITE_EPI_ACC_FULL);
    ok = __all_sync(0xFFFFFFFFu, ok);
    if (ok && mt * C::BM + q * 32 < M) {                 // this 32-row group holds at least one token
      tc_fence_after_sync();
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16);
      const uint32_t stage_buf = smem_base + out_off + (uint32_t)(warp - 2) * C::OUT_WARP_BYTES;
      const uint32_t my_row = stage_buf + lane * 128;
      const uint32_t sw = (uint32_t)(lane & 7);
#pragma unroll 1
      for (int bb = 0; bb < BN / 32; ++bb) {
        uint32_t v[32];
        tmem_ld_32x32(tacc + bb * 32, v);
        tmem_ld_wait();
        if (bb > 0) {                                    // the previous store has read the buffer
          if (lane == 0) bulk_wait_group_read<0>();
          __syncwarp();
        }
#pragma unroll
        for (int p = 0; p < 8; ++p)
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                       ::"r"(my_row + (((uint32_t)p ^ sw) << 4)), "r"(v[4 * p]), "r"(v[4 * p + 1]),
                         "r"(v[4 * p + 2]), "r"(v[4 * p + 3]) : "memory");
        fence_proxy_async_smem();
        __syncwarp();
        const int col = nt * BN + bb * 32;
        if (lane == 0 && col < d) {
          tma_store_2d(&tmP, col, (ks * m_tiles + mt) * C::BM + q * 32, stage_buf);
          bulk_commit_group();
        }
      }
      if (lane == 0) bulk_wait_group<0>();
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before_sync();
  __syncthreads();
  if (*cta_abort) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

// Second phase: one CTA of 8 warps per (32-block b, group of 32 rows).
//  1. All warps add the partials P[s][row][32 b + j] in split order into a shared-memory tile
//     (a warp reads one row's 128 bytes per split; all loads of the CTA are in flight together, so
//     the phase costs one memory latency).
//  2. The intra-block rotation z = y R_intra[b] of the 32 x 32 tile on the warp-level tensor-core
//     path (two warps, 16 rows each): y split into three bf16 terms, R_intra exact in bf16, fp32
//     accumulation -- 48 MMAs instead of a thousand FMA instructions per warp, which is what the
//     kernel's time was.  Then Eq. 1 on the accumulator fragments (four lanes share a row: block
//     maximum by two shuffles, a 4 x 4 byte transpose so that each lane stores 4 contiguous code
//     bytes).  Without R_intra: four threads per row on the sums themselves.
// Rows M .. (group end) and K-blocks d/32 .. (padded to 4) only get their padding scale byte (0).
// FMT_NVFP4: the 32 columns are two 16-element blocks (two threads each), E4M3 scales at twice the
// block index, `tensor_scale` the tensor's float32 scale; the grid covers the padded 16-blocks in pairs.
// FMT_MXINT4: integer codes as one E4M3 operand byte per element (`codes` is [M, d] bytes).
template <int FMT = FMT_MXFP4>
__global__ void __launch_bounds__(256)
splitk_reduce_quantize_kernel(const float* __restrict__ P, const __nv_bfloat16* __restrict__ R_intra,
                              int M, int d, int splits, float tensor_scale, uint8_t* __restrict__ codes,
                              uint8_t* __restrict__ scales) {
  __shared__ float y_s[32 * 33];                         // row stride 33: conflict-free by row and by column
  __shared__ __align__(16) uint8_t r_s[32 * 80];         // R_intra[b], bf16, 80-byte rows: conflict-free ldmatrix
  griddep_launch_dependents();
  griddep_wait();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int nb = d / 32;
  const int kb4 = FMT == FMT_NVFP4 ? (2 * nb + 3) / 4 : (nb + 3) / 4;   // 4-byte scale groups per row
  const int nbp = FMT == FMT_NVFP4 ? kb4 * 2 : kb4 * 4;                  // padded count of 32-column blocks
  const int b = blockIdx.x % nbp, rg = blockIdx.x / nbp;  // row group: rows 32 rg .. 32 rg + 31
  const int m_tiles = (M + 127) / 128;
  const int row0 = rg * 32;
  const int rows = max(0, min(32, M - row0));            // real rows of this group
  if (b >= nb || rows == 0) {                            // padding only: zero scale bytes
    if (threadIdx.x < 32) {
      if constexpr (FMT == FMT_NVFP4) {
        scales[scale_offset(row0 + threadIdx.x, 2 * b, kb4)] = 0;
        scales[scale_offset(row0 + threadIdx.x, 2 * b + 1, kb4)] = 0;
      } else {
        scales[scale_offset(row0 + threadIdx.x, b, kb4)] = 0;
      }
    }
    return;
  }
  const size_t split_stride = (size_t)m_tiles * 128 * d;
  // ---- 1. partial sums -> shared memory
#pragma unroll 4
  for (int r = warp; r < rows; r += nwarps) {
    const float* p = P + (size_t)(row0 + r) * d + b * 32 + lane;
    constexpr int MS = RotSplitCfg::MAX_SPLITS;          // every split's partial is loaded before the first add
    float part[MS];
#pragma unroll
    for (int s = 0; s < MS; ++s) part[s] = s < splits ? __ldg(p + s * split_stride) : 0.f;
    float y = 0.f;
#pragma unroll
    for (int s = 0; s < MS; ++s) if (s < splits) y += part[s];
    y_s[r * 33 + lane] = y;
  }
  for (int r = rows + warp; r < 32; r += nwarps) y_s[r * 33 + lane] = 0.f;     // rows past M: zeros
  if (R_intra != nullptr && threadIdx.x < 128) {
    const int i = threadIdx.x >> 2, c = (threadIdx.x & 3) * 8;
    *reinterpret_cast<uint4*>(r_s + i * 80 + c * 2) =
        __ldg(reinterpret_cast<const uint4*>(R_intra + (size_t)b * 1024 + threadIdx.x * 8));
  }
  __syncthreads();
  if (R_intra != nullptr) {
    // ---- 2a. two warps, 16 rows each, on the warp-level tensor cores
    if (warp >= 2) return;
    const int p = lane & 3, r8 = lane >> 2;
    uint32_t bfrag[2][4][2];                             // [k chunk][n tile][2]
    {
      // lane l: row l % 8 of matrix l / 8; matrices (k 0-7, n), (k 8-15, n), (k 0-7, n+8), (k 8-15, n+8)
      const uint32_t rb = smem_u32(r_s) + (uint32_t)(((lane >> 3) & 1) * 8 + (lane & 7)) * 80 + (uint32_t)(lane >> 4) * 16;
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
        const float* yp = y_s + (16 * warp + r8 + 8 * rh) * 33 + 8 * n + 2 * p;
        const int ai = (n >> 1) * 4 + (n & 1) * 2 + rh;
        split3_bf16x2(__float_as_uint(yp[0]), __float_as_uint(yp[1]), ah[ai], am[ai], al[ai]);
      }
    float acc[4][4];
#pragma unroll
    for (int n = 0; n < 4; ++n) { acc[n][0] = 0.f; acc[n][1] = 0.f; acc[n][2] = 0.f; acc[n][3] = 0.f; }
#pragma unroll
    for (int kc = 0; kc < 2; ++kc)
#pragma unroll
      for (int n = 0; n < 4; ++n) {
        mma_16816_bf16(acc[n], al + 4 * kc, bfrag[kc][n]);
        mma_16816_bf16(acc[n], am + 4 * kc, bfrag[kc][n]);
        mma_16816_bf16(acc[n], ah + 4 * kc, bfrag[kc][n]);
      }
#pragma unroll
    for (int rh = 0; rh < 2; ++rh) {
      const float v[8] = {acc[0][2 * rh], acc[0][2 * rh + 1], acc[1][2 * rh], acc[1][2 * rh + 1],
                          acc[2][2 * rh], acc[2][2 * rh + 1], acc[3][2 * rh], acc[3][2 * rh + 1]};
      const int r = 16 * warp + r8 + 8 * rh;
      const int row = row0 + r;
      uint32_t word, sb;
      if constexpr (FMT == FMT_MXINT4) {
        uint32_t pr[4];
        mxint4_quantize_row_fragment(v, pr, sb);
        if (r < rows) {
          uint8_t* dst = codes + (size_t)row * d + b * 32 + 2 * p;
#pragma unroll
          for (int nt = 0; nt < 4; ++nt) *reinterpret_cast<uint16_t*>(dst + 8 * nt) = (uint16_t)pr[nt];
        }
      } else {
        if constexpr (FMT == FMT_NVFP4) nv_quantize_row_fragment(v, p, nv_scale(tensor_scale), word, sb);
        else quantize_row_fragment(v, p, word, sb);
        if (r < rows) *reinterpret_cast<uint32_t*>(codes + (size_t)row * (d / 2) + b * 16 + 4 * p) = word;
      }
      if (p == 0) {
        if constexpr (FMT == FMT_NVFP4) {
          scales[scale_offset(row, 2 * b, kb4)] = r < rows ? (uint8_t)(sb & 0xFF) : (uint8_t)0;
          scales[scale_offset(row, 2 * b + 1, kb4)] = r < rows ? (uint8_t)(sb >> 8) : (uint8_t)0;
        } else {
          scales[scale_offset(row, b, kb4)] = r < rows ? (uint8_t)sb : (uint8_t)0;
        }
      }
    }
    return;
  }
  // ---- 2b. no intra rotation: four threads per row on the sums
  if (threadIdx.x >= 128) return;
  const int r = threadIdx.x >> 2, p = threadIdx.x & 3;
  const int row = row0 + r;
  float z[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) z[j] = y_s[r * 33 + 8 * p + j];
  float amax = 0.f;
#pragma unroll
  for (int j = 0; j < 8; ++j) amax = fmaxf(amax, fabsf(z[j]));
  amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
  if constexpr (FMT == FMT_NVFP4) {                      // a 16-element block = two threads
    uint32_t sb;
    float rr;
    nv_block_scale(amax, nv_scale(tensor_scale), sb, rr);
    if (r < rows) {
      const uint32_t w = pack8_e2m1(__fmul_rn(z[0], rr), __fmul_rn(z[1], rr), __fmul_rn(z[2], rr), __fmul_rn(z[3], rr),
                                    __fmul_rn(z[4], rr), __fmul_rn(z[5], rr), __fmul_rn(z[6], rr), __fmul_rn(z[7], rr));
      *reinterpret_cast<uint32_t*>(codes + (size_t)row * (d / 2) + b * 16 + 4 * p) = w;
    }
    if ((p & 1) == 0) scales[scale_offset(row, 2 * b + (p >> 1), kb4)] = r < rows ? (uint8_t)sb : (uint8_t)0;
    return;
  }
  amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
  uint32_t sbyte;
  float inv;
  block_scale(amax, sbyte, inv);
  if (r < rows) {
    if constexpr (FMT == FMT_MXINT4) {
      *reinterpret_cast<uint2*>(codes + (size_t)row * d + b * 32 + 8 * p) = make_uint2(
          pack4_e4m3(int4_round(z[0] * inv), int4_round(z[1] * inv), int4_round(z[2] * inv), int4_round(z[3] * inv)),
          pack4_e4m3(int4_round(z[4] * inv), int4_round(z[5] * inv), int4_round(z[6] * inv), int4_round(z[7] * inv)));
    } else {
      const uint32_t w = pack8_e2m1(z[0] * inv, z[1] * inv, z[2] * inv, z[3] * inv, z[4] * inv, z[5] * inv,
                                    z[6] * inv, z[7] * inv);
      *reinterpret_cast<uint32_t*>(codes + (size_t)row * (d / 2) + b * 16 + 4 * p) = w;
    }
  }
  if (p == 0) scales[scale_offset(row, b, kb4)] = r < rows ? (uint8_t)sbyte : (uint8_t)0;
}

}  // namespace torq
