// Block-scaled MXFP4 x MXFP4 GEMM (Algorithm 3 step 5, option B) on the tcgen05 FP4 tensor
// cores: Y[m,n] = sum_k a^[m,k] w^[n,k] with one E8M0 scale per 32 elements of K on each side.
//
// Persistent, warp-specialised, one CTA per SM:
//   warp 0      TMA producer  : A / W tiles (128-byte swizzle) and their scale tiles into a
//                               ring of shared-memory stages
//   warp 1      MMA issuer    : copies the scale tiles shared -> tensor memory (tcgen05.cp),
//                               issues tcgen05.mma kind::mxf4.block_scale, commits to barriers
//   warps 2..5  epilogue      : tensor memory -> registers -> Y (fp32 or bf16), 32 rows per warp
// Tile = 128 x BN x 256 (one stage = 128 bytes of K per row = one swizzle atom).  NACC
// accumulator buffers in tensor memory let the epilogue of one tile overlap the next mainloop.
//
// The same kernel serves the NVFP4 variant (FMT_NVFP4: kind::mxf4nvf4, one E4M3 scale per 16
// elements of K, the product of the two tensor scales applied in the epilogue).  Scale bytes come
// in 512-byte chunks of 128 rows x 4 bytes; one chunk covers 128 elements of K in MXFP4 and 64 in
// NVFP4, so a stage holds CH = 2 or 4 chunks per 128 rows, four tensor-memory columns each.
//
// FMT_MXINT4: the integer codes arrive as E4M3 operand bytes, one per element (kind::mxf8f6f4, E8M0
// scale per 32 elements of K).  A stage is still 128 bytes of K per row, now 128 elements: one
// scale chunk, four instructions of K = 32 that take bytes 0..3 of the chunk's 4-byte cells.
#pragma once
#include <cuda_bf16.h>
#include "sm100_ptx.cuh"

namespace torq {

template <int BN, int NACC, int FMT = FMT_MXFP4>
struct GemmCfg {
  static constexpr int BM = 128;
  static constexpr int BK = FMT == FMT_MXINT4 ? 128 : 256;   // elements of K per stage (128 bytes per row)
  static constexpr int A_BYTES = BM * 128;             // 16 KiB
  static constexpr int B_BYTES = BN * 128;
  static constexpr int CH = FMT == FMT_NVFP4 ? 4 : (FMT == FMT_MXINT4 ? 1 : 2);   // scale chunks per stage and 128 rows
  static constexpr int SFA_BYTES = CH * 512;
  static constexpr int SFB_BYTES = (BN / 128) * SFA_BYTES;
  static constexpr int STAGE_BYTES = (A_BYTES + B_BYTES + SFA_BYTES + SFB_BYTES + 1023) / 1024 * 1024;   // swizzle atoms need 1 KiB
  static constexpr int STAGES = (BN == 256) ? 4 : 6;
  static constexpr int BAR_BYTES = 256;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + BAR_BYTES + 1024;  // + align slack
  static constexpr int ACC_COLS = NACC * BN;
  static constexpr int SFA_COL = ACC_COLS;             // CH chunks x 4 columns
  static constexpr int SFB_COL = ACC_COLS + 4 * CH;    // CH chunks x BN/32 columns
  static constexpr int TMEM_COLS = 512;
  static constexpr int THREADS = 192;
  static_assert(SFB_COL + CH * (BN / 32) <= TMEM_COLS, "tensor memory budget");
  static_assert(SMEM_BYTES <= 232448, "shared memory budget");
};

template <int BN, int NACC, int FMT = FMT_MXFP4>
__global__ void __launch_bounds__(192, 1)
mxfp4_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const uint8_t* __restrict__ As, const uint8_t* __restrict__ Ws,
                  void* __restrict__ Y, int y_is_bf16, int M, int N, int K, float alpha, int* err_word) {
  using C = GemmCfg<BN, NACC, FMT>;
  constexpr int CH = C::CH;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + C::STAGES * C::STAGE_BYTES;
  // barrier map (8 bytes each): full[s], empty[s], acc_full[a], acc_empty[a]
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (C::STAGES + s); };
  auto accf_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + a); };
  auto acce_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + NACC + a); };
  volatile uint32_t* tmem_slot =
      reinterpret_cast<volatile uint32_t*>(smem_gen + C::STAGES * C::STAGE_BYTES + 192);
  volatile int* cta_abort =
      reinterpret_cast<volatile int*>(smem_gen + C::STAGES * C::STAGE_BYTES + 200);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_tiles = (M + C::BM - 1) / C::BM;
  const int n_tiles = (N + BN - 1) / BN;
  const int total_tiles = m_tiles * n_tiles;
  const int k_tiles = (K + C::BK - 1) / C::BK;          // K % 128 == 0: last stage may be half
  const int kb4 = K / (C::BK / CH);                     // scale chunks (4 K-blocks each) per row
  const int n_rowtiles = (N + 127) / 128;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < NACC; ++a) { mbar_init(accf_bar(a), 1); mbar_init(acce_bar(a), 4); }
    *cta_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::TMEM_COLS); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // Set-up above touched no global memory.  The weights and their scales are constants of the
  // layer, never the output of the kernel that runs just before this one: the first stages' W
  // loads go out right away; everything else waits until that kernel has completed.
  griddep_launch_dependents();
  const int pre = (int)blockIdx.x < total_tiles ? (k_tiles < C::STAGES ? k_tiles : C::STAGES) : 0;
  if (warp == 0) {
    if (elect_one()) {
      tma_prefetch_desc(&tmA);
      tma_prefetch_desc(&tmB);
      const int mt = blockIdx.x % m_tiles, nt = blockIdx.x / m_tiles;
      const int rt0 = nt * (BN / 128);
      const int n_sfb_tiles = min(BN / 128, n_rowtiles - rt0);
      (void)mt;
      for (int kt = 0; kt < pre; ++kt) {
        const uint32_t sf_bytes = 512u * min(CH, kb4 - CH * kt);
        const uint32_t st = smem_base + kt * C::STAGE_BYTES;
        mbar_arrive_expect_tx(full_bar(kt), C::A_BYTES + C::B_BYTES + sf_bytes * (1 + n_sfb_tiles));
        tma_load_2d(st + C::A_BYTES, &tmB, kt * 128, nt * BN, full_bar(kt));
        for (int t = 0; t < n_sfb_tiles; ++t)
          bulk_load_1d(st + C::A_BYTES + C::B_BYTES + C::SFA_BYTES + t * C::SFA_BYTES,
                       Ws + ((size_t)(rt0 + t) * kb4 + CH * kt) * 512, sf_bytes, full_bar(kt));
      }
    }
    __syncwarp();
  }
  griddep_wait();

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    uint32_t it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int mt = tile % m_tiles, nt = tile / m_tiles;
      const int rt0 = nt * (BN / 128);
      const int n_sfb_tiles = min(BN / 128, n_rowtiles - rt0);
      for (int kt = 0; kt < k_tiles; ++kt, ++it) {
        const int s = it % C::STAGES;
        if (!mbar_wait_warp(empty_bar(s), ((it / C::STAGES) & 1) ^ 1, cta_abort, err_word,
                       SITE_PRODUCER_EMPTY)) { ok = false; break; }
        const int nchunk = min(CH, kb4 - CH * kt);
        const uint32_t sf_bytes = 512u * nchunk;
        const uint32_t st = smem_base + s * C::STAGE_BYTES;
        if (elect_one()) {
          const bool w_issued = it < (uint32_t)pre;      // W side of this stage went out before the wait above
          if (!w_issued) mbar_arrive_expect_tx(full_bar(s), C::A_BYTES + C::B_BYTES + sf_bytes * (1 + n_sfb_tiles));
          tma_load_2d(st, &tmA, kt * 128, mt * C::BM, full_bar(s));
          bulk_load_1d(st + C::A_BYTES + C::B_BYTES, As + ((size_t)mt * kb4 + CH * kt) * 512, sf_bytes,
                       full_bar(s));
          if (!w_issued) {
            tma_load_2d(st + C::A_BYTES, &tmB, kt * 128, nt * BN, full_bar(s));
            for (int t = 0; t < n_sfb_tiles; ++t)
              bulk_load_1d(st + C::A_BYTES + C::B_BYTES + C::SFA_BYTES + t * C::SFA_BYTES,
                           Ws + ((size_t)(rt0 + t) * kb4 + CH * kt) * 512, sf_bytes, full_bar(s));
          }
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    uint32_t it = 0, tcount = 0;
    bool ok = true;
    constexpr uint32_t idesc0 = FMT == FMT_NVFP4 ? idesc_nvf4(128, BN) : idesc_mxf4(128, BN, 0, 0);
    constexpr uint32_t idesc2 = FMT == FMT_NVFP4 ? idesc_nvf4(128, BN) : idesc_mxf4(128, BN, 2, 2);
    const uint32_t sfa_t = tmem_base + C::SFA_COL, sfb_t = tmem_base + C::SFB_COL;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
      const int a = tcount % NACC;
      if (!mbar_wait_warp(acce_bar(a), ((tcount / NACC) & 1) ^ 1, cta_abort, err_word,
                     SITE_MMA_ACC_EMPTY)) { ok = false; break; }
      tc_fence_after_sync();
      const uint32_t acc = tmem_base + a * BN;
      for (int kt = 0; kt < k_tiles; ++kt, ++it) {
        const int s = it % C::STAGES;
        if (!mbar_wait_warp(full_bar(s), (it / C::STAGES) & 1, cta_abort, err_word, SITE_MMA_FULL)) {
          ok = false; break;
        }
        tc_fence_after_sync();
        const bool two = (kb4 - CH * kt) >= CH;            // K % 256 == 128: the last stage is half
        const uint32_t st = smem_base + s * C::STAGE_BYTES;
        const uint64_t adesc = make_desc(st, 16, 1024, kSwizzle128);
        const uint64_t bdesc = make_desc(st + C::A_BYTES, 16, 1024, kSwizzle128);
        const uint64_t sfa_d = make_desc(st + C::A_BYTES + C::B_BYTES, 0, 128, 0);
        const uint64_t sfb_d = make_desc(st + C::A_BYTES + C::B_BYTES + C::SFA_BYTES, 0, 128, 0);
        if (elect_one()) {
          // scale chunks shared -> tensor memory (descriptor address unit = 16 B: +32 = next
          // chunk, + SFA_BYTES / 16 = next 128-row tile of W), then 64 elements of K per instruction
#pragma unroll
          for (int c = 0; c < CH; ++c) {
            if (c < CH / 2 || two) {
              tmem_cp_32x128b_warpx4(sfa_t + 4 * c, sfa_d + 32 * c);
#pragma unroll
              for (int t = 0; t < BN / 128; ++t)
                tmem_cp_32x128b_warpx4(sfb_t + c * (BN / 32) + 4 * t, sfb_d + (C::SFA_BYTES / 16) * t + 32 * c);
            }
          }
          if constexpr (FMT == FMT_MXINT4) {               // a quarter chunk (one scale byte) per instruction
            mma_mxf8(acc, adesc, bdesc, idesc_mxf8(128, BN, 0), sfa_t, sfb_t, kt != 0);
            mma_mxf8(acc, adesc + 2, bdesc + 2, idesc_mxf8(128, BN, 1), sfa_t, sfb_t, 1);
            mma_mxf8(acc, adesc + 4, bdesc + 4, idesc_mxf8(128, BN, 2), sfa_t, sfb_t, 1);
            mma_mxf8(acc, adesc + 6, bdesc + 6, idesc_mxf8(128, BN, 3), sfa_t, sfb_t, 1);
          } else if constexpr (FMT == FMT_NVFP4) {         // one chunk per instruction
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (j < 2 || two)
                mma_nvf4(acc, adesc + 2 * j, bdesc + 2 * j, idesc0, sfa_t + 4 * j, sfb_t + j * (BN / 32), (kt | j) != 0);
          } else {                                         // half a chunk (two scale bytes) per instruction
            mma_mxf4(acc, adesc, bdesc, idesc0, sfa_t, sfb_t, kt != 0);
            mma_mxf4(acc, adesc + 2, bdesc + 2, idesc2, sfa_t, sfb_t, 1);
            if (two) {
              mma_mxf4(acc, adesc + 4, bdesc + 4, idesc0, sfa_t + 4, sfb_t + BN / 32, 1);
              mma_mxf4(acc, adesc + 6, bdesc + 6, idesc2, sfa_t + 4, sfb_t + BN / 32, 1);
            }
          }
          tc_commit(empty_bar(s));
        }
        __syncwarp();
      }
      if (ok && elect_one()) tc_commit(accf_bar(a));
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int q = warp & 3;                              // lane quarter this warp may read
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
      const int mt = tile % m_tiles, nt = tile / m_tiles;
      const int a = tcount % NACC;
      ok = mbar_wait(accf_bar(a), (tcount / NACC) & 1, cta_abort, err_word, SITE_EPI_ACC_FULL);
      ok = __all_sync(0xFFFFFFFFu, ok);                  // keep the warp together on the way out
      if (!ok) break;
      tc_fence_after_sync();
      const int64_t row = (int64_t)mt * C::BM + q * 32 + lane;
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + a * BN;
#pragma unroll 1
      for (int cc = 0; cc < BN / 32; ++cc) {
        uint32_t v[32];
        tmem_ld_32x32(tacc + cc * 32, v);
        tmem_ld_wait();
        if constexpr (FMT == FMT_NVFP4) {                // product of the two tensor scales
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * alpha);
        }
        if (cc == BN / 32 - 1) {                         // accumulator fully read: hand it back
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(acce_bar(a));
        }
        const int64_t col = (int64_t)nt * BN + cc * 32;
        if (row < M && col < N) {
          if (y_is_bf16) {
            __nv_bfloat16* yp = reinterpret_cast<__nv_bfloat16*>(Y) + row * N + col;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              if (col + 8 * g + 8 <= N) {
                uint4 o;
                uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                  __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[8 * g + 2 * p]),
                                                           __uint_as_float(v[8 * g + 2 * p + 1]));
                  ow[p] = *reinterpret_cast<uint32_t*>(&h);
                }
                *reinterpret_cast<uint4*>(yp + 8 * g) = o;
              }
            }
          } else {
            float* yp = reinterpret_cast<float*>(Y) + row * N + col;
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              if (col + 4 * g + 4 <= N)
                *reinterpret_cast<uint4*>(yp + 4 * g) =
                    make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
            }
          }
        }
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before_sync();
  __syncthreads();
  if (*cta_abort) {
    // A wait gave up: give in-flight copies and MMAs time to land before the CTA's shared and
    // tensor memory go away.
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

}  // namespace torq
