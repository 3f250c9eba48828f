// Block-scaled MXFP4 GEMM on CTA pairs (M > 128): two CTAs share one 256 x 256 output tile through
// tcgen05.mma cta_group::2 kind::mxf4.block_scale.  Each CTA stages its own 128 rows of A, its own
// 128 rows of W, its own A scales and the full tile's W scales (35 KiB per 256 elements of K
// instead of 51 KiB), five stages deep.  Every CTA loads only for itself.
//
// The 128 x 256 fp32 accumulator of each CTA fills half of tensor memory and the scale factors
// need columns too, so there is a single accumulator buffer; to keep the tensor pipe busy the
// eight epilogue warps first drain the whole accumulator into registers (128 values per thread),
// hand it back to the MMA warp at once, and only then convert and store: each warp writes its
// rows into a 4 KiB swizzled staging buffer in shared memory and one lane issues a TMA store of
// the [32 rows x 128 bytes] box, so that Y is written in whole 128-byte lines (one thread writing
// 16 bytes of its own row per instruction made 32 partial-sector writes per warp store and ran at
// a third of the speed).
//
// Tiles are dealt round robin from the list MixedTiles describes: 256 x 256 tiles, and where those
// would leave the last wave partly empty, 256 x 192 tiles in its place (N = 192 instructions, 96
// rows of W per CTA; the tile's W scales are still two whole 128-row chunks, read from two columns
// further on when the tile starts 64 rows into its first chunk).
//
// Roles per CTA: warp 0 TMA producer, warp 1 MMA issuer (leader CTA only), warps 2..9 epilogue
// (warp w reads lane quarter w%4, column half (w-2)/4).  Barriers as in the pair rotation kernel;
// acc_empty takes one arrival per epilogue warp of both CTAs (16).
//
// FMT_NVFP4 runs the same pipeline with kind::mxf4nvf4 (one E4M3 scale per 16 elements of K:
// four 512-byte scale chunks per stage and 128 rows instead of two) and multiplies the result by
// the product of the two tensor scales in the epilogue.
//
// FMT_MXINT4: integer codes as E4M3 operand bytes (kind::mxf8f6f4, E8M0 scale per 32 elements of K):
// a stage is 128 elements of K, one scale chunk, four instructions of K = 32 taking bytes 0..3 of
// the chunk's 4-byte cells.
#pragma once
#include <cuda_bf16.h>
#include "sm100_ptx.cuh"

namespace torq {

template <int FMT = FMT_MXFP4>
struct GemmPairCfgT {
  static constexpr int BN = 256;
  static constexpr int BM = 128;                       // rows per CTA
  static constexpr int BK = FMT == FMT_MXINT4 ? 128 : 256;   // elements of K per stage (128 bytes per row)
  static constexpr int A_BYTES = BM * 128;             // 16 KiB
  static constexpr int B_BYTES = (BN / 2) * 128;       // 16 KiB
  static constexpr int CH = FMT == FMT_NVFP4 ? 4 : (FMT == FMT_MXINT4 ? 1 : 2);   // scale chunks per stage and 128 rows
  static constexpr int SF_BOXES = CH == 1 ? 1 : CH / 2;       // scale loads per stage and 128 rows:
  static constexpr int SF_BOX_WORDS = CH == 1 ? 128 : 256;    // 1 KiB (two chunks), or the single chunk
  static constexpr int SFA_BYTES = CH * 512;
  static constexpr int SFB_BYTES = 2 * SFA_BYTES;      // both 128-row tiles of the W scales
  static constexpr int STAGE_TX = A_BYTES + B_BYTES + SFA_BYTES + SFB_BYTES;      // bytes one CTA loads per stage
  static constexpr int STAGE_BYTES = (STAGE_TX + 1023) / 1024 * 1024;             // 35 / 38 / 34 KiB (swizzle atoms need 1 KiB)
  static constexpr int STAGES = 5;
  static constexpr int OUT_WARP_BYTES = 32 * 128;      // per epilogue warp: 32 rows x 128 B, swizzled
  static constexpr int OUT_BYTES = 8 * OUT_WARP_BYTES;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + OUT_BYTES + 256 + 1024;
  static constexpr int SFA_COL = 256;                  // CH chunks x 4 columns
  static constexpr int SFB_COL = 256 + 4 * CH;         // CH chunks x 8 columns
  static constexpr int TMEM_COLS = 512;
  static constexpr int THREADS = 320;
  static_assert(SMEM_BYTES <= 232448, "shared memory budget");
};
using GemmPairCfg = GemmPairCfgT<FMT_MXFP4>;

template <int FMT = FMT_MXFP4>
__global__ void __launch_bounds__(320, 1)
mxfp4_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                       const __grid_constant__ CUtensorMap tmSFA, const __grid_constant__ CUtensorMap tmSFB,
                       const __grid_constant__ CUtensorMap tmY, const __grid_constant__ CUtensorMap tmBn,
                       const MixedTiles tiles, int y_is_bf16, int M, int N, int K, float alpha, int* err_word) {
  using C = GemmPairCfgT<FMT>;
  constexpr int CH = C::CH;
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
  const uint32_t acce_bar = bar_base + 8u * (2 * C::STAGES + 1);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + bar_off + 192);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(smem_gen + bar_off + 200);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int total_tiles = tiles.total;
  const int k_tiles = (K + C::BK - 1) / C::BK;
  const int kb4 = K / (C::BK / CH);                    // scale chunks per row

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(accf_bar, 1);
    mbar_init(acce_bar, 16);
    *cta_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::TMEM_COLS); tmem_relinquish_pair(); }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_after_init();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // Set-up above touched no global memory.  The weights and their scales are constants of the
  // layer, never the output of the kernel that runs just before this one, so the producer starts
  // the first stages' W loads right away; everything else waits until that kernel has completed
  // (its output, the activations' codes and scales, is what the A-side loads read).
  griddep_launch_dependents();
  const int pre = pair < total_tiles ? (k_tiles < C::STAGES ? k_tiles : C::STAGES) : 0;
  if (warp == 0) {
    if (elect_one()) {
      tma_prefetch_desc(&tmA); tma_prefetch_desc(&tmB);
      tma_prefetch_desc(&tmSFA); tma_prefetch_desc(&tmSFB);
      int mp0 = 0, col0 = 0;
      bool narrow = false;
      if (pre > 0) { mixed_tile_coords(pair, tiles, mp0, col0, narrow); tma_prefetch_desc(&tmBn); }
      (void)mp0;
      const int bn_half = narrow ? kNarrowCols / 2 : BN / 2;
      for (int kt = 0; kt < pre; ++kt) {
        const uint32_t st = smem_base + kt * C::STAGE_BYTES;
        const uint32_t leader_full = map_to_cta(full_bar(kt), 0);
        if (rank == 0) mbar_arrive_expect_tx(full_bar(kt), 2 * (C::STAGE_TX - (BN / 2 - bn_half) * 128));
        tma_load_2d_pair(st + C::A_BYTES, narrow ? &tmBn : &tmB, kt * 128, col0 + (int)rank * bn_half, leader_full);
#pragma unroll
        for (int t = 0; t < 2; ++t)                      // one 1 KiB box = two chunks
#pragma unroll
          for (int b = 0; b < C::SF_BOXES; ++b)
            tma_load_2d_pair(st + C::A_BYTES + C::B_BYTES + C::SFA_BYTES + t * C::SFA_BYTES + b * 1024, &tmSFB,
                             kt * CH * 128 + b * 256, (col0 >> 7) + t, leader_full);
      }
    }
    __syncwarp();
  }
  griddep_wait();

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    uint32_t it = 0;
    bool ok = true;
    for (int tile = pair; tile < total_tiles && ok; tile += npairs) {
      int mp, tcol;
      bool narrow;
      mixed_tile_coords(tile, tiles, mp, tcol, narrow);
      const int mt = 2 * mp + (int)rank;
      // a 192-column tile takes 96 rows of W per CTA; its scale rows start at a multiple of 64, so the two
      // 128-row scale chunks from (tcol / 128) on still cover it
      const int bn_half = narrow ? kNarrowCols / 2 : BN / 2;
      const uint32_t stage_tx = 2 * (C::STAGE_TX - (BN / 2 - bn_half) * 128);
      for (int kt = 0; kt < k_tiles; ++kt, ++it) {
        const int s = it % C::STAGES;
        if (!mbar_wait_cluster_warp(empty_bar(s), ((it / C::STAGES) & 1) ^ 1, cta_abort, err_word,
                               SITE_PRODUCER_EMPTY)) { ok = false; break; }
        const uint32_t st = smem_base + s * C::STAGE_BYTES;
        const uint32_t leader_full = map_to_cta(full_bar(s), 0);
        if (elect_one()) {
          const bool w_issued = it < (uint32_t)pre;      // W side of this stage went out before the wait above
          if (rank == 0 && !w_issued) mbar_arrive_expect_tx(full_bar(s), stage_tx);
          tma_load_2d_pair(st, &tmA, kt * 128, mt * C::BM, leader_full);
          if (!w_issued)
            tma_load_2d_pair(st + C::A_BYTES, narrow ? &tmBn : &tmB, kt * 128, tcol + (int)rank * bn_half, leader_full);
          // scale tiles: one row of the [row tile, chunk x 512 B] view per 128 rows, in boxes of
          // 1 KiB (two chunks); anything outside the buffer arrives as zeros (scale 2^-127 or 0,
          // multiplying operand data that is zero there as well).
#pragma unroll
          for (int b = 0; b < C::SF_BOXES; ++b)
            tma_load_2d_pair(st + C::A_BYTES + C::B_BYTES + b * 1024, &tmSFA, kt * CH * 128 + b * 256, mt,
                             leader_full);
          if (!w_issued) {
#pragma unroll
            for (int t = 0; t < 2; ++t)
#pragma unroll
              for (int b = 0; b < C::SF_BOXES; ++b)
                tma_load_2d_pair(st + C::A_BYTES + C::B_BYTES + C::SFA_BYTES + t * C::SFA_BYTES + b * 1024, &tmSFB,
                                 kt * CH * 128 + b * 256, (tcol >> 7) + t, leader_full);
          }
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    if (rank == 0) {
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      // instruction descriptors differ between the two tile widths only in the N field ([17,23) = N >> 3)
      constexpr uint32_t n_less = (uint32_t)((BN - kNarrowCols) >> 3) << 17;
      const uint32_t sfa_t = tmem_base + C::SFA_COL, sfb_t = tmem_base + C::SFB_COL;
      for (int tile = pair; tile < total_tiles && ok; tile += npairs, ++tcount) {
        int mp, tcol;
        bool narrow;
        mixed_tile_coords(tile, tiles, mp, tcol, narrow);
        (void)mp;
        const uint32_t nsub = narrow ? n_less : 0u;
        const uint32_t idesc0 = (FMT == FMT_NVFP4 ? idesc_nvf4(256, BN) : idesc_mxf4(256, BN, 0, 0)) - nsub;
        const uint32_t idesc2 = (FMT == FMT_NVFP4 ? idesc_nvf4(256, BN) : idesc_mxf4(256, BN, 2, 2)) - nsub;
        // The W scales of rows 32 j .. 32 j + 31 of a 128-row chunk sit in column j of the chunk's four
        // columns: a tile that starts 64 rows into its first chunk reads them from two columns further on.
        const uint32_t sfb_m = sfb_t + ((tcol & 127) ? 2u : 0u);
        if (!mbar_wait_cluster_warp(acce_bar, (tcount & 1) ^ 1, cta_abort, err_word, SITE_MMA_ACC_EMPTY)) {
          ok = false; break;
        }
        tc_fence_after_sync();
        for (int kt = 0; kt < k_tiles; ++kt, ++it) {
          const int s = it % C::STAGES;
          if (!mbar_wait_cluster_warp(full_bar(s), (it / C::STAGES) & 1, cta_abort, err_word, SITE_MMA_FULL)) {
            ok = false; break;
          }
          tc_fence_after_sync();
          const bool two = (kb4 - CH * kt) >= CH;          // K % 256 == 128: the last stage is half
          const uint32_t st = smem_base + s * C::STAGE_BYTES;
          const uint64_t adesc = make_desc(st, 16, 1024, kSwizzle128);
          const uint64_t bdesc = make_desc(st + C::A_BYTES, 16, 1024, kSwizzle128);
          const uint64_t sfa_d = make_desc(st + C::A_BYTES + C::B_BYTES, 0, 128, 0);
          const uint64_t sfb_d = make_desc(st + C::A_BYTES + C::B_BYTES + C::SFA_BYTES, 0, 128, 0);
          if (elect_one()) {
            // scale chunks shared -> tensor memory (descriptor address unit = 16 B: +32 = next
            // chunk, + SFA_BYTES / 16 = second 128-row tile of W), then 64 elements of K per instruction
#pragma unroll
            for (int c = 0; c < CH; ++c) {
              if (c < CH / 2 || two) {
                tmem_cp_32x128b_warpx4_pair(sfa_t + 4 * c, sfa_d + 32 * c);
                tmem_cp_32x128b_warpx4_pair(sfb_t + 8 * c, sfb_d + 32 * c);
                tmem_cp_32x128b_warpx4_pair(sfb_t + 8 * c + 4, sfb_d + 32 * c + C::SFA_BYTES / 16);
              }
            }
            if constexpr (FMT == FMT_MXINT4) {             // a quarter chunk (one scale byte) per instruction
              mma_mxf8_pair(tmem_base, adesc, bdesc, idesc_mxf8(256, BN, 0) - nsub, sfa_t, sfb_m, kt != 0);
              mma_mxf8_pair(tmem_base, adesc + 2, bdesc + 2, idesc_mxf8(256, BN, 1) - nsub, sfa_t, sfb_m, 1);
              mma_mxf8_pair(tmem_base, adesc + 4, bdesc + 4, idesc_mxf8(256, BN, 2) - nsub, sfa_t, sfb_m, 1);
              mma_mxf8_pair(tmem_base, adesc + 6, bdesc + 6, idesc_mxf8(256, BN, 3) - nsub, sfa_t, sfb_m, 1);
            } else if constexpr (FMT == FMT_NVFP4) {       // one chunk per instruction
#pragma unroll
              for (int j = 0; j < 4; ++j)
                if (j < 2 || two)
                  mma_nvf4_pair(tmem_base, adesc + 2 * j, bdesc + 2 * j, idesc0, sfa_t + 4 * j, sfb_m + 8 * j,
                                (kt | j) != 0);
            } else {                                       // half a chunk (two scale bytes) per instruction
              mma_mxf4_pair(tmem_base, adesc, bdesc, idesc0, sfa_t, sfb_m, kt != 0);
              mma_mxf4_pair(tmem_base, adesc + 2, bdesc + 2, idesc2, sfa_t, sfb_m, 1);
              if (two) {
                mma_mxf4_pair(tmem_base, adesc + 4, bdesc + 4, idesc0, sfa_t + 4, sfb_m + 8, 1);
                mma_mxf4_pair(tmem_base, adesc + 6, bdesc + 6, idesc2, sfa_t + 4, sfb_m + 8, 1);
              }
            }
            tc_commit_pair(empty_bar(s), 3);
          }
          __syncwarp();
        }
        if (ok && elect_one()) tc_commit_pair(accf_bar, 3);
        __syncwarp();
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (8 warps per CTA)
    const int q = warp & 3;
    const int h = (warp - 2) >> 2;                       // column half
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = pair; tile < total_tiles && ok; tile += npairs, ++tcount) {
      int mp, tcol;
      bool narrow;
      mixed_tile_coords(tile, tiles, mp, tcol, narrow);
      const int mt = 2 * mp + (int)rank;
      const bool half_only = narrow && h == 1;           // columns 128..191 of a 192-column tile
      ok = mbar_wait_cluster(accf_bar, tcount & 1, cta_abort, err_word, SITE_EPI_ACC_FULL);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + h * 128;
      uint32_t v0[32], v1[32], v2[32], v3[32];
      tmem_ld_32x32(tacc, v0);
      tmem_ld_32x32(tacc + 32, v1);
      if (!half_only) {
        tmem_ld_32x32(tacc + 64, v2);
        tmem_ld_32x32(tacc + 96, v3);
      }
      tmem_ld_wait();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(acce_bar, 0));   // accumulator is free again
      if constexpr (FMT == FMT_NVFP4) {                    // product of the two tensor scales
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          v0[j] = __float_as_uint(__uint_as_float(v0[j]) * alpha);
          v1[j] = __float_as_uint(__uint_as_float(v1[j]) * alpha);
          v2[j] = __float_as_uint(__uint_as_float(v2[j]) * alpha);
          v3[j] = __float_as_uint(__uint_as_float(v3[j]) * alpha);
        }
      }
      // Registers -> this warp's staging buffer (one 128-byte row per lane, 16-byte pieces XORed
      // with row % 8 as the 128-byte TMA swizzle expects) -> TMA store of a [32 rows x 128 B] box.
      // The store clips rows >= M and columns >= N by itself.
      const int row0 = mt * C::BM + q * 32;
      const int col0 = tcol + h * 128;
      const uint32_t stage_buf = smem_base + out_off + (uint32_t)(warp - 2) * C::OUT_WARP_BYTES;
      const uint32_t my_row = stage_buf + lane * 128;
      const uint32_t sw = (uint32_t)(lane & 7);
      auto put16 = [&](int piece, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                     ::"r"(my_row + (((uint32_t)piece ^ sw) << 4)), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
      };
      auto pack2 = [](uint32_t lo, uint32_t hi) {
        __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(lo), __uint_as_float(hi));
        return *reinterpret_cast<uint32_t*>(&hh);
      };
      auto flush = [&](int col) {                        // whole warp
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0 && row0 < M && col < N) {
          tma_store_2d(&tmY, col, row0, stage_buf);
          bulk_commit_group();
        }
      };
      auto reuse = [&]() {                               // the previous store has read the buffer
        if (lane == 0) bulk_wait_group_read<0>();
        __syncwarp();
      };
      if (y_is_bf16) {
        auto half64 = [&](const uint32_t (&lo)[32], const uint32_t (&hi)[32], int col) {
          reuse();
#pragma unroll
          for (int p = 0; p < 4; ++p)
            put16(p, pack2(lo[8 * p], lo[8 * p + 1]), pack2(lo[8 * p + 2], lo[8 * p + 3]),
                  pack2(lo[8 * p + 4], lo[8 * p + 5]), pack2(lo[8 * p + 6], lo[8 * p + 7]));
#pragma unroll
          for (int p = 0; p < 4; ++p)
            put16(4 + p, pack2(hi[8 * p], hi[8 * p + 1]), pack2(hi[8 * p + 2], hi[8 * p + 3]),
                  pack2(hi[8 * p + 4], hi[8 * p + 5]), pack2(hi[8 * p + 6], hi[8 * p + 7]));
          flush(col);
        };
        half64(v0, v1, col0);
        if (!half_only) half64(v2, v3, col0 + 64);
      } else {
        auto quarter32 = [&](const uint32_t (&v)[32], int col) {
          reuse();
#pragma unroll
          for (int p = 0; p < 8; ++p) put16(p, v[4 * p], v[4 * p + 1], v[4 * p + 2], v[4 * p + 3]);
          flush(col);
        };
        quarter32(v0, col0);
        quarter32(v1, col0 + 32);
        if (!half_only) {
          quarter32(v2, col0 + 64);
          quarter32(v3, col0 + 96);
        }
      }
    }
    if (lane == 0) bulk_wait_group_read<0>();            // shared memory must outlive the stores' reads
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before_sync();
  __syncthreads();
  if (*cta_abort) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
  }
}

}  // namespace torq
