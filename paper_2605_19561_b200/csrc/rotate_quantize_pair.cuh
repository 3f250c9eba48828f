// Rotate + quantize for M > 128 on CTA pairs: the same computation and epilogue as
// rotate_quantize_kernel, but two CTAs (a cluster of 2, one per SM) share one 256 x 256 output
// tile through tcgen05.mma cta_group::2.  Each CTA stages only its own 128 rows of X and its own
// 128 columns of R_inter per K step (32 KiB instead of 48 KiB per 128 x 256 x 64 of work), which
// is what the single-CTA kernel is short of: it cannot keep enough bytes in flight from L2 to
// feed the tensor pipe.  Every CTA loads only for itself; operand sharing happens inside the MMA, which
// reads both CTAs' shared memory.
//
// Tiles are dealt round robin from the list MixedTiles describes: 256 x 256 tiles, and where those
// would leave the last wave partly empty, 256 x 192 tiles in its place (N = 192 instructions, 96
// columns of R_inter per CTA, three 32-blocks per epilogue warp instead of four).
//
// Roles per CTA: warp 0 TMA producer (both CTAs), warp 1 MMA issuer (leader CTA only; both
// allocate tensor memory), warps 2..9 epilogue (each CTA drains its own 128 x 256 accumulator).
// Barriers: full[s] lives in the leader and counts the bytes of both CTAs' loads; empty[s] and
// acc_full[a] are local to each CTA and are signalled by the leader's tcgen05.commit to both;
// acc_empty[a] lives in the leader and takes one arrival per epilogue warp of both CTAs (16).
#pragma once
#include <cuda_bf16.h>
#include "nvfp4_quantize.cuh"
#include "mxint4_quantize.cuh"
#include "sm100_ptx.cuh"

namespace torq {

struct RotPairCfg {
  static constexpr int BN = 256;                       // tile columns (both CTAs see all of them)
  static constexpr int BM = 128;                       // rows per CTA (256 per pair)
  static constexpr int BK = 64;
  static constexpr int A_BYTES = BM * BK * 2;          // 16 KiB
  static constexpr int B_BOX_BYTES = 64 * BK * 2;      // 64(n) x 64(k) bf16 = 8 KiB
  static constexpr int B_BYTES = (BN / 2 / 64) * B_BOX_BYTES;   // this CTA's 128 columns = 16 KiB
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;         // 32 KiB
  static constexpr int STAGES = 6;
  static constexpr int RI_ROW_BYTES = 80;              // 32 bf16 + 16 B pad: conflict-free ldmatrix
  static constexpr int RI_BLOCK_BYTES = 32 * RI_ROW_BYTES;
  static constexpr int RI_BYTES = (BN / 32) * 32 * 32 * 4;     // the tile's R_intra blocks: fp32, or bf16 padded
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + RI_BYTES + 256 + 1024;
  static constexpr int NACC = 2;
  static constexpr int TMEM_COLS = 512;
  static constexpr int THREADS = 320;               // producer, MMA issuer, 8 epilogue warps
  static_assert(SMEM_BYTES <= 232448, "shared memory budget");
};

// FMT_NVFP4: the same kernel with the NVFP4 quantizer in the epilogue (two 16-element blocks per
// 32 columns, E4M3 scales, `tensor_scale` the tensor's float32 scale; unused for MXFP4).  R_intra
// is still [d/32, 32, 32]; 16-wide rotations arrive as its block-diagonal form.
// FMT_MXINT4: integer codes written as one E4M3 operand byte per element (`codes` is [M, d] bytes),
// the scale bytes as for MXFP4.
// FMT_F32OUT: no quantizer; `codes` is a float32 [M, d] array that receives Z itself (`scales` unused).
// `x_terms` > 1: X is the sum of that many bfloat16 matrices stored side by side, tmX = [M, x_terms * d]
// (an fp32 matrix split exactly into three bf16 terms); the contraction then runs over all of them
// against the same R_inter, i.e. Z = (X_0 + X_1 + ...) R_inter in one fp32 accumulation.  d % 64 == 0 then.
template <int FMT = FMT_MXFP4>
__global__ void __launch_bounds__(320, 1)
rotate_quantize_pair_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmR,
                            const __grid_constant__ CUtensorMap tmRn, const __nv_bfloat16* __restrict__ R_intra, uint8_t* __restrict__ codes,
                            uint8_t* __restrict__ scales, int M, int d, float tensor_scale, int x_terms,
                            const MixedTiles tiles, int* err_word) {
  using C = RotPairCfg;
  constexpr int BN = C::BN;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  uint8_t* ri_smem = smem_gen + C::STAGES * C::STAGE_BYTES;
  const uint32_t bar_off = C::STAGES * C::STAGE_BYTES + C::RI_BYTES;
  const uint32_t bar_base = smem_base + bar_off;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (C::STAGES + s); };
  auto accf_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + a); };
  auto acce_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + C::NACC + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + bar_off + 192);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(smem_gen + bar_off + 200);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();             // 0 = leader
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int m_tiles = (M + 127) / 128;                 // 128-row tiles that exist
  const int total_tiles = tiles.total;                 // 256-row pair tiles, 256 or 192 columns wide
  const int kr_tiles = (d + C::BK - 1) / C::BK;         // K steps over R_inter; X has x_terms times as many
  const int k_tiles = kr_tiles * x_terms;
  const int nblocks = d / 32;
  const int kb4 = (nblocks + 3) / 4;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < C::NACC; ++a) { mbar_init(accf_bar(a), 1); mbar_init(acce_bar(a), 16); }
    *cta_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::TMEM_COLS); tmem_relinquish_pair(); }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_after_init();                                  // both CTAs' barriers exist before any remote arrive
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // Set-up above touched no global memory; from here on the previous kernel's results are needed.
  // R_inter is a constant of the layer, never the output of the kernel that runs just before this
  // one: the producer starts the first stages' R_inter loads right away; the X loads and all
  // other global accesses wait until that kernel has completed.
  griddep_launch_dependents();
  const int pre = pair < total_tiles ? (k_tiles < C::STAGES ? k_tiles : C::STAGES) : 0;
  if (warp == 0) {
    if (elect_one()) {
      tma_prefetch_desc(&tmX);
      tma_prefetch_desc(&tmR);
      int mp0 = 0, col0 = 0;
      bool narrow = false;
      if (pre > 0) mixed_tile_coords(pair, tiles, mp0, col0, narrow);
      (void)mp0;
      const int my_col = col0 + (int)rank * (narrow ? kNarrowCols / 2 : BN / 2);
      if (narrow) tma_prefetch_desc(&tmRn);
      for (int kt = 0; kt < pre; ++kt) {
        const uint32_t st = smem_base + kt * C::STAGE_BYTES;
        const uint32_t leader_full = map_to_cta(full_bar(kt), 0);
        if (rank == 0) mbar_arrive_expect_tx(full_bar(kt), 2 * (C::STAGE_BYTES - (narrow ? C::B_BOX_BYTES / 2 : 0)));
        tma_load_2d_pair(st + C::A_BYTES, &tmR, my_col, (kt % kr_tiles) * C::BK, leader_full);
        tma_load_2d_pair(st + C::A_BYTES + C::B_BOX_BYTES, narrow ? &tmRn : &tmR, my_col + 64, (kt % kr_tiles) * C::BK,
                         leader_full);
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
      // A 192-column tile takes 96 columns of R_inter per CTA: one 64-column box and one 32-column box.
      // Under the 128-byte swizzle a box whose rows are 64 bytes long still lands on a 128-byte pitch, i.e.
      // as the first half of the 64-column layout the instruction's descriptor describes.
      const int my_col = tcol + (int)rank * (narrow ? kNarrowCols / 2 : BN / 2);
      const uint32_t stage_tx = 2 * (C::STAGE_BYTES - (narrow ? C::B_BOX_BYTES / 2 : 0));
      for (int kt = 0, kr = 0; kt < k_tiles; ++kt, ++it, kr = (kr + 1 == kr_tiles ? 0 : kr + 1)) {
        const int s = it % C::STAGES;
        if (!mbar_wait_cluster_warp(empty_bar(s), ((it / C::STAGES) & 1) ^ 1, cta_abort, err_word,
                               SITE_PRODUCER_EMPTY)) { ok = false; break; }
        const uint32_t st = smem_base + s * C::STAGE_BYTES;
        const uint32_t leader_full = map_to_cta(full_bar(s), 0);
        if (elect_one()) {
          const bool r_issued = it < (uint32_t)pre;      // R side of this stage went out before the wait above
          if (rank == 0 && !r_issued) mbar_arrive_expect_tx(full_bar(s), stage_tx);
          tma_load_2d_pair(st, &tmX, kt * C::BK, mt * C::BM, leader_full);
          if (!r_issued) {
            tma_load_2d_pair(st + C::A_BYTES, &tmR, my_col, kr * C::BK, leader_full);
            tma_load_2d_pair(st + C::A_BYTES + C::B_BOX_BYTES, narrow ? &tmRn : &tmR, my_col + 64, kr * C::BK, leader_full);
          }
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    if (rank == 0) {
      constexpr uint32_t idesc_wide = idesc_bf16(256, BN, /*A MN-major*/ false, /*B MN-major*/ true);
      constexpr uint32_t idesc_narrow = idesc_bf16(256, kNarrowCols, false, true);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = pair; tile < total_tiles && ok; tile += npairs, ++tcount) {
        int mp, tcol;
        bool narrow;
        mixed_tile_coords(tile, tiles, mp, tcol, narrow);
        (void)mp; (void)tcol;
        const uint32_t idesc = narrow ? idesc_narrow : idesc_wide;
        const int a = tcount % C::NACC;
        if (!mbar_wait_cluster_warp(acce_bar(a), ((tcount / C::NACC) & 1) ^ 1, cta_abort, err_word,
                               SITE_MMA_ACC_EMPTY)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t acc = tmem_base + a * BN;
        for (int kt = 0; kt < k_tiles; ++kt, ++it) {
          const int s = it % C::STAGES;
          if (!mbar_wait_cluster_warp(full_bar(s), (it / C::STAGES) & 1, cta_abort, err_word, SITE_MMA_FULL)) {
            ok = false; break;
          }
          tc_fence_after_sync();
          const uint32_t st = smem_base + s * C::STAGE_BYTES;
          const uint64_t adesc = make_desc(st, 16, 1024, kSwizzle128);
          const uint64_t bdesc = make_desc(st + C::A_BYTES, C::B_BOX_BYTES, 1024, kSwizzle128);
          if (elect_one()) {
#pragma unroll
            for (int j = 0; j < C::BK / 16; ++j)
              mma_bf16_pair(acc, adesc + 2 * j, bdesc + 128 * j, idesc, (kt | j) != 0);
            tc_commit_pair(empty_bar(s), 3);             // stage free in both CTAs
          }
          __syncwarp();
        }
        if (ok && elect_one()) tc_commit_pair(accf_bar(a), 3);   // accumulator ready in both CTAs
        __syncwarp();
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (8 warps per CTA)
    // warp w reads lane quarter w % 4 (32 rows) and column half (w - 2) / 4 (four 32-blocks = one
    // 4-byte group of scale bytes; three blocks in a 192-column tile).  Two forms of the intra-block rotation:
    //  * fp32 FMAs, one row per thread, R_intra broadcast from shared memory as fp32.  Bound by
    //    that broadcast (8 bytes per lane and cycle): about 3/4 of a mainloop per tile, which does
    //    not matter while the next tile's mainloop runs beside it on the tensor pipe.
    //  * warp-level tensor-core MMAs on the accumulator fragment layout (y split into three bf16
    //    terms, R_intra exact in bf16, fp32 accumulation): half the time when the tensor pipe is
    //    otherwise idle, but it fights the mainloop when both run.  Used for the CTA's LAST tile,
    //    whose epilogue nothing overlaps.
    const int q = warp & 3;
    const int h = (warp - 2) >> 2;
    const int et = (warp - 2) * 32 + lane;               // 0..255 among the epilogue threads
    const int p = lane & 3, r8 = lane >> 2;
    const uint32_t ri_saddr = smem_u32(ri_smem);
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = pair; tile < total_tiles; tile += npairs, ++tcount) {
      int mp, tcol;
      bool narrow;
      mixed_tile_coords(tile, tiles, mp, tcol, narrow);
      const int mt = 2 * mp + (int)rank;
      const int a = tcount % C::NACC;
      const int b0 = tcol >> 5;                          // first 32-block of the tile: even, 2 mod 4 for some narrow tiles
      const int nbb = narrow ? 3 : 4;                    // this warp's blocks: half of the tile's 8 or 6
      const bool last = FMT != FMT_F32OUT && tile + npairs >= total_tiles;
      if (R_intra != nullptr) {
        // Executed by every epilogue thread for every tile, also after a wait has given up.
        named_barrier_sync(1, 256);
        for (int idx = et * 8; ok && idx < (BN / 32) * 1024; idx += 256 * 8) {
          const int lb = idx >> 10, blk = b0 + lb;
          if (last) {                                    // bf16 rows of 80 bytes: conflict-free ldmatrix
            const int i = (idx & 1023) >> 5, c = idx & 31;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (blk < nblocks) v = __ldg(reinterpret_cast<const uint4*>(R_intra + (size_t)blk * 1024 + (idx & 1023)));
            *reinterpret_cast<uint4*>(ri_smem + lb * C::RI_BLOCK_BYTES + i * C::RI_ROW_BYTES + c * 2) = v;
          } else {                                       // fp32, dense
            float v[8];
            if (blk < nblocks) load8(R_intra + (size_t)blk * 1024 + (idx & 1023), v);
            else {
#pragma unroll
              for (int i = 0; i < 8; ++i) v[i] = 0.f;
            }
            float* dst = reinterpret_cast<float*>(ri_smem) + idx;
            *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
            *reinterpret_cast<float4*>(dst + 4) = make_float4(v[4], v[5], v[6], v[7]);
          }
        }
        named_barrier_sync(1, 256);
      }
      if (ok) ok = mbar_wait_cluster(accf_bar(a), (tcount / C::NACC) & 1, cta_abort, err_word, SITE_EPI_ACC_FULL);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) continue;
      tc_fence_after_sync();
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + a * BN + h * nbb * 32;
      // Scale bytes: block blk of row r sits in byte blk % 4 of the 4-byte cell of (r, blk / 4).  The four
      // bytes of a wide tile's half are one cell; the three of a narrow tile's half go out one by one.
      const int fb = b0 + h * nbb;
      auto put_scales = [&](uint32_t w, size_t in_tile) {  // byte bb of w = scale of block fb + bb
        if (nbb == 4) {
          if ((fb >> 2) < kb4) *reinterpret_cast<uint32_t*>(scales + ((size_t)mt * kb4 + (fb >> 2)) * 512 + in_tile) = w;
        } else {
          for (int j = 0; j < nbb; ++j) {
            const int blk = fb + j;
            if ((blk >> 2) < kb4) scales[((size_t)mt * kb4 + (blk >> 2)) * 512 + in_tile + (blk & 3)] = (uint8_t)(w >> (8 * j));
          }
        }
      };
      // NVFP4: two bytes per block, cells of two blocks
      auto put_scales16 = [&](uint32_t w01, uint32_t w23, size_t in_tile, int kb4n) {
        if (nbb == 4) {
          if ((fb >> 1) < kb4n) *reinterpret_cast<uint32_t*>(scales + ((size_t)mt * kb4n + (fb >> 1)) * 512 + in_tile) = w01;
          if ((fb >> 1) + 1 < kb4n)
            *reinterpret_cast<uint32_t*>(scales + ((size_t)mt * kb4n + (fb >> 1) + 1) * 512 + in_tile) = w23;
        } else {
          for (int j = 0; j < nbb; ++j) {
            const int blk = fb + j;
            if ((blk >> 1) < kb4n)
              *reinterpret_cast<uint16_t*>(scales + ((size_t)mt * kb4n + (blk >> 1)) * 512 + in_tile + 2 * (blk & 1)) =
                  (uint16_t)((j < 2 ? w01 : w23) >> (16 * (j & 1)));
          }
        }
      };
      if (!last) {
        // ---- one row per thread, fp32 FMAs
        const int64_t row = (int64_t)mt * C::BM + q * 32 + lane;
        uint32_t sc_word = 0, sc_word2 = 0;              // NVFP4: two groups of four 16-blocks
        NvScale nvs = {};
        if constexpr (FMT == FMT_NVFP4) nvs = nv_scale(tensor_scale);
#pragma unroll 1
        for (int bb = 0; bb < nbb; ++bb) {
          uint32_t yv[32];
          tmem_ld_32x32(tacc + bb * 32, yv);
          tmem_ld_wait();
          if (bb == nbb - 1) {                           // this warp's share is read: tell the leader
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(acce_bar(a), 0));
          }
          float z[32];
          if (R_intra != nullptr) {
            intra_rotate32(yv, ri_saddr + (uint32_t)(h * nbb + bb) * 4096, z);
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) z[j] = __uint_as_float(yv[j]);
          }
          const int blk = fb + bb;
          if constexpr (FMT == FMT_F32OUT) {               // the rotated values themselves
            if (row < M && blk < nblocks) {
              float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(codes) + row * (int64_t)d + (int64_t)blk * 32);
#pragma unroll
              for (int j = 0; j < 8; ++j) dst[j] = make_float4(z[4 * j], z[4 * j + 1], z[4 * j + 2], z[4 * j + 3]);
            }
            continue;
          }
          uint4 cw;
          uint32_t sbyte;
          if constexpr (FMT == FMT_MXINT4) {               // one operand byte per element
            uint4 cw2;
            mxint4_quantize_block32(z, cw, cw2, sbyte);
            if (row < M && blk < nblocks) {
              uint4* dst = reinterpret_cast<uint4*>(codes + row * (int64_t)d + (int64_t)blk * 32);
              dst[0] = cw;
              dst[1] = cw2;
            }
          } else {
            if constexpr (FMT == FMT_NVFP4) nv_quantize_2x16(z, nvs, cw, sbyte);
            else quantize_block32(z, cw, sbyte);
            if (row < M && blk < nblocks)
              *reinterpret_cast<uint4*>(codes + row * (int64_t)(d / 2) + (int64_t)blk * 16) = cw;
          }
          if constexpr (FMT == FMT_NVFP4) {
            if (blk >= nblocks) sbyte = 0;               // padding blocks decode to zero
            if (bb < 2) sc_word |= sbyte << (16 * bb);
            else sc_word2 |= sbyte << (16 * (bb - 2));
          } else {
            sc_word |= sbyte << (8 * bb);
          }
        }
        if constexpr (FMT == FMT_F32OUT) {
          continue;
        } else if constexpr (FMT == FMT_NVFP4) {
          const int kb4n = (2 * nblocks + 3) / 4;        // 4-byte groups of 16-block scales per row: blocks fb, fb + 1
          if (mt < m_tiles) put_scales16(sc_word, sc_word2, (size_t)lane * 16 + q * 4, kb4n);
        } else {
          if (mt < m_tiles) put_scales(sc_word, (size_t)lane * 16 + q * 4);   // the pair's second row tile may not exist
        }
        continue;
      }
      // ---- accumulator fragment layout (16 rows at a time): thread t holds rows t/4 and t/4 + 8,
      //      eight columns of each per block
      const int64_t row_base = (int64_t)mt * C::BM + q * 32 + r8;     // + 16 mh + 8 rh
      uint32_t sc_word[4] = {0u, 0u, 0u, 0u};            // rows r8 + 16 mh + 8 rh -> index 2 mh + rh
      uint32_t sc_hi[4] = {0u, 0u, 0u, 0u};              // NVFP4: second group of four 16-blocks
      NvScale nvs = {};
      if constexpr (FMT == FMT_NVFP4) nvs = nv_scale(tensor_scale);
#pragma unroll 1
      for (int bb = 0; bb < nbb; ++bb) {
        const int blk = fb + bb;
        uint32_t bfrag[2][4][2];                         // [k chunk][n tile][2]
        if (R_intra != nullptr) {
          // lane l: row l % 8 of matrix l / 8; matrices (k 0-7, n), (k 8-15, n), (k 0-7, n+8), (k 8-15, n+8)
          const uint32_t rb = ri_saddr + (uint32_t)(h * nbb + bb) * C::RI_BLOCK_BYTES +
                              (uint32_t)(((lane >> 3) & 1) * 8 + (lane & 7)) * C::RI_ROW_BYTES +
                              (uint32_t)(lane >> 4) * 16;
#pragma unroll
          for (int kc = 0; kc < 2; ++kc)
#pragma unroll
            for (int np = 0; np < 2; ++np)
              ldmatrix_x4_trans(rb + kc * 16 * C::RI_ROW_BYTES + np * 32, bfrag[kc][2 * np][0], bfrag[kc][2 * np][1],
                                bfrag[kc][2 * np + 1][0], bfrag[kc][2 * np + 1][1]);
        }
#pragma unroll
        for (int mh = 0; mh < 2; ++mh) {
          uint32_t y[16];
          tmem_ld_16x256b_x4(tacc + ((uint32_t)(16 * mh) << 16) + bb * 32, y);
          tmem_ld_wait();
          if (bb == nbb - 1 && mh == 1) {                // this warp's share is read: tell the leader
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(acce_bar(a), 0));
          }
          float acc[4][4];
          if (R_intra != nullptr) {
            uint32_t ah[8], am[8], al[8];                // A fragments: [k chunk * 4 + (n & 1) * 2 + row half]
#pragma unroll
            for (int n = 0; n < 4; ++n)
#pragma unroll
              for (int rh = 0; rh < 2; ++rh) {
                const int ai = (n >> 1) * 4 + (n & 1) * 2 + rh;
                split3_bf16x2(y[4 * n + 2 * rh], y[4 * n + 2 * rh + 1], ah[ai], am[ai], al[ai]);
              }
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
          } else {
#pragma unroll
            for (int n = 0; n < 4; ++n)
#pragma unroll
              for (int e = 0; e < 4; ++e) acc[n][e] = __uint_as_float(y[4 * n + e]);
          }
#pragma unroll
          for (int rh = 0; rh < 2; ++rh) {
            const float v[8] = {acc[0][2 * rh], acc[0][2 * rh + 1], acc[1][2 * rh], acc[1][2 * rh + 1],
                                acc[2][2 * rh], acc[2][2 * rh + 1], acc[3][2 * rh], acc[3][2 * rh + 1]};
            uint32_t word, sbyte;
            const int64_t row = row_base + 16 * mh + 8 * rh;
            if constexpr (FMT == FMT_MXINT4) {             // two operand bytes per 8 columns and lane
              uint32_t pr[4];
              mxint4_quantize_row_fragment(v, pr, sbyte);
              if (row < M && blk < nblocks) {
                uint8_t* dst = codes + row * (int64_t)d + (int64_t)blk * 32 + 2 * p;
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) *reinterpret_cast<uint16_t*>(dst + 8 * nt) = (uint16_t)pr[nt];
              }
            } else {
              if constexpr (FMT == FMT_NVFP4) nv_quantize_row_fragment(v, p, nvs, word, sbyte);
              else quantize_row_fragment(v, p, word, sbyte);
              if (row < M && blk < nblocks)
                *reinterpret_cast<uint32_t*>(codes + row * (int64_t)(d / 2) + (int64_t)blk * 16 + 4 * p) = word;
            }
            if constexpr (FMT == FMT_NVFP4) {
              if (blk >= nblocks) sbyte = 0;
              if (bb < 2) sc_word[2 * mh + rh] |= sbyte << (16 * bb);
              else sc_hi[2 * mh + rh] |= sbyte << (16 * (bb - 2));
            } else {
              sc_word[2 * mh + rh] |= sbyte << (8 * bb);
            }
          }
        }
      }
      if constexpr (FMT == FMT_NVFP4) {
        const int kb4n = (2 * nblocks + 3) / 4;
        if (p == 0 && mt < m_tiles) {
#pragma unroll
          for (int rs = 0; rs < 4; ++rs) {
            put_scales16(sc_word[rs], sc_hi[rs], (size_t)(r8 + 16 * (rs >> 1) + 8 * (rs & 1)) * 16 + q * 4, kb4n);
          }
        }
      } else if (p == 0 && mt < m_tiles) {               // the pair's second row tile may not exist
#pragma unroll
        for (int rs = 0; rs < 4; ++rs)
          put_scales(sc_word[rs], (size_t)(r8 + 16 * (rs >> 1) + 8 * (rs & 1)) * 16 + q * 4);
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before_sync();
  __syncthreads();
  if (*cta_abort) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  cluster_sync_all();                                  // the peer no longer touches this CTA's memory
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
  }
}

}  // namespace torq
