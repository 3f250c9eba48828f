// Algorithm 3 steps 1-5 in ONE persistent kernel on CTA pairs (M > 128, MXFP4): the tile loops of
// rotate_quantize_pair_kernel and of mxfp4_gemm_pair_kernel run back to back inside every CTA pair,
// so that pairs which run out of rotation tiles start on GEMM tiles instead of idling until the
// rotation kernel's last wave has drained (at 2048 x 4096 -> 6144: 128 rotation tiles on 74 pairs
// leave 20 pairs idle for a whole tile, 22 us, and the GEMM's 192 tiles need three waves).
//
// What makes that legal:
//   * the rotation walks its tiles row tile by row tile, and every epilogue warp, once its share of
//     a tile's codes and scales is in global memory, adds one to the tile row's counter (release);
//   * the producer of a GEMM tile waits (bounded) until the counter of its row tile shows all
//     16 x (column tiles) arrivals (acquire), then loads the activations' codes and scales with TMA;
//   * a pair only ever waits for rotation tiles, which wait for nothing, and every pair works
//     through its own rotation tiles first: no cycle.  All CTAs must be resident (the grid never
//     exceeds the number of CTA pairs that fit, and the launch is cooperative).
// Between the two loops each role passes a hand-over: the GEMM's loads reuse the rotation's
// shared-memory stages and its scale factors the second rotation accumulator in tensor memory, so
// the GEMM producer waits for the rotation's last MMAs and the GEMM issuer for the rotation's last
// accumulator reads.
//
// GEMM tiles are dealt out by a closed rule, not a queue.  With P pairs and the rotation's last
// wave only partly filled, the P0 pairs without a tile in that wave take `early` GEMM tiles each
// from the rows that are complete before that wave; all other GEMM tiles go round-robin over all
// pairs, row tile by row tile.
#pragma once
#include <cuda_bf16.h>
#include "mxfp4_gemm_pair.cuh"
#include "rotate_quantize_pair.cuh"
#include "sm100_ptx.cuh"

namespace torq {

struct FusedCfg {
  using R = RotPairCfg;
  using G = GemmPairCfg;
  static constexpr int R_ARENA = R::STAGES * R::STAGE_BYTES + R::RI_BYTES;
  static constexpr int G_ARENA = G::STAGES * G::STAGE_BYTES + G::OUT_BYTES;
  static constexpr int ARENA = R_ARENA > G_ARENA ? R_ARENA : G_ARENA;
  static constexpr int BAR_BYTES = 512;
  static constexpr int SMEM_BYTES = ARENA + BAR_BYTES + 1024;
  static constexpr int THREADS = 320;
  static constexpr int TMEM_COLS = 512;
  static constexpr int ARRIVALS_PER_TILE = 16;         // 8 epilogue warps in each of the two CTAs
  static_assert(SMEM_BYTES <= 232448, "shared memory budget");
};

// The GEMM tile (row-major index) that pair `pair` takes as its i-th, or -1 when it has no i-th.
struct FusedSchedule {
  int P, P1, P0, early, Ge, total_g;
  __device__ __forceinline__ int tile(int pair, int i) const {
    const bool is_early = pair >= P1;                  // pairs P1 .. P-1 have no tile in the rotation's last wave
    int first_rr = 0;                                  // how many of the pair's tiles come from the early share
    if (is_early && P0 > 0) {
      const int e = pair - P1;
      // early tiles e, e + P0, e + 2 P0, ... below Ge
      const int mine = e < Ge ? (Ge - 1 - e) / P0 + 1 : 0;
      if (i < mine) return e + i * P0;
      first_rr = mine;
    }
    const int g = Ge + pair + (i - first_rr) * P;
    return g < total_g ? g : -1;
  }
};

__device__ __forceinline__ FusedSchedule fused_schedule(int P, int total_r, int n_tiles_r, int n_tiles_g,
                                                        int total_g, int early) {
  FusedSchedule s;
  s.P = P;
  s.total_g = total_g;
  s.early = early;
  const int nr_max = (total_r + P - 1) / P;            // rotation tiles of the busiest pairs
  const int last = total_r - (nr_max - 1) * P;         // tiles in the last wave
  s.P1 = last;                                         // pairs 0 .. P1-1 work in the last wave
  s.P0 = P - last;
  const int rows_ready = ((nr_max - 1) * P) / n_tiles_r;   // row tiles complete before the last wave
  const int ready = rows_ready * n_tiles_g;
  const int want = s.P0 * early;
  s.Ge = s.P0 > 0 ? (ready < want ? ready : want) : 0;
  if (s.Ge > total_g) s.Ge = total_g;
  return s;
}

// Bounded wait until *counter >= target (acquire at device scope).  Same limits and error latch as the
// barrier waits.
__device__ __forceinline__ bool wait_counter(const int* counter, int target, volatile int* cta_abort,
                                             int* err_word, int site) {
  unsigned long long t0 = 0;
  for (uint32_t it = 1;; ++it) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
    if (v >= target) return true;
    if ((it & 0xFFu) == 0) {
      if (*cta_abort) return false;
      unsigned long long now = globaltimer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) {
        *cta_abort = 1;
        atomicCAS(err_word, 0, kErrTimeout | (site << 8));
        return false;
      }
    }
  }
}

// tmX, tmR: rotation operands (as rotate_quantize_pair_kernel).  codes / scales: where the rotation
// writes (the caller's workspace); tmA / tmSFA read the same memory for the GEMM; tmB, tmSFB, tmY as
// mxfp4_gemm_pair_kernel.  row_done: one zeroed int per 256-row tile.
__global__ void __launch_bounds__(320, 1)
rotated_linear_pair_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmR,
                           const __nv_bfloat16* __restrict__ R_intra, uint8_t* __restrict__ codes,
                           uint8_t* __restrict__ scales, const __grid_constant__ CUtensorMap tmA,
                           const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmSFA,
                           const __grid_constant__ CUtensorMap tmSFB, const __grid_constant__ CUtensorMap tmY,
                           int y_is_bf16, int M, int d, int N, int* __restrict__ row_done, int early,
                           int* err_word) {
  using C = FusedCfg;
  using RC = RotPairCfg;
  using GC = GemmPairCfg;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + C::ARENA;
  // barrier map (8 bytes each): rotation full[6] empty[6] acc_full[2] acc_empty[2], GEMM full[5] empty[5]
  // acc_full acc_empty, hand-over
  auto r_full = [&](int s) { return bar_base + 8u * s; };
  auto r_empty = [&](int s) { return bar_base + 8u * (6 + s); };
  auto r_accf = [&](int a) { return bar_base + 8u * (12 + a); };
  auto r_acce = [&](int a) { return bar_base + 8u * (14 + a); };
  auto g_full = [&](int s) { return bar_base + 8u * (16 + s); };
  auto g_empty = [&](int s) { return bar_base + 8u * (21 + s); };
  const uint32_t g_accf = bar_base + 8u * 26, g_acce = bar_base + 8u * 27;
  const uint32_t handover_bar = bar_base + 8u * 28;    // the rotation's last MMAs are complete (both CTAs)
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + C::ARENA + 400);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(smem_gen + C::ARENA + 408);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int m_tiles = (M + 127) / 128;
  const int mp_tiles = (M + 255) / 256;
  // rotation geometry
  const int n_tiles_r = (d + RC::BN - 1) / RC::BN;
  const int total_r = mp_tiles * n_tiles_r;
  const int k_tiles_r = (d + RC::BK - 1) / RC::BK;
  const int nblocks = d / 32;
  const int kb4_r = (nblocks + 3) / 4;
  // GEMM geometry (K = d)
  const int n_tiles_g = (N + GC::BN - 1) / GC::BN;
  const int total_g = mp_tiles * n_tiles_g;
  const int k_tiles_g = (d + GC::BK - 1) / GC::BK;
  const int kb4_g = d / 128;
  const FusedSchedule sched = fused_schedule(npairs, total_r, n_tiles_r, n_tiles_g, total_g, early);
  const int my_r = pair < total_r ? (total_r - 1 - pair) / npairs + 1 : 0;     // this pair's rotation tiles
  const int row_target = C::ARRIVALS_PER_TILE * n_tiles_r;

  if (threadIdx.x == 0) {
    for (int s = 0; s < RC::STAGES; ++s) { mbar_init(r_full(s), 1); mbar_init(r_empty(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(r_accf(a), 1); mbar_init(r_acce(a), 16); }
    for (int s = 0; s < GC::STAGES; ++s) { mbar_init(g_full(s), 1); mbar_init(g_empty(s), 1); }
    mbar_init(g_accf, 1);
    mbar_init(g_acce, 16);
    mbar_init(handover_bar, 1);
    *cta_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::TMEM_COLS); tmem_relinquish_pair(); }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_after_init();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ================================================================== TMA producer (both CTAs)
    if (elect_one()) {
      tma_prefetch_desc(&tmX); tma_prefetch_desc(&tmR); tma_prefetch_desc(&tmA); tma_prefetch_desc(&tmB);
      tma_prefetch_desc(&tmSFA); tma_prefetch_desc(&tmSFB);
    }
    bool ok = true;
    // ---- rotation tiles, row tile by row tile
    uint32_t it = 0;
    for (int i = 0; i < my_r && ok; ++i) {
      const int t = pair + i * npairs;
      const int mp = t / n_tiles_r, nt = t - mp * n_tiles_r;
      const int mt = 2 * mp + (int)rank;
      for (int kt = 0; kt < k_tiles_r; ++kt, ++it) {
        const int s = it % RC::STAGES;
        if (!mbar_wait_cluster_warp(r_empty(s), ((it / RC::STAGES) & 1) ^ 1, cta_abort, err_word,
                                    SITE_PRODUCER_EMPTY)) { ok = false; break; }
        const uint32_t st = smem_base + s * RC::STAGE_BYTES;
        const uint32_t leader_full = map_to_cta(r_full(s), 0);
        if (elect_one()) {
          if (rank == 0) mbar_arrive_expect_tx(r_full(s), 2 * RC::STAGE_BYTES);
          tma_load_2d_pair(st, &tmX, kt * RC::BK, mt * RC::BM, leader_full);
#pragma unroll
          for (int b = 0; b < RC::BN / 2 / 64; ++b)
            tma_load_2d_pair(st + RC::A_BYTES + b * RC::B_BOX_BYTES, &tmR,
                             nt * RC::BN + (int)rank * (RC::BN / 2) + b * 64, kt * RC::BK, leader_full);
        }
        __syncwarp();
      }
    }
    // ---- hand-over: the GEMM stages lie over the rotation's; its last MMAs must have read them
    if (ok) ok = mbar_wait_cluster_warp(handover_bar, 0, cta_abort, err_word, SITE_PRODUCER_EMPTY);
    // ---- GEMM tiles
    it = 0;
    for (int i = 0; ok; ++i) {
      const int g = sched.tile(pair, i);
      if (g < 0) break;
      const int mp = g / n_tiles_g, nt = g - mp * n_tiles_g;
      const int mt = 2 * mp + (int)rank;
      // the activations of this row tile: every epilogue warp of every rotation tile of the row has arrived
      bool ready = true;
      if (lane == 0) ready = wait_counter(row_done + mp, row_target, cta_abort, err_word, SITE_PRODUCER_EMPTY);
      ready = __shfl_sync(0xFFFFFFFFu, (int)ready, 0) != 0;
      if (!ready) { ok = false; break; }
      fence_proxy_async_all();                           // their plain stores, before this thread's TMA reads
      for (int kt = 0; kt < k_tiles_g; ++kt, ++it) {
        const int s = it % GC::STAGES;
        if (!mbar_wait_cluster_warp(g_empty(s), ((it / GC::STAGES) & 1) ^ 1, cta_abort, err_word,
                                    SITE_PRODUCER_EMPTY)) { ok = false; break; }
        const uint32_t st = smem_base + s * GC::STAGE_BYTES;
        const uint32_t leader_full = map_to_cta(g_full(s), 0);
        if (elect_one()) {
          if (rank == 0) mbar_arrive_expect_tx(g_full(s), 2 * GC::STAGE_BYTES);
          tma_load_2d_pair(st, &tmA, kt * 128, mt * GC::BM, leader_full);
          tma_load_2d_pair(st + GC::A_BYTES, &tmB, kt * 128, nt * GC::BN + (int)rank * (GC::BN / 2), leader_full);
          tma_load_2d_pair(st + GC::A_BYTES + GC::B_BYTES, &tmSFA, kt * 256, mt, leader_full);
          tma_load_2d_pair(st + GC::A_BYTES + GC::B_BYTES + GC::SFA_BYTES, &tmSFB, kt * 256, 2 * nt, leader_full);
          tma_load_2d_pair(st + GC::A_BYTES + GC::B_BYTES + GC::SFA_BYTES + 1024, &tmSFB, kt * 256, 2 * nt + 1,
                           leader_full);
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    // ================================================================== MMA issuer (leader only)
    if (rank == 0) {
      bool ok = true;
      // ---- rotation
      {
        constexpr uint32_t idesc = idesc_bf16(256, RC::BN, /*A MN-major*/ false, /*B MN-major*/ true);
        uint32_t it = 0;
        for (int i = 0; i < my_r && ok; ++i) {
          const int a = i & 1;
          if (!mbar_wait_cluster_warp(r_acce(a), ((i >> 1) & 1) ^ 1, cta_abort, err_word, SITE_MMA_ACC_EMPTY)) {
            ok = false; break;
          }
          tc_fence_after_sync();
          const uint32_t acc = tmem_base + a * RC::BN;
          for (int kt = 0; kt < k_tiles_r; ++kt, ++it) {
            const int s = it % RC::STAGES;
            if (!mbar_wait_cluster_warp(r_full(s), (it / RC::STAGES) & 1, cta_abort, err_word, SITE_MMA_FULL)) {
              ok = false; break;
            }
            tc_fence_after_sync();
            const uint32_t st = smem_base + s * RC::STAGE_BYTES;
            const uint64_t adesc = make_desc(st, 16, 1024, kSwizzle128);
            const uint64_t bdesc = make_desc(st + RC::A_BYTES, RC::B_BOX_BYTES, 1024, kSwizzle128);
            if (elect_one()) {
#pragma unroll
              for (int j = 0; j < RC::BK / 16; ++j)
                mma_bf16_pair(acc, adesc + 2 * j, bdesc + 128 * j, idesc, (kt | j) != 0);
              tc_commit_pair(r_empty(s), 3);
            }
            __syncwarp();
          }
          if (ok && elect_one()) tc_commit_pair(r_accf(a), 3);
          __syncwarp();
        }
      }
      // ---- hand-over: tell both producers once every rotation MMA has completed; the GEMM's scale
      //      factors go into the columns of the second rotation accumulator, so its last reader must be done
      if (elect_one()) tc_commit_pair(handover_bar, 3);
      __syncwarp();
      if (ok && my_r >= 1) {
        // the accumulator buffers last used by tiles my_r - 1 and (if any) my_r - 2 have been read
        for (int back = 1; back <= 2 && back <= my_r && ok; ++back) {
          const int i = my_r - back;
          ok = mbar_wait_cluster_warp(r_acce(i & 1), (i >> 1) & 1, cta_abort, err_word, SITE_MMA_ACC_EMPTY);
        }
        tc_fence_after_sync();
      }
      // ---- GEMM
      {
        constexpr uint32_t idesc0 = idesc_mxf4(256, GC::BN, 0, 0), idesc2 = idesc_mxf4(256, GC::BN, 2, 2);
        const uint32_t sfa_t = tmem_base + GC::SFA_COL, sfb_t = tmem_base + GC::SFB_COL;
        uint32_t it = 0, tcount = 0;
        for (int i = 0; ok; ++i, ++tcount) {
          if (sched.tile(pair, i) < 0) break;
          if (!mbar_wait_cluster_warp(g_acce, (tcount & 1) ^ 1, cta_abort, err_word, SITE_MMA_ACC_EMPTY)) {
            ok = false; break;
          }
          tc_fence_after_sync();
          for (int kt = 0; kt < k_tiles_g; ++kt, ++it) {
            const int s = it % GC::STAGES;
            if (!mbar_wait_cluster_warp(g_full(s), (it / GC::STAGES) & 1, cta_abort, err_word, SITE_MMA_FULL)) {
              ok = false; break;
            }
            tc_fence_after_sync();
            const bool two = (kb4_g - 2 * kt) >= 2;        // K % 256 == 128: the last stage is half
            const uint32_t st = smem_base + s * GC::STAGE_BYTES;
            const uint64_t adesc = make_desc(st, 16, 1024, kSwizzle128);
            const uint64_t bdesc = make_desc(st + GC::A_BYTES, 16, 1024, kSwizzle128);
            const uint64_t sfa_d = make_desc(st + GC::A_BYTES + GC::B_BYTES, 0, 128, 0);
            const uint64_t sfb_d = make_desc(st + GC::A_BYTES + GC::B_BYTES + GC::SFA_BYTES, 0, 128, 0);
            if (elect_one()) {
              tmem_cp_32x128b_warpx4_pair(sfa_t, sfa_d);
              tmem_cp_32x128b_warpx4_pair(sfb_t, sfb_d);
              tmem_cp_32x128b_warpx4_pair(sfb_t + 4, sfb_d + 64);
              if (two) {
                tmem_cp_32x128b_warpx4_pair(sfa_t + 4, sfa_d + 32);
                tmem_cp_32x128b_warpx4_pair(sfb_t + 8, sfb_d + 32);
                tmem_cp_32x128b_warpx4_pair(sfb_t + 12, sfb_d + 96);
              }
              mma_mxf4_pair(tmem_base, adesc, bdesc, idesc0, sfa_t, sfb_t, kt != 0);
              mma_mxf4_pair(tmem_base, adesc + 2, bdesc + 2, idesc2, sfa_t, sfb_t, 1);
              if (two) {
                mma_mxf4_pair(tmem_base, adesc + 4, bdesc + 4, idesc0, sfa_t + 4, sfb_t + 8, 1);
                mma_mxf4_pair(tmem_base, adesc + 6, bdesc + 6, idesc2, sfa_t + 4, sfb_t + 8, 1);
              }
              tc_commit_pair(g_empty(s), 3);
            }
            __syncwarp();
          }
          if (ok && elect_one()) tc_commit_pair(g_accf, 3);
          __syncwarp();
        }
      }
    }
  } else {
    // ================================================================== epilogue (8 warps per CTA)
    const int q = warp & 3;
    const int h = (warp - 2) >> 2;
    const int et = (warp - 2) * 32 + lane;               // 0..255 among the epilogue threads
    const int p = lane & 3, r8 = lane >> 2;
    uint8_t* ri_smem = smem_gen + RC::STAGES * RC::STAGE_BYTES;
    const uint32_t ri_saddr = smem_u32(ri_smem);
    bool ok = true;
    // ---- rotation tiles: intra-block rotation, Eq. 1, codes and scales, then the row's counter
    for (int i = 0; i < my_r; ++i) {
      const int t = pair + i * npairs;
      const int mp = t / n_tiles_r, nt = t - mp * n_tiles_r;
      const int mt = 2 * mp + (int)rank;
      const int a = i & 1;
      const int b0 = nt * (RC::BN / 32);
      const bool last = i == my_r - 1;                   // nothing of this pair's overlaps it: warp-MMA form
      if (R_intra != nullptr) {
        named_barrier_sync(1, 256);
        for (int idx = et * 8; ok && idx < (RC::BN / 32) * 1024; idx += 256 * 8) {
          const int lb = idx >> 10, blk = b0 + lb;
          if (last) {                                    // bf16 rows of 80 bytes: conflict-free ldmatrix
            const int ii = (idx & 1023) >> 5, c = idx & 31;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (blk < nblocks) v = __ldg(reinterpret_cast<const uint4*>(R_intra + (size_t)blk * 1024 + (idx & 1023)));
            *reinterpret_cast<uint4*>(ri_smem + lb * RC::RI_BLOCK_BYTES + ii * RC::RI_ROW_BYTES + c * 2) = v;
          } else {                                       // fp32, dense
            float v[8];
            if (blk < nblocks) load8(R_intra + (size_t)blk * 1024 + (idx & 1023), v);
            else {
#pragma unroll
              for (int ii = 0; ii < 8; ++ii) v[ii] = 0.f;
            }
            float* dst = reinterpret_cast<float*>(ri_smem) + idx;
            *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
            *reinterpret_cast<float4*>(dst + 4) = make_float4(v[4], v[5], v[6], v[7]);
          }
        }
        named_barrier_sync(1, 256);
      }
      if (ok) ok = mbar_wait_cluster(r_accf(a), (i >> 1) & 1, cta_abort, err_word, SITE_EPI_ACC_FULL);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) continue;
      tc_fence_after_sync();
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + a * RC::BN + h * 128;
      const int chunk = (b0 + h * 4) >> 2;
      if (!last) {
        // ---- one row per thread, fp32 FMAs
        const int64_t row = (int64_t)mt * RC::BM + q * 32 + lane;
        uint32_t sc_word = 0;
#pragma unroll 1
        for (int bb = 0; bb < 4; ++bb) {
          uint32_t yv[32];
          tmem_ld_32x32(tacc + bb * 32, yv);
          tmem_ld_wait();
          if (bb == 3) {                                 // this warp's share is read: tell the leader
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(r_acce(a), 0));
          }
          float z[32];
          if (R_intra != nullptr) {
            intra_rotate32(yv, ri_saddr + (uint32_t)(h * 4 + bb) * 4096, z);
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) z[j] = __uint_as_float(yv[j]);
          }
          uint4 cw;
          uint32_t sbyte;
          quantize_block32(z, cw, sbyte);
          const int blk = b0 + h * 4 + bb;
          if (row < M && blk < nblocks)
            *reinterpret_cast<uint4*>(codes + row * (int64_t)(d / 2) + (int64_t)blk * 16) = cw;
          sc_word |= sbyte << (8 * bb);
        }
        if (chunk < kb4_r && mt < m_tiles)
          *reinterpret_cast<uint32_t*>(scales + ((size_t)mt * kb4_r + chunk) * 512 + lane * 16 + q * 4) = sc_word;
      } else {
        // ---- accumulator fragment layout (16 rows at a time), warp-level tensor cores
        const int64_t row_base = (int64_t)mt * RC::BM + q * 32 + r8;
        uint32_t sc_word[4] = {0u, 0u, 0u, 0u};
#pragma unroll 1
        for (int bb = 0; bb < 4; ++bb) {
          const int blk = b0 + h * 4 + bb;
          uint32_t bfrag[2][4][2];
          if (R_intra != nullptr) {
            const uint32_t rb = ri_saddr + (uint32_t)(h * 4 + bb) * RC::RI_BLOCK_BYTES +
                                (uint32_t)(((lane >> 3) & 1) * 8 + (lane & 7)) * RC::RI_ROW_BYTES +
                                (uint32_t)(lane >> 4) * 16;
#pragma unroll
            for (int kc = 0; kc < 2; ++kc)
#pragma unroll
              for (int np = 0; np < 2; ++np)
                ldmatrix_x4_trans(rb + kc * 16 * RC::RI_ROW_BYTES + np * 32, bfrag[kc][2 * np][0], bfrag[kc][2 * np][1],
                                  bfrag[kc][2 * np + 1][0], bfrag[kc][2 * np + 1][1]);
          }
#pragma unroll
          for (int mh = 0; mh < 2; ++mh) {
            uint32_t y[16];
            tmem_ld_16x256b_x4(tacc + ((uint32_t)(16 * mh) << 16) + bb * 32, y);
            tmem_ld_wait();
            if (bb == 3 && mh == 1) {
              tc_fence_before_sync();
              __syncwarp();
              if (lane == 0) mbar_arrive_cluster(map_to_cta(r_acce(a), 0));
            }
            float acc[4][4];
            if (R_intra != nullptr) {
              uint32_t ah[8], am[8], al[8];
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
              quantize_row_fragment(v, p, word, sbyte);
              const int64_t row = row_base + 16 * mh + 8 * rh;
              if (row < M && blk < nblocks)
                *reinterpret_cast<uint32_t*>(codes + row * (int64_t)(d / 2) + (int64_t)blk * 16 + 4 * p) = word;
              sc_word[2 * mh + rh] |= sbyte << (8 * bb);
            }
          }
        }
        if (p == 0 && chunk < kb4_r && mt < m_tiles) {
#pragma unroll
          for (int rs = 0; rs < 4; ++rs)
            *reinterpret_cast<uint32_t*>(scales + ((size_t)mt * kb4_r + chunk) * 512 +
                                         (r8 + 16 * (rs >> 1) + 8 * (rs & 1)) * 16 + q * 4) = sc_word[rs];
        }
      }
      // this warp's share of the tile is in global memory: count it for the row tile
      fence_proxy_async_all();
      __threadfence();
      __syncwarp();
      if (lane == 0) asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(row_done + mp) : "memory");
    }
    named_barrier_sync(1, 256);                          // every warp is done with the R_intra staging area
    // ---- GEMM tiles: drain the accumulator, stage rows in shared memory, TMA stores of Y
    const uint32_t out_off = GC::STAGES * GC::STAGE_BYTES;
    uint32_t tcount = 0;
    for (int i = 0; ok; ++i, ++tcount) {
      const int g = sched.tile(pair, i);
      if (g < 0) break;
      const int mp = g / n_tiles_g, nt = g - mp * n_tiles_g;
      const int mt = 2 * mp + (int)rank;
      ok = mbar_wait_cluster(g_accf, tcount & 1, cta_abort, err_word, SITE_EPI_ACC_FULL);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + h * 128;
      uint32_t v0[32], v1[32], v2[32], v3[32];
      tmem_ld_32x32(tacc, v0);
      tmem_ld_32x32(tacc + 32, v1);
      tmem_ld_32x32(tacc + 64, v2);
      tmem_ld_32x32(tacc + 96, v3);
      tmem_ld_wait();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(g_acce, 0));
      const int row0 = mt * GC::BM + q * 32;
      const int col0 = nt * GC::BN + h * 128;
      const uint32_t stage_buf = smem_base + out_off + (uint32_t)(warp - 2) * GC::OUT_WARP_BYTES;
      const uint32_t my_row = stage_buf + lane * 128;
      const uint32_t sw = (uint32_t)(lane & 7);
      auto put16 = [&](int piece, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3) {
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                     ::"r"(my_row + (((uint32_t)piece ^ sw) << 4)), "r"(a0), "r"(a1), "r"(a2), "r"(a3) : "memory");
      };
      auto pack2 = [](uint32_t lo, uint32_t hi) {
        __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(lo), __uint_as_float(hi));
        return *reinterpret_cast<uint32_t*>(&hh);
      };
      auto flush = [&](int col) {
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0 && row0 < M && col < N) {
          tma_store_2d(&tmY, col, row0, stage_buf);
          bulk_commit_group();
        }
      };
      auto reuse = [&]() {
        if (lane == 0) bulk_wait_group_read<0>();
        __syncwarp();
      };
      if (y_is_bf16) {
        auto half64 = [&](const uint32_t (&lo)[32], const uint32_t (&hi)[32], int col) {
          reuse();
#pragma unroll
          for (int pp = 0; pp < 4; ++pp)
            put16(pp, pack2(lo[8 * pp], lo[8 * pp + 1]), pack2(lo[8 * pp + 2], lo[8 * pp + 3]),
                  pack2(lo[8 * pp + 4], lo[8 * pp + 5]), pack2(lo[8 * pp + 6], lo[8 * pp + 7]));
#pragma unroll
          for (int pp = 0; pp < 4; ++pp)
            put16(4 + pp, pack2(hi[8 * pp], hi[8 * pp + 1]), pack2(hi[8 * pp + 2], hi[8 * pp + 3]),
                  pack2(hi[8 * pp + 4], hi[8 * pp + 5]), pack2(hi[8 * pp + 6], hi[8 * pp + 7]));
          flush(col);
        };
        half64(v0, v1, col0);
        half64(v2, v3, col0 + 64);
      } else {
        auto quarter32 = [&](const uint32_t (&v)[32], int col) {
          reuse();
#pragma unroll
          for (int pp = 0; pp < 8; ++pp) put16(pp, v[4 * pp], v[4 * pp + 1], v[4 * pp + 2], v[4 * pp + 3]);
          flush(col);
        };
        quarter32(v0, col0);
        quarter32(v1, col0 + 32);
        quarter32(v2, col0 + 64);
        quarter32(v3, col0 + 96);
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
    tmem_dealloc_pair(tmem_base, FusedCfg::TMEM_COLS);
  }
}

}  // namespace torq
