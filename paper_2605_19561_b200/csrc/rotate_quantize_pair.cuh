// Rotate + quantize for M > 128 on CTA pairs: the same computation and epilogue as
// rotate_quantize_kernel, but two CTAs (a cluster of 2, one per SM) share one 256 x 256 output
// tile through tcgen05.mma cta_group::2.  Each CTA stages only its own 128 rows of X and its own
// 128 columns of R_inter per K step (32 KiB instead of 48 KiB per 128 x 256 x 64 of work), which
// is what the single-CTA kernel is short of: it cannot keep enough bytes in flight from L2 to
// feed the tensor pipe.  No multicast load is used; operand sharing happens inside the MMA, which
// reads both CTAs' shared memory.
//
// Roles per CTA: warp 0 TMA producer (both CTAs), warp 1 MMA issuer (leader CTA only; both
// allocate tensor memory), warps 2..5 epilogue (each CTA drains its own 128 x 256 accumulator).
// Barriers: full[s] lives in the leader and counts the bytes of both CTAs' loads; empty[s] and
// acc_full[a] are local to each CTA and are signalled by the leader's tcgen05.commit to both;
// acc_empty[a] lives in the leader and takes one arrival per epilogue warp of both CTAs.
#pragma once
#include <cuda_bf16.h>
#include "quantize.cuh"
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
  static constexpr int RI_BYTES = (BN / 32) * 32 * 32 * 4;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + RI_BYTES + 256 + 1024;
  static constexpr int NACC = 2;
  static constexpr int TMEM_COLS = 512;
  static constexpr int THREADS = 192;
  static_assert(SMEM_BYTES <= 232448, "shared memory budget");
};

__global__ void __launch_bounds__(192, 1)
rotate_quantize_pair_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmR,
                            const __nv_bfloat16* __restrict__ R_intra, uint8_t* __restrict__ codes,
                            uint8_t* __restrict__ scales, int M, int d, int* err_word) {
  using C = RotPairCfg;
  constexpr int BN = C::BN;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  float* ri_smem = reinterpret_cast<float*>(smem_gen + C::STAGES * C::STAGE_BYTES);
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
  const int mp_tiles = (M + 255) / 256;                // 256-row pair tiles
  const int n_tiles = (d + BN - 1) / BN;
  const int total_tiles = mp_tiles * n_tiles;
  const int k_tiles = (d + C::BK - 1) / C::BK;
  const int nblocks = d / 32;
  const int kb4 = (nblocks + 3) / 4;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < C::NACC; ++a) { mbar_init(accf_bar(a), 1); mbar_init(acce_bar(a), 8); }
    *cta_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::TMEM_COLS); tmem_relinquish_pair(); }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();                                  // both CTAs' barriers exist before any remote arrive
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // Set-up above touched no global memory; from here on the previous kernel's results are needed.
  griddep_launch_dependents();
  griddep_wait();

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (elect_one()) { tma_prefetch_desc(&tmX); tma_prefetch_desc(&tmR); }
    uint32_t it = 0;
    bool ok = true;
    for (int tile = pair; tile < total_tiles && ok; tile += npairs) {
      const int mt = 2 * (tile % mp_tiles) + (int)rank, nt = tile / mp_tiles;
      for (int kt = 0; kt < k_tiles; ++kt, ++it) {
        const int s = it % C::STAGES;
        if (!mbar_wait_cluster_warp(empty_bar(s), ((it / C::STAGES) & 1) ^ 1, cta_abort, err_word,
                               SITE_PRODUCER_EMPTY)) { ok = false; break; }
        const uint32_t st = smem_base + s * C::STAGE_BYTES;
        const uint32_t leader_full = map_to_cta(full_bar(s), 0);
        if (elect_one()) {
          if (rank == 0) mbar_arrive_expect_tx(full_bar(s), 2 * C::STAGE_BYTES);
          tma_load_2d_pair(st, &tmX, kt * C::BK, mt * C::BM, leader_full);
#pragma unroll
          for (int b = 0; b < BN / 2 / 64; ++b)
            tma_load_2d_pair(st + C::A_BYTES + b * C::B_BOX_BYTES, &tmR,
                             nt * BN + (int)rank * (BN / 2) + b * 64, kt * C::BK, leader_full);
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    if (rank == 0) {
      constexpr uint32_t idesc = idesc_bf16(256, BN, /*A MN-major*/ false, /*B MN-major*/ true);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = pair; tile < total_tiles && ok; tile += npairs, ++tcount) {
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
    // ------------------------------------------------------------------ epilogue (128 threads per CTA)
    const int q = warp & 3;
    const int et = (warp - 2) * 32 + lane;
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = pair; tile < total_tiles; tile += npairs, ++tcount) {
      const int mt = 2 * (tile % mp_tiles) + (int)rank, nt = tile / mp_tiles;
      const int a = tcount % C::NACC;
      const int b0 = nt * (BN / 32);
      if (R_intra != nullptr) {
        // Executed by every epilogue thread for every tile, also after a wait has given up.
        named_barrier_sync(1, 128);
        for (int idx = et * 8; ok && idx < (BN / 32) * 1024; idx += 128 * 8) {
          const int blk = b0 + (idx >> 10);
          float v[8];
          if (blk < nblocks) load8(R_intra + (size_t)blk * 1024 + (idx & 1023), v);
          else {
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = 0.f;
          }
          *reinterpret_cast<float4*>(ri_smem + idx) = make_float4(v[0], v[1], v[2], v[3]);
          *reinterpret_cast<float4*>(ri_smem + idx + 4) = make_float4(v[4], v[5], v[6], v[7]);
        }
        named_barrier_sync(1, 128);
      }
      if (ok) ok = mbar_wait_cluster(accf_bar(a), (tcount / C::NACC) & 1, cta_abort, err_word, SITE_EPI_ACC_FULL);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) continue;
      tc_fence_after_sync();
      const int64_t row = (int64_t)mt * C::BM + q * 32 + lane;
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + a * BN;
      uint32_t sc_word = 0;
#pragma unroll 1
      for (int bb = 0; bb < BN / 32; ++bb) {
        uint32_t yv[32];
        tmem_ld_32x32(tacc + bb * 32, yv);
        tmem_ld_wait();
        if (bb == BN / 32 - 1) {                         // accumulator fully read: tell the leader
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(map_to_cta(acce_bar(a), 0));
        }
        float z[32];
        if (R_intra != nullptr) {
#pragma unroll
          for (int j = 0; j < 32; ++j) z[j] = 0.f;
          const float4* r = reinterpret_cast<const float4*>(ri_smem + bb * 1024);
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float yi = __uint_as_float(yv[i]);
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              const float4 rv = r[i * 8 + g];
              z[4 * g + 0] = fmaf(yi, rv.x, z[4 * g + 0]);
              z[4 * g + 1] = fmaf(yi, rv.y, z[4 * g + 1]);
              z[4 * g + 2] = fmaf(yi, rv.z, z[4 * g + 2]);
              z[4 * g + 3] = fmaf(yi, rv.w, z[4 * g + 3]);
            }
          }
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) z[j] = __uint_as_float(yv[j]);
        }
        uint4 cw;
        uint32_t sbyte;
        quantize_block32(z, cw, sbyte);
        const int blk = b0 + bb;
        if (row < M && blk < nblocks)
          *reinterpret_cast<uint4*>(codes + row * (int64_t)(d / 2) + (int64_t)blk * 16) = cw;
        sc_word |= sbyte << (8 * (bb & 3));
        if ((bb & 3) == 3) {
          const int chunk = (b0 + bb) >> 2;
          if (chunk < kb4 && mt < m_tiles)               // the pair's second row tile may not exist
            *reinterpret_cast<uint32_t*>(scales + ((size_t)mt * kb4 + chunk) * 512 + lane * 16 + q * 4) =
                sc_word;
          sc_word = 0;
        }
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
