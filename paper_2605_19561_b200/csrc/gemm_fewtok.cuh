// Block-scaled GEMM for few tokens (M <= 128; Algorithm 3 step 5), where the work is streaming the
// weights from HBM once.  One kernel, no scratch in global memory.
//
// Swapped operands: the tensor-core instruction's 128 rows are 128 output FEATURES (rows of the
// stored weight W' [N, K]) and its N columns are the tokens (16, 32, 64 or 128):
//   D[n, m] = sum_k w^[n, k] a^[m, k]
//   A = W tile [128 rows x 128 B of K], scale chunks of W;  B = activation tile [tokens x 128 B],
//   scale chunks of the activations (their single 128-row scale tile).
// A layer has only N / 128 such tiles (40 at N = 5120), so K is split as well: a CLUSTER of S CTAs
// shares one tile, CTA r contracts k range r; the fp32 partial tiles stay on the SMs -- each CTA
// writes its partial [token][feature] into its own shared memory, a cluster barrier publishes them,
// and CTA r then adds, for the tokens m = r (mod S), the S partials in rank order through
// distributed shared memory (plain ld.shared::cluster; fixed order) and stores that token's 128
// outputs as one 256- or 512-byte piece of a row of Y.
//
// Roles per CTA: warp 0 TMA producer, warp 1 MMA issuer (scale chunks shared -> tensor memory, then the
// instructions), warps 2..5 epilogue / reduction.  Shared memory: 4 stages of (16 KiB of W + tokens x
// 128 B + the scale chunks), reused for the partial tile after the mainloop; at most 113 KiB, so these
// CTAs become resident beside those of the few-token rotation that precedes them in the stream and
// fetch their first weight stages while it still runs (the weights are constants of the layer).
#pragma once
#include <cuda_bf16.h>
#include "rotate_fewtok.cuh"
#include "sm100_ptx.cuh"

namespace torq {

template <int FMT = FMT_MXFP4>
struct GemmFewCfg {
  static constexpr int BF = 128;                       // output features per tile = rows of the instruction
  static constexpr int BK = FMT == FMT_MXINT4 ? 128 : 256;   // elements of K per stage (128 bytes per row)
  static constexpr int A_BYTES = BF * 128;             // 16 KiB
  static constexpr int CH = FMT == FMT_NVFP4 ? 4 : (FMT == FMT_MXINT4 ? 1 : 2);   // scale chunks per stage and 128 rows
  static constexpr int SF_BYTES = CH * 512;
  static constexpr int STAGES = 4;
  // the same for every token count: three stages at 128 tokens would let two CTAs share an SM (clusters of 5
  // instead of 3), which measured 4 - 10 % slower than four stages and one CTA per SM
  __host__ __device__ static constexpr int stages(int) { return STAGES; }
  static constexpr int BAR_BYTES = 256;
  static constexpr int THREADS = 192;
  static constexpr int MAX_CLUSTER = 8;
  static constexpr int MAX_TOK = 128;                  // one 128-row scale tile of the activations
  __host__ __device__ static constexpr int stage_bytes(int ntok) {
    return (A_BYTES + ntok * 128 + 2 * SF_BYTES + 1023) / 1024 * 1024;
  }
  __host__ __device__ static constexpr int smem_bytes(int ntok) { return stages(ntok) * stage_bytes(ntok) + BAR_BYTES + 1024; }
  __host__ __device__ static constexpr int ctas_per_sm(int ntok) { return smem_bytes(ntok) <= 113 * 1024 ? 2 : 1; }
  __host__ __device__ static constexpr int max_smem_bytes() {                  // over the token counts in use
    return smem_bytes(64) > smem_bytes(128) ? smem_bytes(64) : smem_bytes(128);
  }
  __host__ __device__ static constexpr uint32_t tmem_cols(int ntok) {
    return ntok + 8 * CH <= 32 ? 32u : (ntok + 8 * CH <= 64 ? 64u : (ntok + 8 * CH <= 128 ? 128u : 256u));
  }
};

// grid = ceil(N / 128) * S CTAs in clusters of S along x: CTA b works feature tile b / S, k split b % S.
// tmW: Wq [N, K bytes] box [128 x 128]; tmA: Aq [M, K bytes] box [ntok x 128]; As / Ws: tiled scales.
// ESETS: sets of four epilogue warps (threads = 64 + 128 ESETS): one set and two CTAs per SM up to 64 tokens;
// two sets at 128 tokens, where a CTA fills an SM by itself and has some forty tokens to add up and store.
template <int FMT = FMT_MXFP4, int ESETS = 1>
__global__ void __launch_bounds__(64 + 128 * ESETS, ESETS == 1 ? 2 : 1)
gemm_fewtok_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmA,
                   const uint8_t* __restrict__ As, const uint8_t* __restrict__ Ws, void* __restrict__ Y,
                   int y_is_bf16, int M, int N, int K, int ntok, int S, float alpha, int* err_word) {
  using C = GemmFewCfg<FMT>;
  constexpr int CH = C::CH;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const int stage_bytes = C::stage_bytes(ntok);
  const int b_bytes = ntok * 128;
  const int nst = C::stages(ntok);
  const uint32_t bar_off = nst * stage_bytes;
  const uint32_t bar_base = smem_base + bar_off;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (C::STAGES + s); };
  const uint32_t accf_bar = bar_base + 8u * (2 * C::STAGES);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + bar_off + 192);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(smem_gen + bar_off + 200);
  float* P = reinterpret_cast<float*>(smem_gen);         // after the mainloop: partial tile [token][feature]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = blockIdx.x % S, nt = blockIdx.x / S;
  const int k_tiles = (K + C::BK - 1) / C::BK;           // K % 128 == 0: the last stage may be half
  const int kb4 = K / (C::BK / CH);                      // scale chunks per row
  const int kt0 = (int)((long long)k_tiles * rank / S), kt1 = (int)((long long)k_tiles * (rank + 1) / S);
  const uint32_t tmem_cols = C::tmem_cols(ntok);

  // The weights and their scales are constants of the layer, never the output of the kernel that runs
  // just before this one: the thread that initialises the barriers sends their loads for the first
  // stages right behind the initialisation (the kernel's time starts with an HBM round trip; tensor-
  // memory allocation and the block-wide barrier come after it instead of before); the activations wait.
  const int pre = (kt1 - kt0) < nst ? (kt1 - kt0) : nst;
  auto stage_tx = [&](int kt) { return (uint32_t)(C::A_BYTES + b_bytes) + 2u * 512u * (uint32_t)min(CH, kb4 - CH * kt); };
  if (threadIdx.x == 0) {
    for (int s = 0; s < nst; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(accf_bar, 1);
    *cta_abort = 0;
    fence_mbar_init();
    fence_proxy_async_smem();                            // the copy engine sees the initialised barriers
    for (int it = 0; it < pre; ++it) {
      const int kt = kt0 + it;
      const uint32_t st = smem_base + it * stage_bytes;
      mbar_arrive_expect_tx(full_bar(it), stage_tx(kt));
      tma_load_2d(st, &tmW, kt * 128, nt * C::BF, full_bar(it));
      bulk_load_1d(st + C::A_BYTES + b_bytes, Ws + ((size_t)nt * kb4 + CH * kt) * 512,
                   512u * (uint32_t)min(CH, kb4 - CH * kt), full_bar(it));
    }
    tma_prefetch_desc(&tmA);
  }
  if (warp == 1) { tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), tmem_cols); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  griddep_launch_dependents();
  griddep_wait();

  bool acc_ok = false;
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    bool ok = true;
    for (int kt = kt0, it = 0; kt < kt1 && ok; ++kt, ++it) {
      const int s = it % nst;
      if (!mbar_wait_warp(empty_bar(s), ((it / nst) & 1) ^ 1, cta_abort, err_word, SITE_PRODUCER_EMPTY)) {
        ok = false; break;
      }
      const uint32_t st = smem_base + s * stage_bytes;
      const uint32_t sf_bytes = 512u * (uint32_t)min(CH, kb4 - CH * kt);
      if (elect_one()) {
        const bool w_issued = it < pre;                  // W side of this stage went out before the wait above
        if (!w_issued) {
          mbar_arrive_expect_tx(full_bar(s), stage_tx(kt));
          tma_load_2d(st, &tmW, kt * 128, nt * C::BF, full_bar(s));
          bulk_load_1d(st + C::A_BYTES + b_bytes, Ws + ((size_t)nt * kb4 + CH * kt) * 512, sf_bytes, full_bar(s));
        }
        tma_load_2d(st + C::A_BYTES, &tmA, kt * 128, 0, full_bar(s));
        bulk_load_1d(st + C::A_BYTES + b_bytes + C::SF_BYTES, As + (size_t)(CH * kt) * 512, sf_bytes, full_bar(s));
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    bool ok = true;
    const uint32_t idesc0 = FMT == FMT_NVFP4 ? idesc_nvf4(128, ntok) : idesc_mxf4(128, ntok, 0, 0);
    const uint32_t idesc2 = FMT == FMT_NVFP4 ? idesc_nvf4(128, ntok) : idesc_mxf4(128, ntok, 2, 2);
    const uint32_t sfa_t = tmem_base + ntok, sfb_t = tmem_base + ntok + 4 * CH;     // 4 columns per chunk each
    for (int kt = kt0, it = 0; kt < kt1 && ok; ++kt, ++it) {
      const int s = it % nst;
      if (!mbar_wait_warp(full_bar(s), (it / nst) & 1, cta_abort, err_word, SITE_MMA_FULL)) {
        ok = false; break;
      }
      tc_fence_after_sync();
      const bool two = (kb4 - CH * kt) >= CH;              // K % 256 == 128: the last stage is half
      const uint32_t st = smem_base + s * stage_bytes;
      const uint64_t adesc = make_desc(st, 16, 1024, kSwizzle128);
      const uint64_t bdesc = make_desc(st + C::A_BYTES, 16, 1024, kSwizzle128);
      const uint64_t sfa_d = make_desc(st + C::A_BYTES + b_bytes, 0, 128, 0);
      const uint64_t sfb_d = make_desc(st + C::A_BYTES + b_bytes + C::SF_BYTES, 0, 128, 0);
      if (elect_one()) {
#pragma unroll
        for (int c = 0; c < CH; ++c) {
          if (c < CH / 2 || two) {
            tmem_cp_32x128b_warpx4(sfa_t + 4 * c, sfa_d + 32 * c);
            tmem_cp_32x128b_warpx4(sfb_t + 4 * c, sfb_d + 32 * c);
          }
        }
        if constexpr (FMT == FMT_MXINT4) {                 // a quarter chunk (one scale byte) per instruction
          mma_mxf8(tmem_base, adesc, bdesc, idesc_mxf8(128, ntok, 0), sfa_t, sfb_t, it != 0);
          mma_mxf8(tmem_base, adesc + 2, bdesc + 2, idesc_mxf8(128, ntok, 1), sfa_t, sfb_t, 1);
          mma_mxf8(tmem_base, adesc + 4, bdesc + 4, idesc_mxf8(128, ntok, 2), sfa_t, sfb_t, 1);
          mma_mxf8(tmem_base, adesc + 6, bdesc + 6, idesc_mxf8(128, ntok, 3), sfa_t, sfb_t, 1);
        } else if constexpr (FMT == FMT_NVFP4) {           // one chunk per instruction
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (j < 2 || two)
              mma_nvf4(tmem_base, adesc + 2 * j, bdesc + 2 * j, idesc0, sfa_t + 4 * j, sfb_t + 4 * j, (it | j) != 0);
        } else {                                           // half a chunk (two scale bytes) per instruction
          mma_mxf4(tmem_base, adesc, bdesc, idesc0, sfa_t, sfb_t, it != 0);
          mma_mxf4(tmem_base, adesc + 2, bdesc + 2, idesc2, sfa_t, sfb_t, 1);
          if (two) {
            mma_mxf4(tmem_base, adesc + 4, bdesc + 4, idesc0, sfa_t + 4, sfb_t + 4, 1);
            mma_mxf4(tmem_base, adesc + 6, bdesc + 6, idesc2, sfa_t + 4, sfb_t + 4, 1);
          }
        }
        tc_commit(empty_bar(s));
      }
      __syncwarp();
    }
    if (ok && elect_one()) tc_commit(accf_bar);
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    // Two passes over the SAME instructions, as in the few-token rotation: pass 0 is a dry run while the
    // mainloop streams (reads this CTA's own shared memory, stores nothing) so that the reduction's code is
    // in the instruction cache when it is needed; pass 1: accumulator -> own shared memory, cluster
    // barrier, then the tokens of this CTA.
    // A warp takes one token per pass: lane l adds features 4 l .. 4 l + 3 (16-byte loads, 512 contiguous
    // bytes per warp and partial) and stores 8 or 16 bytes of the token's row of Y.  Two tokens per
    // iteration, all their loads issued before the first add: few round trips through the cluster.
    const int q = warp & 3;
    const int ew = warp - 2;                             // 0 .. 4 ESETS - 1
    constexpr int NW = 4 * ESETS;
    const int64_t n = (int64_t)nt * C::BF + 4 * lane;
    const uint32_t p_saddr = smem_u32(P);
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {
      const bool live = pass == 1;
      if (live) {
        // ---- epilogue 1: partial tile -> own shared memory
        acc_ok = mbar_wait(accf_bar, 0, cta_abort, err_word, SITE_EPI_ACC_FULL);
        acc_ok = __all_sync(0xFFFFFFFFu, acc_ok);
        if (acc_ok) {
          tc_fence_after_sync();
          const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16);
          float* prow = P + q * 32 + lane;               // feature 32 q + lane of token 0
          for (int c0 = 16 * (ew >> 2); c0 < ntok; c0 += 16 * ESETS) {
            uint32_t v[16];
            tmem_ld_32x32_x16(tacc + c0, v);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j) prow[(c0 + j) * C::BF] = __uint_as_float(v[j]);
          }
        }
        tc_fence_before_sync();
        cluster_sync_all();                              // every CTA's partial tile is visible cluster-wide
      }
      // ---- epilogue 2: add the partials, store Y
      uint32_t p_rank[C::MAX_CLUSTER];
#pragma unroll
      for (int s = 0; s < C::MAX_CLUSTER; ++s)
        p_rank[s] = s < S ? map_to_cta(p_saddr, live ? (uint32_t)s : (uint32_t)rank) : 0u;
      for (int m0 = rank + S * ew; m0 < M; m0 += 2 * NW * S) {
        float4 part[2][C::MAX_CLUSTER];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int m = m0 + NW * S * j;
          if (m < M) {
            const uint32_t off = (uint32_t)((m * C::BF + 4 * lane) * 4);
#pragma unroll
            for (int s = 0; s < C::MAX_CLUSTER; ++s)
              if (s < S)
                asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                             : "=f"(part[j][s].x), "=f"(part[j][s].y), "=f"(part[j][s].z), "=f"(part[j][s].w)
                             : "r"(p_rank[s] + off));
          }
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int m = m0 + NW * S * j;
          if (m < M) {
            float4 y = make_float4(0.f, 0.f, 0.f, 0.f);  // rank order: the result does not depend on timing
#pragma unroll
            for (int s = 0; s < C::MAX_CLUSTER; ++s)
              if (s < S) { y.x += part[j][s].x; y.y += part[j][s].y; y.z += part[j][s].z; y.w += part[j][s].w; }
            if constexpr (FMT == FMT_NVFP4) { y.x *= alpha; y.y *= alpha; y.z *= alpha; y.w *= alpha; }
            if (live && n < N) {                         // N % 8 == 0: four features are inside or outside together
              if (y_is_bf16) {
                __nv_bfloat162 h0 = __floats2bfloat162_rn(y.x, y.y), h1 = __floats2bfloat162_rn(y.z, y.w);
                *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(Y) + (int64_t)m * N + n) =
                    make_uint2(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1));
              } else {
                *reinterpret_cast<float4*>(reinterpret_cast<float*>(Y) + (int64_t)m * N + n) = y;
              }
            }
          }
        }
      }
    }
  }
  if (warp < 2) {                                        // the epilogue warps passed this barrier inside their pass 1
    tc_fence_before_sync();
    cluster_sync_all();
  }

  // ------------------------------------------------------------------ teardown
  __syncthreads();
  if (*cta_abort) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  cluster_sync_all();                                    // no CTA of the cluster reads this one's partial tile any more
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, tmem_cols);
  }
}

}  // namespace torq
