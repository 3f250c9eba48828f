// Rotate + quantize for few tokens (M <= 256), where the work is streaming R_inter from HBM once
// (Algorithm 3 steps 2-4).  One kernel, no scratch in global memory.
//
// Swapped operands: the tensor-core instruction's 128 rows are 128 output FEATURES (four 32-blocks)
// and its N columns are the tokens (16 ... 256), so no row of the instruction is padding and the
// accumulator is small:  D[j, m] = sum_i R_inter[i, j] X[m, i].
//   A = R_inter tile [64 (i) x 128 (j)], features contiguous = MN-major, two 64 x 64 boxes (128-B swizzle)
//   B = X tile [tokens x 64 (i)], K-major
// A layer has only d / 128 feature tiles (40 at d = 5120), too few CTAs to pull R_inter at HBM rate,
// so the contraction is also split: a CLUSTER of S CTAs shares one feature tile, CTA r of the cluster
// contracts k range r.  The fp32 partial tiles never leave the SMs: every CTA writes its partial
// [token][feature] into its own shared memory, a cluster barrier publishes them, and each warp of
// the cluster then owns some (16 tokens x one 32-block) units: it adds the S partials of its unit in
// rank order through distributed shared memory (plain ld.shared::cluster; fixed order, so the result
// does not depend on timing), applies the intra-block rotation on the warp-level tensor cores (y split
// into three bf16 terms, fp32 accumulation) and quantizes (Eq. 1).
//
// Units: epilogue warp w of every CTA owns 32-block w of the tile (its R_intra block is fetched into
// shared memory when the kernel starts, long before it is needed: a first touch of that array from a
// cold TLB costs microseconds); CTA r of the cluster takes the token groups r, r + S, ...
//
// Roles per CTA: warp 0 TMA producer, warp 1 MMA issuer, warps 2..5 epilogue / reduction.
// Shared memory: 4 stages of (16 KiB of R_inter + tokens x 128 B of X); after the mainloop the same
// memory holds the partial tile and the per-warp staging of the reduction.  Up to 64 tokens that is small
// enough (<= 107 KiB) for two CTAs per SM: the grid may exceed the SM count, which keeps more loads in
// flight; with 128 or 256 tokens one CTA fills an SM and the grid stays within the SM count.
#pragma once
#include <cuda_bf16.h>
#include "intra_fragment.cuh"
#include "sm100_ptx.cuh"

namespace torq {

struct RotFewCfg {
  static constexpr int BF = 128;                       // features per tile = rows of the instruction
  static constexpr int BK = 64;
  static constexpr int A_BYTES = BK * BF * 2;          // 16 KiB: two boxes of 64 (k) x 64 (j)
  static constexpr int A_BOX_BYTES = 64 * 64 * 2;
  static constexpr int STAGES = 4;
  // the same for every token count: three stages at 128 tokens would let two CTAs share an SM (clusters of 5
  // instead of 3), which measured 4 - 10 % slower than four stages and one CTA per SM
  __host__ __device__ static constexpr int stages(int) { return STAGES; }
  static constexpr int MAX_TOK = 256;                  // N of the instruction; 16, 32, 64, 128 or 256 are used
  static constexpr int Y_BYTES = 16 * 33 * 4;          // per epilogue warp: 16 tokens x 32 features, row stride 33
  static constexpr int RI_BYTES = 32 * 80;             // per epilogue warp: R_intra[block] as bf16 rows of 80 bytes
  static constexpr int BAR_BYTES = 256;
  static constexpr int THREADS = 192;
  static constexpr int MAX_CLUSTER = 8;
  __host__ __device__ static constexpr int stage_bytes(int ntok) { return A_BYTES + ntok * BK * 2; }
  __host__ __device__ static constexpr int smem_bytes(int ntok) {
    return stages(ntok) * stage_bytes(ntok) + BAR_BYTES + 4 * RI_BYTES + 1024;
  }
  // the partial tile (ntok x 512 B) and the warps' y tiles must fit inside the stages they reuse
  __host__ __device__ static constexpr bool reduction_fits(int ntok) {
    return ntok * BF * 4 + 8 * Y_BYTES <= stages(ntok) * stage_bytes(ntok);   // up to eight epilogue warps
  }
  __host__ __device__ static constexpr int ctas_per_sm(int ntok) { return smem_bytes(ntok) <= 113 * 1024 ? 2 : 1; }
  __host__ __device__ static constexpr int max_smem_bytes() {                  // over the token counts in use
    return smem_bytes(256) > smem_bytes(64) ? smem_bytes(256) : smem_bytes(64);
  }
};
static_assert(RotFewCfg::reduction_fits(16) && RotFewCfg::reduction_fits(32) && RotFewCfg::reduction_fits(64) &&
              RotFewCfg::reduction_fits(128) && RotFewCfg::reduction_fits(256), "reduction buffers");

// grid = (d / 128) * S CTAs in clusters of S along x: CTA b works feature tile b / S, k split b % S.
// tmX: X [M, d] bf16, box [ntok rows x 64]; tmR: R_inter [d, d] bf16, box [64 x 64].  ntok = 16, 32, 64, 128 or 256
// >= M.  d % 128 == 0.  `codes` / `scales` / `tensor_scale` as in rotate_quantize_kernel for FMT.
// ESETS: sets of four epilogue warps (threads = 64 + 128 ESETS).  One set and two CTAs per SM up to 64
// tokens; with 128 or 256 tokens a CTA fills an SM by itself and has several token groups to reduce, rotate
// and quantize, each a dependent chain of about a microsecond for one warp: two sets take them in turn.
template <int FMT = FMT_MXFP4, int ESETS = 1>
__global__ void __launch_bounds__(64 + 128 * ESETS, ESETS == 1 ? 2 : 1)
rotate_fewtok_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmR,
                     const __nv_bfloat16* __restrict__ R_intra, uint8_t* __restrict__ codes,
                     uint8_t* __restrict__ scales, int M, int d, int ntok, int S, float tensor_scale,
                     int* err_word) {
  using C = RotFewCfg;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const int stage_bytes = C::stage_bytes(ntok);
  const int nst = C::stages(ntok);
  const uint32_t bar_off = nst * stage_bytes;
  const uint32_t bar_base = smem_base + bar_off;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (C::STAGES + s); };
  const uint32_t accf_bar = bar_base + 8u * (2 * C::STAGES);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + bar_off + 192);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(smem_gen + bar_off + 200);
  // after the mainloop: partial tile P[token][feature] fp32 at offset 0, then the warps' y tiles
  float* P = reinterpret_cast<float*>(smem_gen);
  uint8_t* y_tiles = smem_gen + ntok * C::BF * 4;
  uint8_t* ri_tiles = smem_gen + bar_off + C::BAR_BYTES;    // not part of the stages: filled at kernel start

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = blockIdx.x % S, ft = blockIdx.x / S;
  const int k_tiles = d / C::BK;
  const int kt0 = (int)((long long)k_tiles * rank / S), kt1 = (int)((long long)k_tiles * (rank + 1) / S);
  const uint32_t tmem_cols = ntok < 32 ? 32u : (uint32_t)ntok;

  // R_inter is a constant of the layer, never the output of the kernel that runs just before this
  // one: the thread that initialises the barriers sends the loads of the first stages' R_inter tiles
  // right behind the initialisation (the kernel's time starts with an HBM round trip; tensor-memory
  // allocation and the block-wide barrier come after it instead of before).  X waits for that kernel.
  const int pre = (kt1 - kt0) < nst ? (kt1 - kt0) : nst;
  if (threadIdx.x == 0) {
    for (int s = 0; s < nst; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(accf_bar, 1);
    *cta_abort = 0;
    fence_mbar_init();
    fence_proxy_async_smem();                            // the copy engine sees the initialised barriers
    for (int it = 0; it < pre; ++it) {
      const uint32_t st = smem_base + it * stage_bytes;
      mbar_arrive_expect_tx(full_bar(it), (uint32_t)stage_bytes);
      tma_load_2d(st, &tmR, ft * C::BF, (kt0 + it) * C::BK, full_bar(it));
      tma_load_2d(st + C::A_BOX_BYTES, &tmR, ft * C::BF + 64, (kt0 + it) * C::BK, full_bar(it));
    }
    tma_prefetch_desc(&tmX);
  }
  if (warp == 1) { tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), tmem_cols); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  griddep_launch_dependents();
  const int groups = ntok / 16;                          // token groups of 16; group g belongs to CTA g % S
  if (warp >= 2 && warp < 6 && R_intra != nullptr && rank < groups) {
    // this warp's R_intra block (a constant of the layer as well), 128 pieces of 16 B: row piece / 4
    uint8_t* r_s = ri_tiles + (warp - 2) * C::RI_BYTES;
    const uint4* src = reinterpret_cast<const uint4*>(R_intra + (size_t)(ft * 4 + (warp - 2)) * 1024);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int piece = lane + 32 * i;
      *reinterpret_cast<uint4*>(r_s + (piece >> 2) * 80 + (piece & 3) * 16) = __ldg(src + piece);
    }
  }
  griddep_wait();

  bool acc_ok = false;                                   // epilogue warps: the accumulator is complete
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    bool ok = true;
    for (int kt = kt0, it = 0; kt < kt1 && ok; ++kt, ++it) {
      const int s = it % nst;
      if (!mbar_wait_warp(empty_bar(s), ((it / nst) & 1) ^ 1, cta_abort, err_word, SITE_PRODUCER_EMPTY)) {
        ok = false; break;
      }
      const uint32_t st = smem_base + s * stage_bytes;
      if (elect_one()) {
        const bool r_issued = it < pre;                  // R side of this stage went out before the wait above
        if (!r_issued) {
          mbar_arrive_expect_tx(full_bar(s), (uint32_t)stage_bytes);
          tma_load_2d(st, &tmR, ft * C::BF, kt * C::BK, full_bar(s));
          tma_load_2d(st + C::A_BOX_BYTES, &tmR, ft * C::BF + 64, kt * C::BK, full_bar(s));
        }
        tma_load_2d(st + C::A_BYTES, &tmX, kt * C::BK, 0, full_bar(s));
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    const uint32_t idesc = idesc_bf16(128, ntok, /*A MN-major*/ true, /*B MN-major*/ false);
    bool ok = true;
    for (int kt = kt0, it = 0; kt < kt1 && ok; ++kt, ++it) {
      const int s = it % nst;
      if (!mbar_wait_warp(full_bar(s), (it / nst) & 1, cta_abort, err_word, SITE_MMA_FULL)) {
        ok = false; break;
      }
      tc_fence_after_sync();
      const uint32_t st = smem_base + s * stage_bytes;
      // A: MN-major.  64 features (128 B) contiguous, k rows 128 B apart, 8-row groups 1024 B apart
      // (stride offset), the next 64 features one box (8 KiB) further (leading offset).
      const uint64_t adesc = make_desc(st, C::A_BOX_BYTES, 1024, kSwizzle128);
      // B: K-major, token rows of 128 B, 8-row groups 1024 B apart.
      const uint64_t bdesc = make_desc(st + C::A_BYTES, 16, 1024, kSwizzle128);
      if (elect_one()) {
#pragma unroll
        for (int j = 0; j < C::BK / 16; ++j)             // K = 16 per instruction: 16 k rows of A = 2 KiB, 32 B of B
          mma_bf16(tmem_base, adesc + 128 * j, bdesc + 2 * j, idesc, (it | j) != 0);
        tc_commit(empty_bar(s));
      }
      __syncwarp();
    }
    if (ok && elect_one()) tc_commit(accf_bar);
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    // Two passes over the SAME instructions.  Pass 0 is a dry run while the mainloop streams: it reads
    // this CTA's own shared memory (whatever it holds), computes, and stores nothing.  Its only purpose
    // is to have the reduction's code in the instruction cache: executed cold, after the mainloop,
    // that code cost about 2.5 us of instruction fetches -- a fifth of the kernel.  Pass 1 is the
    // real one: accumulator -> own shared memory, cluster barrier, then the units of this warp.
    const int q = warp & 3;
    const int ew = (warp - 2) & 3;                       // 0..3 = 32-block of the tile
    const int es = (warp - 2) >> 2;                      // set of epilogue warps
    const int nblocks = d / 32;
    const int blk = ft * 4 + ew;
    float* y_s = reinterpret_cast<float*>(y_tiles + (es * 4 + ew) * C::Y_BYTES);
    const uint32_t r_saddr = smem_u32(ri_tiles + ew * C::RI_BYTES);
    const uint32_t p_saddr = smem_u32(P);
    // lane l adds tokens (l / 8) + 4 j, j = 0..3, features 4 (l % 8) .. + 3 of the block, two tokens at a
    // time: their 2 S loads of 16 bytes go out before the first add, so a unit costs two round trips
    // through the cluster
    const int tr = lane >> 3, fc = (lane & 7) * 4;
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {
      const bool live = pass == 1;
      if (live) {
        // ---- epilogue 1: partial tile -> own shared memory
        acc_ok = mbar_wait(accf_bar, 0, cta_abort, err_word, SITE_EPI_ACC_FULL);
        acc_ok = __all_sync(0xFFFFFFFFu, acc_ok);
        if (acc_ok) {
          tc_fence_after_sync();
          // every load into the stages has landed and every instruction that read them has completed
          const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16);
          float* prow = P + q * 32 + lane;               // feature 32 q + lane of token 0
          for (int c0 = 16 * es; c0 < ntok; c0 += 16 * ESETS) {
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
      // ---- epilogue 2: reduce, intra-rotate, quantize
      uint32_t p_rank[C::MAX_CLUSTER];
#pragma unroll
      for (int s = 0; s < C::MAX_CLUSTER; ++s)
        p_rank[s] = s < S ? map_to_cta(p_saddr, live ? (uint32_t)s : (uint32_t)rank) : 0u;
      for (int g = rank + es * S; g < groups; g += S * ESETS) {
#pragma unroll
        for (int jh = 0; jh < 2; ++jh) {
          if (16 * g + 8 * jh >= M) break;               // rows 8 jh .. 8 jh + 7 of the group hold no token
          float4 part[2][C::MAX_CLUSTER];
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const uint32_t off = (uint32_t)(((16 * g + tr + 4 * (2 * jh + j)) * C::BF + ew * 32 + fc) * 4);
#pragma unroll
            for (int s = 0; s < C::MAX_CLUSTER; ++s)
              if (s < S)
                asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                             : "=f"(part[j][s].x), "=f"(part[j][s].y), "=f"(part[j][s].z), "=f"(part[j][s].w)
                             : "r"(p_rank[s] + off));
          }
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            float4 y = make_float4(0.f, 0.f, 0.f, 0.f);  // rank order: the result does not depend on timing
#pragma unroll
            for (int s = 0; s < C::MAX_CLUSTER; ++s)
              if (s < S) { y.x += part[j][s].x; y.y += part[j][s].y; y.z += part[j][s].z; y.w += part[j][s].w; }
            if (live) {                                  // the y tile lies inside the stages: untouched while they are in use
              float* dst = y_s + (tr + 4 * (2 * jh + j)) * 33 + fc;
              dst[0] = y.x; dst[1] = y.y; dst[2] = y.z; dst[3] = y.w;
            }
          }
        }
        __syncwarp();
        intra_quantize_rows16<FMT>(y_s, r_saddr, R_intra != nullptr, lane, 16 * g, M, blk, d, nblocks, tensor_scale,
                                   codes, scales, live);
        __syncwarp();
      }
    }
    // scale bytes of the rows no unit covers (ntok .. 127 of the single 128-row scale tile): zero
    if (rank == 0 && es == 0) {
      const int row = ew * 32 + lane;
      if (row >= ntok) {
        if constexpr (FMT == FMT_NVFP4) {
          *reinterpret_cast<uint32_t*>(scales + (size_t)(2 * ft) * 512 + (row & 31) * 16 + (row >> 5) * 4) = 0u;
          *reinterpret_cast<uint32_t*>(scales + (size_t)(2 * ft + 1) * 512 + (row & 31) * 16 + (row >> 5) * 4) = 0u;
        } else {
          *reinterpret_cast<uint32_t*>(scales + (size_t)ft * 512 + (row & 31) * 16 + (row >> 5) * 4) = 0u;
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
