// Rotate + quantize (Algorithm 3 steps 1-4): Z = (X . R_inter) then per 32-block Z_b . R_intra[b],
// then MXFP4 (Eq. 1).  The inter-block rotation is a dense bf16 contraction and runs on the
// tcgen05 tensor cores with fp32 accumulators in tensor memory; the rotated activations never
// touch HBM -- the epilogue warps read them from tensor memory one 32-column block per thread,
// apply the 32x32 intra-block rotation in fp32 FMAs (R_intra staged in shared memory as fp32),
// take the block maximum, derive the E8M0 scale, convert to e2m1 and write packed codes plus the
// scale byte in the tiled layout the FP4 GEMM reads.
//
// Persistent, warp-specialised, one CTA per SM:
//   warp 0      TMA producer : X tile [128 x 64] (K-major) and R_inter tile [64 x BN] (N-major,
//                              as BN/64 boxes of 64 x 64), 128-byte swizzle
//   warp 1      MMA issuer   : tcgen05.mma kind::f16 (bf16 x bf16 -> fp32), M=128, N=BN, K=16
//   warps 2..5  epilogue     : one row (token) per thread
// Two accumulator buffers (2 x BN columns) overlap the epilogue with the next tile's mainloop.
#pragma once
#include <cuda_bf16.h>
#include "nvfp4_quantize.cuh"
#include "mxint4_quantize.cuh"
#include "sm100_ptx.cuh"

namespace torq {

template <int BN>
struct RotCfg {
  static constexpr int BM = 128;
  static constexpr int BK = 64;                        // bf16 elements of the contraction per stage
  static constexpr int A_BYTES = BM * BK * 2;          // 16 KiB
  static constexpr int B_BOX_BYTES = 64 * BK * 2;      // one 64(n) x 64(k) box = 8 KiB
  static constexpr int B_BYTES = (BN / 64) * B_BOX_BYTES;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (BN == 256) ? 4 : 6;
  static constexpr int RI_BYTES = (BN / 32) * 32 * 32 * 4;   // fp32 copy of the tile's R_intra blocks
  static constexpr int BAR_BYTES = 256;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + RI_BYTES + BAR_BYTES + 1024;
  static constexpr int NACC = 2;
  static constexpr int TMEM_COLS = (NACC * BN <= 256) ? 256 : 512;
  static constexpr int THREADS = 192;
  static_assert(SMEM_BYTES <= 232448, "shared memory budget");
};

// FMT_NVFP4: NVFP4 quantizer in the epilogue (two 16-element blocks per 32 columns, E4M3 scales,
// `tensor_scale` the tensor's float32 scale; unused for MXFP4).  FMT_MXINT4: integer codes as one
// E4M3 operand byte per element (`codes` is [M, d] bytes), scale bytes as for MXFP4.
// FMT_F32OUT: no quantizer; `codes` is a float32 [M, d] array that receives Z itself.  `x_terms` > 1:
// X = the sum of that many bfloat16 matrices side by side in tmX = [M, x_terms * d], contracted
// against the same R_inter in one fp32 accumulation (d % 64 == 0 then).
template <int BN, int FMT = FMT_MXFP4>
__global__ void __launch_bounds__(192, 1)
rotate_quantize_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmR,
                       const __nv_bfloat16* __restrict__ R_intra, uint8_t* __restrict__ codes,
                       uint8_t* __restrict__ scales, int M, int d, float tensor_scale, int x_terms,
                       int* err_word) {
  using C = RotCfg<BN>;
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
  const int m_tiles = (M + C::BM - 1) / C::BM;
  const int n_tiles = (d + BN - 1) / BN;
  const int total_tiles = m_tiles * n_tiles;
  const int kr_tiles = (d + C::BK - 1) / C::BK;         // K steps over R_inter; X has x_terms times as many
  const int k_tiles = kr_tiles * x_terms;
  const int nblocks = d / 32;
  const int kb4 = (nblocks + 3) / 4;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < C::NACC; ++a) { mbar_init(accf_bar(a), 1); mbar_init(acce_bar(a), 4); }
    *cta_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::TMEM_COLS); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // Set-up above touched no global memory; from here on the previous kernel's results are needed.
  griddep_launch_dependents();
  griddep_wait();

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (elect_one()) { tma_prefetch_desc(&tmX); tma_prefetch_desc(&tmR); }
    uint32_t it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int mt = tile % m_tiles, nt = tile / m_tiles;
      for (int kt = 0, kr = 0; kt < k_tiles; ++kt, ++it, kr = (kr + 1 == kr_tiles ? 0 : kr + 1)) {
        const int s = it % C::STAGES;
        if (!mbar_wait_warp(empty_bar(s), ((it / C::STAGES) & 1) ^ 1, cta_abort, err_word,
                       SITE_PRODUCER_EMPTY)) { ok = false; break; }
        const uint32_t st = smem_base + s * C::STAGE_BYTES;
        if (elect_one()) {
          mbar_arrive_expect_tx(full_bar(s), C::STAGE_BYTES);
          tma_load_2d(st, &tmX, kt * C::BK, mt * C::BM, full_bar(s));
#pragma unroll
          for (int b = 0; b < BN / 64; ++b)
            tma_load_2d(st + C::A_BYTES + b * C::B_BOX_BYTES, &tmR, nt * BN + b * 64, kr * C::BK,
                        full_bar(s));
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    constexpr uint32_t idesc = idesc_bf16(128, BN, /*A MN-major*/ false, /*B MN-major*/ true);
    uint32_t it = 0, tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
      const int a = tcount % C::NACC;
      if (!mbar_wait_warp(acce_bar(a), ((tcount / C::NACC) & 1) ^ 1, cta_abort, err_word,
                     SITE_MMA_ACC_EMPTY)) { ok = false; break; }
      tc_fence_after_sync();
      const uint32_t acc = tmem_base + a * BN;
      for (int kt = 0; kt < k_tiles; ++kt, ++it) {
        const int s = it % C::STAGES;
        if (!mbar_wait_warp(full_bar(s), (it / C::STAGES) & 1, cta_abort, err_word, SITE_MMA_FULL)) {
          ok = false; break;
        }
        tc_fence_after_sync();
        const uint32_t st = smem_base + s * C::STAGE_BYTES;
        // A: K-major, rows of 128 B, 8-row groups 1024 B apart.
        const uint64_t adesc = make_desc(st, 16, 1024, kSwizzle128);
        // B: N-major.  64 n-elements (128 B) contiguous, k rows 128 B apart, 8-row groups
        // 1024 B apart (stride offset), next 64 n-elements one box (8 KiB) further (leading
        // offset).
        const uint64_t bdesc = make_desc(st + C::A_BYTES, C::B_BOX_BYTES, 1024, kSwizzle128);
        if (elect_one()) {
#pragma unroll
          for (int j = 0; j < C::BK / 16; ++j)          // K = 16 per instruction
            mma_bf16(acc, adesc + 2 * j /* 32 B */, bdesc + 128 * j /* 16 k-rows = 2 KiB */, idesc,
                     (kt | j) != 0);
          tc_commit(empty_bar(s));
        }
        __syncwarp();
      }
      if (ok && elect_one()) tc_commit(accf_bar(a));
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------------ epilogue (128 threads)
    const int q = warp & 3;
    const int et = (warp - 2) * 32 + lane;               // 0..127 among the epilogue threads
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++tcount) {
      const int mt = tile % m_tiles, nt = tile / m_tiles;
      const int a = tcount % C::NACC;
      const int b0 = nt * (BN / 32);                     // first 32-block of this tile
      if (R_intra != nullptr) {
        // The two named barriers are executed by every epilogue thread for every tile, also
        // after a wait has given up (ok == false), so that no warp is left behind in one.
        named_barrier_sync(1, 128);                      // everyone is done with the previous copy
        // BN/32 blocks x 1024 bf16 -> fp32, 8 elements per thread per step
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
      if (ok) ok = mbar_wait(accf_bar(a), (tcount / C::NACC) & 1, cta_abort, err_word, SITE_EPI_ACC_FULL);
      ok = __all_sync(0xFFFFFFFFu, ok);                  // keep the warp together on the way out
      if (!ok) continue;
      tc_fence_after_sync();
      const int64_t row = (int64_t)mt * C::BM + q * 32 + lane;
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + a * BN;
      uint32_t sc_word = 0;
      NvScale nvs = {};
      if constexpr (FMT == FMT_NVFP4) nvs = nv_scale(tensor_scale);
#pragma unroll 1
      for (int bb = 0; bb < BN / 32; ++bb) {
        uint32_t yv[32];
        tmem_ld_32x32(tacc + bb * 32, yv);
        tmem_ld_wait();
        if (bb == BN / 32 - 1) {                         // accumulator fully read: hand it back
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(acce_bar(a));
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
              const float4 rv = r[i * 8 + g];            // same address in every lane: broadcast
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
        const int blk = b0 + bb;
        if constexpr (FMT == FMT_F32OUT) {                 // the rotated values themselves
          if (row < M && blk < nblocks) {
            float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(codes) + row * (int64_t)d + (int64_t)blk * 32);
#pragma unroll
            for (int j = 0; j < 8; ++j) dst[j] = make_float4(z[4 * j], z[4 * j + 1], z[4 * j + 2], z[4 * j + 3]);
          }
          continue;
        }
        uint4 cw;
        uint32_t sbyte;
        if constexpr (FMT == FMT_MXINT4) {                 // one operand byte per element
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
        if constexpr (FMT == FMT_NVFP4) {                  // two 16-blocks = half a 4-byte group
          sc_word |= sbyte << (16 * (bb & 1));
          if (bb & 1) {
            const int kb4n = (2 * nblocks + 3) / 4;
            const int chunk = (b0 + bb) >> 1;
            if (chunk < kb4n)
              *reinterpret_cast<uint32_t*>(scales + ((size_t)mt * kb4n + chunk) * 512 + lane * 16 + q * 4) = sc_word;
            sc_word = 0;
          }
          continue;
        }
        sc_word |= sbyte << (8 * (bb & 3));
        if ((bb & 3) == 3) {                             // four K-blocks = one 4-byte group
          const int chunk = (b0 + bb) >> 2;
          if (chunk < kb4)
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
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

}  // namespace torq
