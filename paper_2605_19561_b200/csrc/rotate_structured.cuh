// Rotate + quantize with the rotation in the structure the paper gives it (Section 5, Algorithm 3,
// App. A.7): ONE B x B inter-block matrix R_B that mixes the B = d/32 blocks of a token position
// by position (Y = R_B X on the token's B x 32 reshape) and ONE 32 x 32 intra-block matrix shared
// by all blocks (Z = Y R_intra).  Per token that is 2 d (B + 32) flop instead of 2 d^2: the kernel
// is bound by reading X and writing the codes, not by the tensor pipe.
//
// Step 2 as a tensor-core contraction without moving X: D[b', (t, k)] = sum_b R_B[b', b] X[b, (t, k)]
//   A operand = R_B tile [128 b' x 64 b], K-major (b contiguous), plain 2-D TMA;
//   B operand = X, N-major with the 64-byte swizzle: row b of a token's sub-tile is that token's
//   32 positions of block b (64 contiguous bytes of X).  A 3-D tensor map over X with dimensions
//   (k: 32, stride 1; token: M, stride d; block: B, stride 32) and box (32, 1, 64) lands in shared
//   memory in exactly that layout, one 4 KiB sub-tile per token.  (With the 128-byte swizzle a
//   64-byte inner box row is padded to a 128-byte pitch, so two tokens cannot share a line.)
// The accumulator then has lanes = output block b' and columns = (token, position): the 32 columns
// of one token are one (token, block) row of step 3, which the epilogue reads in the warp-MMA
// fragment layout, rotates on the warp-level tensor-core path (three bf16 terms of y against
// R_intra, whose fragments stay in registers for the whole kernel) and quantizes (Eq. 1).
//
// Persistent, warp-specialised: warp 0 TMA producer, warp 1 MMA issuer, warps 2..9 epilogue
// (lane quarter w % 4, tokens 4 * ((w - 2) / 4) .. + 3 of the tile's eight).
#pragma once
#include <cuda_bf16.h>
#include "quantize.cuh"
#include "sm100_ptx.cuh"

namespace torq {

struct RotStructCfg {
  static constexpr int BM = 128;                       // output blocks b' per tile (MMA M)
  static constexpr int TOK = 8;                        // tokens per tile
  static constexpr int BN = TOK * 32;                  // MMA N = 256
  static constexpr int BK = 64;                        // input blocks b per stage
  static constexpr int A_BYTES = BM * BK * 2;          // 16 KiB
  static constexpr int B_BOX_BYTES = 32 * BK * 2;      // one token x 64 blocks = 4 KiB
  static constexpr int B_BYTES = TOK * B_BOX_BYTES;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;   // 48 KiB
  static constexpr int STAGES = 4;
  static constexpr int RI_ROW_BYTES = 80;              // 32 bf16 + 16 B pad: conflict-free ldmatrix
  static constexpr int RI_BYTES = 32 * RI_ROW_BYTES;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + RI_BYTES + 256 + 1024;
  static constexpr int NACC = 2;
  static constexpr int TMEM_COLS = 512;
  static constexpr int THREADS = 320;
  static_assert(SMEM_BYTES <= 232448, "shared memory budget");
};

// tmRB: R_B [B, B] bf16, box [128 x 64], 128-byte swizzle.  tmX3: X as (k, token, block), box (32, 1, 64),
// 64-byte swizzle.
__global__ void __launch_bounds__(320, 1)
rotate_structured_kernel(const __grid_constant__ CUtensorMap tmRB, const __grid_constant__ CUtensorMap tmX3,
                         const __nv_bfloat16* __restrict__ R_intra, uint8_t* __restrict__ codes,
                         uint8_t* __restrict__ scales, int M, int d, int* err_word) {
  using C = RotStructCfg;
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
  const int nblocks = d / 32;                          // B
  const int b_tiles = (nblocks + C::BM - 1) / C::BM;
  const int t_tiles = (M + C::TOK - 1) / C::TOK;
  const int total_tiles = b_tiles * t_tiles;
  const int k_tiles = (nblocks + C::BK - 1) / C::BK;
  const int kb4 = (nblocks + 3) / 4;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < C::NACC; ++a) { mbar_init(accf_bar(a), 1); mbar_init(acce_bar(a), 8); }
    *cta_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::TMEM_COLS); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  griddep_launch_dependents();
  griddep_wait();

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (elect_one()) { tma_prefetch_desc(&tmRB); tma_prefetch_desc(&tmX3); }
    uint32_t it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const int bt = tile % b_tiles, tg = tile / b_tiles;
      for (int kt = 0; kt < k_tiles; ++kt, ++it) {
        const int s = it % C::STAGES;
        if (!mbar_wait_warp(empty_bar(s), ((it / C::STAGES) & 1) ^ 1, cta_abort, err_word,
                            SITE_PRODUCER_EMPTY)) { ok = false; break; }
        const uint32_t st = smem_base + s * C::STAGE_BYTES;
        if (elect_one()) {
          mbar_arrive_expect_tx(full_bar(s), C::STAGE_BYTES);
          tma_load_2d(st, &tmRB, kt * C::BK, bt * C::BM, full_bar(s));
#pragma unroll
          for (int j = 0; j < C::TOK; ++j)              // one token per box
            tma_load_3d(st + C::A_BYTES + j * C::B_BOX_BYTES, &tmX3, 0, tg * C::TOK + j, kt * C::BK,
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
        const uint64_t adesc = make_desc(st, 16, 1024, kSwizzle128);
        // B: N-major, 64-byte swizzle: 32 n-elements (64 B) contiguous, k rows 64 B apart, 8-row
        // groups 512 B apart (stride offset), next 32 n-elements = next token's sub-tile (leading offset)
        const uint64_t bdesc = make_desc(st + C::A_BYTES, C::B_BOX_BYTES, 512, kSwizzle64);
        if (elect_one()) {
#pragma unroll
          for (int j = 0; j < C::BK / 16; ++j)          // 16 k-rows = 1 KiB
            mma_bf16(acc, adesc + 2 * j, bdesc + 64 * j, idesc, (kt | j) != 0);
          tc_commit(empty_bar(s));
        }
        __syncwarp();
      }
      if (ok && elect_one()) tc_commit(accf_bar(a));
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------------ epilogue (8 warps)
    const int q = warp & 3;
    const int h = (warp - 2) >> 2;
    const int et = (warp - 2) * 32 + lane;
    const int p = lane & 3, r8 = lane >> 2;
    // R_intra -> shared memory (bf16 rows of 80 bytes) -> B fragments, once
    uint32_t bfrag[2][4][2];
    if (R_intra != nullptr) {
      if (et < 128) {
        const int i = et >> 2, c = (et & 3) * 8;
        *reinterpret_cast<uint4*>(ri_smem + i * C::RI_ROW_BYTES + c * 2) =
            __ldg(reinterpret_cast<const uint4*>(R_intra + i * 32 + c));
      }
      named_barrier_sync(1, 256);
      const uint32_t rb = smem_u32(ri_smem) + (uint32_t)(((lane >> 3) & 1) * 8 + (lane & 7)) * C::RI_ROW_BYTES +
                          (uint32_t)(lane >> 4) * 16;
#pragma unroll
      for (int kc = 0; kc < 2; ++kc)
#pragma unroll
        for (int np = 0; np < 2; ++np)
          ldmatrix_x4_trans(rb + kc * 16 * C::RI_ROW_BYTES + np * 32, bfrag[kc][2 * np][0], bfrag[kc][2 * np][1],
                            bfrag[kc][2 * np + 1][0], bfrag[kc][2 * np + 1][1]);
    }
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
      const int bt = tile % b_tiles, tg = tile / b_tiles;
      const int a = tcount % C::NACC;
      ok = mbar_wait(accf_bar(a), (tcount / C::NACC) & 1, cta_abort, err_word, SITE_EPI_ACC_FULL);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + a * BN + h * 128;
      const int blk_base = bt * C::BM + q * 32 + r8;     // + 16 mh + 8 rh
#pragma unroll 1
      for (int t = 0; t < 4; ++t) {
        const int64_t token = (int64_t)tg * C::TOK + h * 4 + t;
#pragma unroll
        for (int mh = 0; mh < 2; ++mh) {
          uint32_t y[16];
          tmem_ld_16x256b_x4(tacc + ((uint32_t)(16 * mh) << 16) + t * 32, y);
          tmem_ld_wait();
          if (t == 3 && mh == 1) {                       // this warp's share of the accumulator is read
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce_bar(a));
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
            const int blk = blk_base + 16 * mh + 8 * rh;
            if (token < M && blk < nblocks) {
              *reinterpret_cast<uint32_t*>(codes + token * (int64_t)(d / 2) + (int64_t)blk * 16 + 4 * p) = word;
              if (p == 0) scales[scale_offset(token, blk, kb4)] = (uint8_t)sbyte;
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
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

// Padding of the scale tiles (rows M .. next multiple of 128, and K-blocks d/32 .. padded to 4)
// := 0; the main kernel writes only real (token, block) entries.  One thread per padding byte.
__global__ void scale_padding_kernel(uint8_t* __restrict__ scales, int64_t M, int64_t nb) {
  const int64_t kb4 = (nb + 3) / 4, kc = kb4 * 4;
  const int64_t mpad = (M + 127) / 128 * 128;
  const int64_t tail_rows = (mpad - M) * kc;             // whole rows below the last token
  const int64_t total = tail_rows + M * (kc - nb);       // plus the padding K-blocks of real rows
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
    int64_t row, c;
    if (t < tail_rows) { row = M + t / kc; c = t % kc; }
    else { const int64_t u = t - tail_rows; row = u / (kc - nb); c = nb + u % (kc - nb); }
    scales[scale_offset(row, c, kb4)] = 0;
  }
}

}  // namespace torq
