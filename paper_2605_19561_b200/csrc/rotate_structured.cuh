// Rotate + quantize with the rotation in the structure the paper gives it (Section 5, Algorithm 3,
// App. A.7): ONE B x B inter-block matrix R_B that mixes the B = d/32 blocks of a token position
// by position (Y = R_B X on the token's B x 32 reshape) and ONE 32 x 32 intra-block matrix shared
// by all blocks (Z = Y R_intra).  Per token that is 2 d (B + 32) flop instead of 2 d^2: the kernel
// should be bound by reading X and writing the codes, so both steps run on the tcgen05 tensor
// cores and the CUDA cores only split, quantize and store.
//
// Step 2 without moving X: D1[b', (t, k)] = sum_b R_B[b', b] X[b, (t, k)]
//   A operand = R_B tile [128 b' x 64 b], K-major (b contiguous), 2-D TMA, 128-byte swizzle;
//   B operand = X, N-major with the 64-byte swizzle: row b of a token's sub-tile is that token's
//   32 positions of block b (64 contiguous bytes of X).  A 3-D tensor map over X with dimensions
//   (k: 32, stride 1; token: M, stride d; block: B, stride 32) and box (32, 1, 64) lands in shared
//   memory in exactly that layout, one 4 KiB sub-tile per token.  (With the 128-byte swizzle a
//   64-byte inner box row is padded to a 128-byte pitch, so two tokens cannot share a line.)
//   D1 has lanes = output block b' and columns = (token, position).
// Step 3 as a second contraction: D2[b', j] = sum_k y[b', k] R_intra[k, j] per token, with y (fp32,
//   read back from tensor memory) split into three bf16 terms y = hi + mid + lo (to 2^-24) that the
//   epilogue writes to shared memory as K-major A tiles (rows of 64 bytes, 64-byte swizzle), and
//   R_intra (bf16, exact) as the N-major B tile.  Six small MMAs (M 128, N 32, K 16) per token.
//   D2 has lanes = b', 32 columns per token: one thread reads one (token, block) row and runs Eq. 1.
//
// Persistent, warp-specialised: warp 0 TMA producer, warp 1 issues the step-2 MMAs, warp 18 the step-3
// MMAs, warps 2..17 epilogue in four groups of four (lane quarter w % 4; group (w - 2) / 4 owns that
// token of the tile's four): read y from tensor memory, split it, write the terms back to tensor
// memory as the A operand of step 3, wait for the token's six MMAs, read D2, quantize, store.
#pragma once
#include <cuda_bf16.h>
#include "nvfp4_quantize.cuh"
#include "mxint4_quantize.cuh"
#include "sm100_ptx.cuh"

namespace torq {

struct RotStructCfg {
  static constexpr int BM = 128;                       // output blocks b' per tile (MMA M)
  static constexpr int TOK = 4;                        // tokens per tile
  static constexpr int BN = TOK * 32;                  // step-2 MMA N = 128
  static constexpr int BK = 64;                        // input blocks b per stage
  static constexpr int A_BYTES = BM * BK * 2;          // 16 KiB
  static constexpr int B_BOX_BYTES = 32 * BK * 2;      // one token x 64 blocks = 4 KiB
  static constexpr int B_BYTES = TOK * B_BOX_BYTES;    // 16 KiB
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;   // 32 KiB
  static constexpr int STAGES = 6;
  static constexpr int RI_BYTES = 32 * 64;             // R_intra, 64-byte swizzle
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + RI_BYTES + 256 + 1024;
  static constexpr int ACC2_COL = 2 * BN;              // D1 double-buffered in columns [0, 256); D2 in [256, 384)
  static constexpr int LO_COL = ACC2_COL + BN;         // third split term: 16 columns per token, [384, 448)
  static constexpr int TMEM_COLS = 512;
  static constexpr int THREADS = 608;                  // producer, step-2 issuer, 16 epilogue warps, step-3 issuer
  static_assert(SMEM_BYTES <= 232448, "shared memory budget");
};

// tmRB: R_B [B, B] bf16, box [128 x 64], 128-byte swizzle.  tmX3: X as (k, token, block), box (32, 1, 64),
// 64-byte swizzle.
// FMT_NVFP4: the NVFP4 quantizer at the end (two 16-element blocks per row of 32, E4M3 scales,
// `tensor_scale` the tensor's float32 scale; unused for MXFP4); R_intra stays a 32 x 32 matrix (two
// 16 x 16 blocks on its diagonal for a 16-wide intra rotation).  FMT_MXINT4: integer codes as one E4M3
// operand byte per element (`codes` is [M, d] bytes), scale bytes as for MXFP4.
template <int FMT = FMT_MXFP4>
__global__ void __launch_bounds__(608, 1)
rotate_structured_kernel(const __grid_constant__ CUtensorMap tmRB, const __grid_constant__ CUtensorMap tmX3,
                         const __nv_bfloat16* __restrict__ R_intra, uint8_t* __restrict__ codes,
                         uint8_t* __restrict__ scales, int M, int d, float tensor_scale, int* err_word) {
  using C = RotStructCfg;
  constexpr int BN = C::BN;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t ri_base = smem_base + C::STAGES * C::STAGE_BYTES;
  const uint32_t bar_off = C::STAGES * C::STAGE_BYTES + C::RI_BYTES;
  const uint32_t bar_base = smem_base + bar_off;
  // barrier map (8 bytes each)
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (C::STAGES + s); };
  auto acc1f_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + a); };
  auto acc1e_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + 2 + a); };
  auto a2f_bar = [&](int tok) { return bar_base + 8u * (2 * C::STAGES + 4 + tok); };   // epilogue -> MMA
  auto a2d_bar = [&](int tok) { return bar_base + 8u * (2 * C::STAGES + 8 + tok); };   // MMA -> epilogue
  auto d1free_bar = [&](int a) { return bar_base + 8u * (2 * C::STAGES + 12 + a); };   // step 3 of a tile done -> its D1 buffer
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + bar_off + 240);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(smem_gen + bar_off + 248);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nblocks = d / 32;                          // B
  const int b_tiles = (nblocks + C::BM - 1) / C::BM;
  const int t_tiles = (M + C::TOK - 1) / C::TOK;
  const int total_tiles = b_tiles * t_tiles;
  const int k_tiles = (nblocks + C::BK - 1) / C::BK;
  const int kb4 = (nblocks + 3) / 4;
  const bool intra = R_intra != nullptr;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(acc1f_bar(a), 1); mbar_init(acc1e_bar(a), 16); }
    for (int t = 0; t < C::TOK; ++t) { mbar_init(a2f_bar(t), 4); mbar_init(a2d_bar(t), 1); }
    for (int a = 0; a < 2; ++a) mbar_init(d1free_bar(a), 1);
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
    // ------------------------------------------------------------------ step-2 issuer
    constexpr uint32_t idesc1 = idesc_bf16(128, BN, /*A MN-major*/ false, /*B MN-major*/ true);
    uint32_t it = 0;
    bool ok = true;
    // step 2 of tile number `tc` (this CTA's count) into D1 buffer tc % 2
    auto step2 = [&](uint32_t tc) {
      const int a = tc & 1;
      if (!mbar_wait_warp(acc1e_bar(a), ((tc >> 1) & 1) ^ 1, cta_abort, err_word, SITE_MMA_ACC_EMPTY)) {
        ok = false; return;
      }
      // with step 3, the split terms of the tile two back sit in this buffer until its step-3 MMAs
      // (issued by another warp, so not ordered against these by the pipe) have completed
      if (intra && !mbar_wait_warp(d1free_bar(a), ((tc >> 1) & 1) ^ 1, cta_abort, err_word, SITE_MMA_ACC_EMPTY)) {
        ok = false; return;
      }
      tc_fence_after_sync();
      const uint32_t acc = tmem_base + a * BN;
      for (int kt = 0; kt < k_tiles; ++kt, ++it) {
        const int s = it % C::STAGES;
        if (!mbar_wait_warp(full_bar(s), (it / C::STAGES) & 1, cta_abort, err_word, SITE_MMA_FULL)) {
          ok = false; return;
        }
        tc_fence_after_sync();
        const uint32_t st = smem_base + s * C::STAGE_BYTES;
        const uint64_t adesc = make_desc(st, 16, 1024, kSwizzle128);
        // B: N-major, 64-byte swizzle: 32 n-elements (64 B) contiguous, k rows 64 B apart, 8-row
        // groups 512 B apart (stride offset), next 32 n-elements = next token's sub-tile (leading offset)
        const uint64_t bdesc = make_desc(st + C::A_BYTES, C::B_BOX_BYTES, 512, kSwizzle64);
        if (elect_one()) {
#pragma unroll
          for (int j = 0; j < C::BK / 16; ++j)          // 16 k-rows = 1 KiB; steps past the last block are skipped
            if (kt * C::BK + j * 16 < nblocks) mma_bf16(acc, adesc + 2 * j, bdesc + 64 * j, idesc1, (kt | j) != 0);
          tc_commit(empty_bar(s));
        }
        __syncwarp();
      }
      if (elect_one()) tc_commit(acc1f_bar(a));
      __syncwarp();
    };
    uint32_t tcount = 0;
    if (blockIdx.x < (unsigned)total_tiles) step2(0);
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
      if (tile + (int)gridDim.x < total_tiles) step2(tcount + 1);    // next tile's step 2 runs beside this tile's step 3
      if (!ok) break;
    }
  } else if (warp == 18) {
    // ------------------------------------------------------------------ step-3 issuer
    // Its own warp: issuing step 2 of the next tile and step 3 of this one from one thread made that
    // thread's loop the kernel's critical path.
    constexpr uint32_t idesc2 = idesc_bf16(128, 32, /*A MN-major*/ false, /*B MN-major*/ true);
    const uint64_t rdesc = make_desc(ri_base, 2048, 512, kSwizzle64);
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; intra && tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
      for (int tok = 0; tok < C::TOK && ok; ++tok) {
        if (!mbar_wait_warp(a2f_bar(tok), tcount & 1, cta_abort, err_word, SITE_MMA_FULL)) { ok = false; break; }
        tc_fence_after_sync();
        if (elect_one()) {
          const uint32_t d2 = tmem_base + C::ACC2_COL + tok * 32;
          const uint32_t d1 = tmem_base + (tcount & 1) * BN + tok * 32;       // hi, mid: over the token's y
          const uint32_t lo = tmem_base + C::LO_COL + tok * 16;
          mma_bf16_tmem_a(d2, d1, rdesc, idesc2, 0);
          mma_bf16_tmem_a(d2, d1 + 8, rdesc + 64, idesc2, 1);                // k 16..31: +8 columns of A, +16 rows of R
          mma_bf16_tmem_a(d2, d1 + 16, rdesc, idesc2, 1);
          mma_bf16_tmem_a(d2, d1 + 24, rdesc + 64, idesc2, 1);
          mma_bf16_tmem_a(d2, lo, rdesc, idesc2, 1);
          mma_bf16_tmem_a(d2, lo + 8, rdesc + 64, idesc2, 1);
          tc_commit(a2d_bar(tok));
          if (tok == C::TOK - 1) tc_commit(d1free_bar(tcount & 1));
        }
        __syncwarp();
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (four groups of 4 warps)
    // Group g owns token g of every tile; inside a group warp q reads lane quarter q (32 output
    // blocks).  Sixteen warps = four per scheduler: while one group waits for its step-3 MMAs the
    // others split or quantize.  A warp whose 32 rows lie wholly beyond the last block (the second
    // strip of a 160-block layer has 32 real rows of 128) only makes its barrier arrivals.
    const int q = warp & 3;
    const int tok = (warp - 2) >> 2;
    const int et = (warp - 2) * 32 + lane;
    if (intra) {
      // R_intra -> shared memory once: row k = 64 bytes, 16-byte piece c stored at c ^ ((k >> 1) & 3)
      if (et < 128) {
        const int k = et >> 2, c = et & 3;
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(R_intra + k * 32 + c * 8));
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                     ::"r"(ri_base + (uint32_t)k * 64 + (uint32_t)((c ^ ((k >> 1) & 3)) << 4)), "r"(v.x), "r"(v.y),
                       "r"(v.z), "r"(v.w) : "memory");
      }
      fence_proxy_async_smem();                          // visible to the tensor core's reads
      named_barrier_sync(1, 512);
    }
    const int row = q * 32 + lane;                       // b' within the tile = tensor-memory lane
    const uint32_t tlane = tmem_base + ((uint32_t)(q * 32) << 16);
    uint32_t tcount = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
      const int bt = tile % b_tiles, tg = tile / b_tiles;
      const int a = tcount & 1;
      const int blk = bt * C::BM + row;
      const bool live = bt * C::BM + q * 32 < nblocks;   // warp-uniform
      const int64_t token = (int64_t)tg * C::TOK + tok;
      ok = mbar_wait(acc1f_bar(a), (tcount >> 1) & 1, cta_abort, err_word, SITE_EPI_ACC_FULL);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      uint32_t y[32];
      if (live) {
        tmem_ld_32x32(tlane + a * BN + tok * 32, y);
        tmem_ld_wait();
      }
      if (!intra) {                                      // no step 3: D1 is the result
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc1e_bar(a));
      } else {
        // y -> hi + mid + lo bf16, written back to tensor memory as the A operand of step 3 (row b' =
        // lane, two K-elements per column): hi and mid over the token's y, lo in its own columns.  The
        // MMA warp issues step 2 of the tile after next only after this tile's step 3, so D1 is free
        // for it by the order of the tensor pipe; acc1e just counts the warps.
        if (live) {
          uint32_t hi[16], mid[16], lo[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) split3_trunc_bf16x2(y[2 * e], y[2 * e + 1], hi[e], mid[e], lo[e]);
          tmem_st_32x32_x16(tlane + a * BN + tok * 32, hi);
          tmem_st_32x32_x16(tlane + a * BN + tok * 32 + 16, mid);
          tmem_st_32x32_x16(tlane + C::LO_COL + tok * 16, lo);
          tmem_st_wait();
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) { mbar_arrive(acc1e_bar(a)); mbar_arrive(a2f_bar(tok)); }
        ok = mbar_wait(a2d_bar(tok), tcount & 1, cta_abort, err_word, SITE_EPI_ACC_FULL);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        tc_fence_after_sync();
        if (live) {
          tmem_ld_32x32(tlane + C::ACC2_COL + tok * 32, y);
          tmem_ld_wait();
        }
        tc_fence_before_sync();
      }
      if (live) {
        float z[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) z[i] = __uint_as_float(y[i]);
        uint4 cw, cw2;
        uint32_t sbyte;
        if constexpr (FMT == FMT_MXINT4) mxint4_quantize_block32(z, cw, cw2, sbyte);
        else if constexpr (FMT == FMT_NVFP4) nv_quantize_2x16(z, nv_scale(tensor_scale), cw, sbyte);
        else quantize_block32(z, cw, sbyte);
        if (token < M && blk < nblocks) {
          if constexpr (FMT == FMT_MXINT4) {             // one operand byte per element
            uint4* dst = reinterpret_cast<uint4*>(codes + token * (int64_t)d + (int64_t)blk * 32);
            dst[0] = cw;
            dst[1] = cw2;
          } else {
            *reinterpret_cast<uint4*>(codes + token * (int64_t)(d / 2) + (int64_t)blk * 16) = cw;
          }
          if constexpr (FMT == FMT_NVFP4) {              // two scale bytes, adjacent in the tiled layout
            *reinterpret_cast<uint16_t*>(scales + scale_offset(token, 2 * blk, (2 * nblocks + 3) / 4)) = (uint16_t)sbyte;
          } else {
            scales[scale_offset(token, blk, kb4)] = (uint8_t)sbyte;
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
