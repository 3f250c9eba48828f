// Measurement tool, not part of the layer: how fast this GPU's tensor cores execute the block-scaled
// FP4 instruction the GEMM uses (tcgen05.mma cta_group::2 kind::mxf4.block_scale, 256 x 256 x 64 per
// instruction) when nothing else is in the way -- operands already in shared memory (random codes), scale
// factors already in tensor memory, no loads, no epilogue.  One CTA pair per two SMs; the issuing
// warp keeps a few groups of four MMAs in flight, paced by tcgen05.commit on a ring of barriers as
// the real kernel's pipeline is.  The result (flop / time) is the denominator the GEMM's roofline
// fraction is quoted against when no vendor-measured FP4 peak is available.
#pragma once
#include "sm100_ptx.cuh"

namespace torq {

struct Fp4ProbeCfg {
  static constexpr int A_BYTES = 128 * 128;            // 128 rows x 256 e2m1 = 16 KiB
  static constexpr int B_BYTES = 128 * 128;            // this CTA's 128 of the 256 columns
  static constexpr int SF_BYTES = 1024;
  static constexpr int RING = 6;
  static constexpr int SMEM_BYTES = A_BYTES + B_BYTES + SF_BYTES + 256 + 1024;
  static constexpr int THREADS = 128;
};

// `groups` groups of four MMAs per CTA pair (each group = K 256 of a 256 x 256 tile).
__global__ void __launch_bounds__(128, 1) fp4_peak_probe_kernel(int groups, int* err_word) {
  using C = Fp4ProbeCfg;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_off = C::A_BYTES + C::B_BYTES + C::SF_BYTES;
  const uint32_t bar_base = smem_base + bar_off;
  auto ring_bar = [&](int s) { return bar_base + 8u * s; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + bar_off + 192);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(smem_gen + bar_off + 200);
  const int warp = threadIdx.x >> 5;
  const uint32_t rank = cluster_ctarank();

  // operands: pseudo-random e2m1 codes (every 4-bit pattern is a finite value; all-zero operands
  // would draw less power than real data and flatter the clock); scale bytes: 2^-4 .. 2^3
  for (uint32_t i = threadIdx.x * 16; i < (uint32_t)bar_off; i += blockDim.x * 16) {
    uint32_t w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t h = (i + 4 * j + 0x9E3779B9u * (blockIdx.x + 1)) * 2654435761u;
      h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
      w[j] = i < (uint32_t)(C::A_BYTES + C::B_BYTES) ? h : (0x7B7B7B7Bu + (h & 0x07070707u));
    }
    *reinterpret_cast<uint4*>(smem_gen + i) = make_uint4(w[0], w[1], w[2], w[3]);
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < C::RING; ++s) mbar_init(ring_bar(s), 1);
    *cta_abort = 0;
    fence_mbar_init();
  }
  fence_proxy_async_smem();
  if (warp == 1) { tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512); tmem_relinquish_pair(); }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_after_init();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 1 && rank == 0) {
    constexpr uint32_t idesc0 = idesc_mxf4(256, 256, 0, 0), idesc2 = idesc_mxf4(256, 256, 2, 2);
    const uint32_t sfa_t = tmem_base + 256, sfb_t = tmem_base + 264;
    const uint64_t adesc = make_desc(smem_base, 16, 1024, kSwizzle128);
    const uint64_t bdesc = make_desc(smem_base + C::A_BYTES, 16, 1024, kSwizzle128);
    const uint64_t sf_d = make_desc(smem_base + C::A_BYTES + C::B_BYTES, 0, 128, 0);
    if (elect_one()) {                                   // scale factors -> tensor memory, once
      for (int c = 0; c < 6; ++c) tmem_cp_32x128b_warpx4_pair(sfa_t + 4 * c, sf_d + 32 * (c & 1));
    }
    __syncwarp();
    bool ok = true;
    for (int gi = 0; gi < groups && ok; ++gi) {
      const int s = gi % C::RING;
      if (gi >= C::RING &&
          !mbar_wait_warp(ring_bar(s), ((gi / C::RING) & 1) ^ 1, cta_abort, err_word, SITE_MMA_FULL)) {
        ok = false; break;
      }
      if (elect_one()) {
        mma_mxf4_pair(tmem_base, adesc, bdesc, idesc0, sfa_t, sfb_t, gi != 0);
        mma_mxf4_pair(tmem_base, adesc + 2, bdesc + 2, idesc2, sfa_t, sfb_t, 1);
        mma_mxf4_pair(tmem_base, adesc + 4, bdesc + 4, idesc0, sfa_t + 4, sfb_t + 8, 1);
        mma_mxf4_pair(tmem_base, adesc + 6, bdesc + 6, idesc2, sfa_t + 4, sfb_t + 8, 1);
        tc_commit_pair(ring_bar(s), 1);                  // arrives on the leader's barrier only
      }
      __syncwarp();
    }
    // drain: the last commit of every ring slot
    for (int s = 0; s < C::RING && ok; ++s) {
      const int last = ((groups - 1 - s) / C::RING) * C::RING + s;     // last group that used slot s
      if (last >= 0 && last < groups)
        ok = mbar_wait_warp(ring_bar(s), (last / C::RING) & 1, cta_abort, err_word, SITE_TEARDOWN);
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, 512);
  }
}

}  // namespace torq
