// Self-test of the bounded waits (no counterpart in the paper).  Every wait inside the tensor-core
// kernels gives up after a time limit, latches TORQ_ERR_TIMEOUT with the id of the wait site in the
// device error word, raises the CTA's abort flag so that the other roles leave their loops, and the
// kernel then drains and returns.  In a healthy run no wait ever runs out, so that path would never
// execute; this kernel makes it execute on purpose and harmlessly: one CTA, two barriers on which
// nothing ever arrives, the same wait functions the real kernels use, a limit chosen by the caller.
//   warp 1 ("consumer") waits on barrier 0 with the given limit: its wait runs out, latches the
//           error word and raises the abort flag;
//   warp 0 ("producer") waits on barrier 1 with the kernels' own long limit: it must leave through
//           the abort flag, long before that limit;
//   then the teardown the real kernels share (sleep when aborted, then exit).
// result[0] = 1 when warp 1's wait gave up by itself, result[1] = 1 when warp 0 left through the
// abort flag, result[2] = nanoseconds warp 0 spent waiting.
#pragma once
#include "sm100_ptx.cuh"

namespace torq {

__global__ void __launch_bounds__(64, 1)
wait_selftest_kernel(unsigned long long limit_ns, int* err_word, unsigned long long* result) {
  __shared__ __align__(8) unsigned long long bars[2];
  __shared__ int abort_flag;
  volatile int* cta_abort = &abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bars[0]), 1);
    mbar_init(smem_u32(&bars[1]), 1);
    abort_flag = 0;
    fence_mbar_init();
  }
  __syncthreads();
  if (warp == 1) {
    const bool ok = mbar_wait_warp(smem_u32(&bars[0]), 0, cta_abort, err_word, SITE_SELFTEST, limit_ns);
    if (lane == 0) result[0] = ok ? 0ull : 1ull;
  } else {
    const unsigned long long t0 = globaltimer_ns();
    const bool ok = mbar_wait_warp(smem_u32(&bars[1]), 0, cta_abort, err_word, SITE_PRODUCER_EMPTY);
    if (lane == 0) {
      result[1] = (!ok && *cta_abort) ? 1ull : 0ull;
      result[2] = globaltimer_ns() - t0;
    }
  }
  __syncthreads();
  if (*cta_abort) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
}

}  // namespace torq
