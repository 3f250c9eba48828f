// Offline weight side of Algorithm 3 step 5, option B ("weight fusion"): W' = R~^T W with
// R~ = R_inter . blockdiag(R_intra), stored with K = d contiguous, i.e. row n of the stored matrix is
//   W'^T[n, :] = (W^T[n, :] . R_inter) then per 32-block . R_intra[b]
// -- the rotation of Algorithm 3 steps 2-3 applied to the rows of W^T.  The rotation kernels take
// bfloat16 operands; a float32 weight is the exact sum of three bfloat16 numbers (3 x 8 significant
// bits), so W^T is written as three bf16 matrices side by side and the tensor cores contract all three
// against R_inter in one fp32 accumulation: every product is exact, the sum is an fp32 sum of 3 d terms.
#pragma once
#include <cuda_bf16.h>
#include "sm100_ptx.cuh"

namespace torq {

// W [d, N] float32 row-major -> T [N, 3 d] bfloat16: T[n, t d + i] = term t of W[i, n], with
// W = term 0 + term 1 + term 2 exactly (each term the leading eight significant bits of what the
// terms before it left).  32 x 32 tiles through shared memory so that both sides are coalesced.
__global__ void __launch_bounds__(256) transpose_split3_kernel(const float* __restrict__ W, int64_t d, int64_t N,
                                                               __nv_bfloat16* __restrict__ T) {
  __shared__ float tile[32][33];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;              // 32 x 8
  const int64_t tiles_n = (N + 31) / 32, tiles_i = (d + 31) / 32;
  for (int64_t t = blockIdx.x; t < tiles_n * tiles_i; t += gridDim.x) {
    const int64_t n0 = (t % tiles_n) * 32, i0 = (t / tiles_n) * 32;
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int64_t i = i0 + ty + 8 * r, n = n0 + tx;
      tile[ty + 8 * r][tx] = (i < d && n < N) ? W[i * N + n] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int64_t n = n0 + ty + 8 * r, i = i0 + tx;
      if (n < N && i < d) {
        const uint32_t x = __float_as_uint(tile[tx][ty + 8 * r]);
        const uint32_t h = x & 0xFFFF0000u;
        const uint32_t r1 = __float_as_uint(__uint_as_float(x) - __uint_as_float(h));     // exact
        const uint32_t m = r1 & 0xFFFF0000u;
        const uint32_t l = __float_as_uint(__uint_as_float(r1) - __uint_as_float(m));     // exact, <= 8 bits
        unsigned short* row = reinterpret_cast<unsigned short*>(T) + n * 3 * d + i;
        row[0] = (unsigned short)(h >> 16);
        row[d] = (unsigned short)(m >> 16);
        row[2 * d] = (unsigned short)(l >> 16);
      }
    }
  }
}

// max |z| over a float32 array, as the bit pattern of a non-negative float in *out (zeroed by the
// caller beforehand; the order of non-negative floats is the order of their bit patterns).
__global__ void __launch_bounds__(256) absmax_kernel(const float* __restrict__ Z, int64_t n, unsigned int* out) {
  float m = 0.f;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    m = fmaxf(m, fabsf(Z[i]));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  if ((threadIdx.x & 31) == 0 && m > 0.f) atomicMax(out, __float_as_uint(m));
}

}  // namespace torq
