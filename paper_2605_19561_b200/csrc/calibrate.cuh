// Offline calibration of the inter-block rotation (Section 5.1 of the paper): the covariance across
// the blocks of a token, and Algorithm 1, the sequence of Givens rotations that makes its diagonal
// constant.  Not on the inference path: small, float64, and sequential where the method is.
//
// Algorithm 1 as implemented (the printed angle zeroes the off-diagonal entry, which spreads the two
// variances and cannot reach the output the algorithm states; this is the Schur-Horn construction
// instead): c = tr(Sigma) / B; repeat: i = block of largest sigma_ii - c, j = block of smallest
// (ties to the lowest index); stop when both are within eps; rotate in the (i, j) plane by the
// angle that makes sigma_ii = c exactly,
//     t = tan(theta) = (sigma_ii - c) / (sigma_ij + sgn(sigma_ij) sqrt(sigma_ij^2 - (sigma_ii - c)(sigma_jj - c))),
// Sigma <- G^T Sigma G, Q <- G^T Q.  Each rotation settles one block, so there are at most B - 1.
// Every float64 operation is issued unfused (__dmul_rn / __dadd_rn ...), one rounding each, so that
// a host implementation that follows the same steps reproduces the result bit for bit.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace torq {

// Sigma[b, b'] = (1 / (T 32)) sum_t sum_k x[t, b, k] x[t, b', k], float64 accumulation in (t, k) order.
// Grid (ceil(B/16), ceil(B/16)), 256 threads = one 16 x 16 tile of Sigma.
__global__ void __launch_bounds__(256) block_covariance_kernel(const __nv_bfloat16* __restrict__ X, int64_t T,
                                                               int64_t d, double* __restrict__ Sigma) {
  constexpr int TT = 4;                                  // tokens per shared-memory round
  __shared__ float xa[TT][16][33], xb[TT][16][33];       // 33: rows of different blocks fall on different banks
  const int64_t B = d / 32;
  const int bi = threadIdx.x >> 4, bj = threadIdx.x & 15;
  const int64_t b0 = (int64_t)blockIdx.y * 16, c0 = (int64_t)blockIdx.x * 16;
  double acc = 0.0;
  for (int64_t t0 = 0; t0 < T; t0 += TT) {
    for (int e = threadIdx.x; e < TT * 16 * 32; e += 256) {
      const int tt = e >> 9, blk = (e >> 5) & 15, k = e & 31;
      const int64_t t = t0 + tt;
      float va = 0.f, vb = 0.f;
      if (t < T) {
        if (b0 + blk < B) va = __bfloat162float(X[t * d + (b0 + blk) * 32 + k]);
        if (c0 + blk < B) vb = __bfloat162float(X[t * d + (c0 + blk) * 32 + k]);
      }
      xa[tt][blk][k] = va;
      xb[tt][blk][k] = vb;
    }
    __syncthreads();
#pragma unroll
    for (int tt = 0; tt < TT; ++tt)
#pragma unroll 8
      for (int k = 0; k < 32; ++k) acc = fma((double)xa[tt][bi][k], (double)xb[tt][bj][k], acc);   // product exact
    __syncthreads();
  }
  if (b0 + bi < B && c0 + bj < B) Sigma[(b0 + bi) * B + c0 + bj] = __ddiv_rn(acc, (double)(T * 32));
}

// Algorithm 1 on S [B, B] (in: Sigma; out: Q Sigma Q^T) in one CTA.  Q [B, B] float64, optional
// bfloat16 copy Qb (rounded through float32), optional count of rotations.
__global__ void __launch_bounds__(512) givens_equalize_kernel(double* __restrict__ S, int B, double eps,
                                                              double* __restrict__ Q, __nv_bfloat16* __restrict__ Qb,
                                                              int* __restrict__ n_rot_out, int max_rot) {
  __shared__ double s_maxv[16], s_minv[16];
  __shared__ int s_maxi[16], s_mini[16];
  __shared__ double s_c, s_cs, s_sn;
  __shared__ int s_i, s_j, s_stop;
  const int tid = threadIdx.x, nth = blockDim.x, lane = tid & 31, warp = tid >> 5;
  for (int64_t idx = tid; idx < (int64_t)B * B; idx += nth) Q[idx] = (idx / B == idx % B) ? 1.0 : 0.0;
  if (tid == 0) {
    double tr = 0.0;
    for (int b = 0; b < B; ++b) tr = __dadd_rn(tr, S[(int64_t)b * B + b]);     // in index order
    s_c = __ddiv_rn(tr, (double)B);
  }
  __syncthreads();
  const double c = s_c;
  int n = 0;
  while (n < max_rot) {
    // block of largest and of smallest deviation, ties to the lowest index
    double maxv = -1.0e308, minv = 1.0e308;
    int maxi = 0x7FFFFFFF, mini = 0x7FFFFFFF;
    for (int b = tid; b < B; b += nth) {
      const double dev = __dsub_rn(S[(int64_t)b * B + b], c);
      if (dev > maxv) { maxv = dev; maxi = b; }
      if (dev < minv) { minv = dev; mini = b; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double ov = __shfl_xor_sync(0xFFFFFFFFu, maxv, o);
      const int oi = __shfl_xor_sync(0xFFFFFFFFu, maxi, o);
      if (ov > maxv || (ov == maxv && oi < maxi)) { maxv = ov; maxi = oi; }
      const double uv = __shfl_xor_sync(0xFFFFFFFFu, minv, o);
      const int ui = __shfl_xor_sync(0xFFFFFFFFu, mini, o);
      if (uv < minv || (uv == minv && ui < mini)) { minv = uv; mini = ui; }
    }
    if (lane == 0) { s_maxv[warp] = maxv; s_maxi[warp] = maxi; s_minv[warp] = minv; s_mini[warp] = mini; }
    __syncthreads();
    if (tid == 0) {
      for (int w = 1; w < (nth >> 5); ++w) {
        if (s_maxv[w] > maxv || (s_maxv[w] == maxv && s_maxi[w] < maxi)) { maxv = s_maxv[w]; maxi = s_maxi[w]; }
        if (s_minv[w] < minv || (s_minv[w] == minv && s_mini[w] < mini)) { minv = s_minv[w]; mini = s_mini[w]; }
      }
      int stop = 0;
      const double da = maxv, dd = minv;
      if (fmax(da, -dd) <= eps || maxi == mini) stop = 1;
      if (!stop) {
        const double b = S[(int64_t)maxi * B + mini];
        const double disc = __dsub_rn(__dmul_rn(b, b), __dmul_rn(da, dd));
        const double root = __dsqrt_rn(disc);
        const double den = b >= 0.0 ? __dadd_rn(b, root) : __dsub_rn(b, root);
        if (den == 0.0) stop = 1;
        else {
          const double t = __ddiv_rn(da, den);
          const double cs = __ddiv_rn(1.0, __dsqrt_rn(__dadd_rn(1.0, __dmul_rn(t, t))));
          s_cs = cs;
          s_sn = __dmul_rn(t, cs);
        }
      }
      s_i = maxi; s_j = mini; s_stop = stop;
    }
    __syncthreads();
    if (s_stop) break;
    const int i = s_i, j = s_j;
    const double cs = s_cs, sn = s_sn;
    for (int p = tid; p < B; p += nth) {                 // Sigma <- Sigma G (columns i, j)
      const double ci = S[(int64_t)p * B + i], cj = S[(int64_t)p * B + j];
      S[(int64_t)p * B + i] = __dsub_rn(__dmul_rn(ci, cs), __dmul_rn(cj, sn));
      S[(int64_t)p * B + j] = __dadd_rn(__dmul_rn(ci, sn), __dmul_rn(cj, cs));
    }
    __syncthreads();
    for (int q = tid; q < B; q += nth) {                 // Sigma <- G^T Sigma, Q <- G^T Q (rows i, j)
      const double ri = S[(int64_t)i * B + q], rj = S[(int64_t)j * B + q];
      S[(int64_t)i * B + q] = __dsub_rn(__dmul_rn(ri, cs), __dmul_rn(rj, sn));
      S[(int64_t)j * B + q] = __dadd_rn(__dmul_rn(ri, sn), __dmul_rn(rj, cs));
      const double qi = Q[(int64_t)i * B + q], qj = Q[(int64_t)j * B + q];
      Q[(int64_t)i * B + q] = __dsub_rn(__dmul_rn(qi, cs), __dmul_rn(qj, sn));
      Q[(int64_t)j * B + q] = __dadd_rn(__dmul_rn(qi, sn), __dmul_rn(qj, cs));
    }
    __syncthreads();
    ++n;
  }
  __syncthreads();
  if (Qb != nullptr)
    for (int64_t idx = tid; idx < (int64_t)B * B; idx += nth) Qb[idx] = __float2bfloat16_rn(__double2float_rn(Q[idx]));
  if (tid == 0 && n_rot_out != nullptr) *n_rot_out = n;
}

}  // namespace torq
