// Look-ahead memory estimation over future iterations (the paper's Algorithm 1), float64.
#pragma once
#include "common.cuh"

namespace spx {

constexpr int kLookMaxHorizon = 256;   // iterations i = 1..horizon; the paper uses 64
constexpr int kLookThreads = 256;

// grid = horizon (block b handles look-ahead iteration i = b + 1), block = 256 threads.
// The block tabulates, for w = 0..floor(i/pp): k = i - pp w + w generated tokens and
// p = C(k, i - pp w) theta^(i - pp w) (1 - theta)^w, plus the prefix sums of p over w.  k is
// decreasing in w (each rejection costs pp - 1 >= 0 tokens; for pp = 1 it is constant), so
// sum_w [k_w >= tau] p_w is a prefix of the table.  The threads then stride over the requests
// and the block reduces E[N_fin], E[L_fin] and L_total in a fixed order.
__global__ void __launch_bounds__(kLookThreads) lookahead_kernel(int32_t nreq, const int32_t *ell, const int32_t *tau,
                                                                 const double *prec, int32_t pp, double theta, double *M) {
  const int i = blockIdx.x + 1;
  const int w_max = i / pp;
  __shared__ double s_prefix[kLookMaxHorizon + 2];  // s_prefix[c] = sum_{w < c} p_w
  __shared__ double s_egen;
  __shared__ double s_red[3][kLookThreads / 32];
  // one thread per table entry (the powers and the binomial coefficient dominate), then a serial
  // prefix sum in w order
  __shared__ double s_p[kLookMaxHorizon + 1];
  for (int w = threadIdx.x; w <= w_max; w += kLookThreads) {
    const int t = i - pp * w;
    double binom = 1.0;
    for (int j = 1; j <= w; ++j) binom = binom * (double)(t + j) / (double)j;
    s_p[w] = binom * pow(theta, (double)t) * pow(1.0 - theta, (double)w);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double e_gen = 0.0, run = 0.0;
    s_prefix[0] = 0.0;
    for (int w = 0; w <= w_max; ++w) {
      const int k = i - pp * w + w;
      e_gen += (double)k * s_p[w];
      run += s_p[w];
      s_prefix[w + 1] = run;
    }
    s_egen = e_gen;
  }
  __syncthreads();
  double n_fin = 0.0, l_fin = 0.0, l_tot = 0.0;
  for (int r = threadIdx.x; r < nreq; r += kLookThreads) {
    const int tr = tau[r];
    // number of leading table entries with k_w = i - (pp - 1) w >= tau
    int cut = 0;
    if (i >= tr) cut = (pp == 1) ? w_max + 1 : min((i - tr) / (pp - 1) + 1, w_max + 1);
    const double p_fin = prec[r] * s_prefix[cut];
    n_fin += p_fin;
    l_fin += (double)ell[r] * p_fin;
    l_tot += (double)ell[r];
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    n_fin += __shfl_xor_sync(0xffffffffu, n_fin, o);
    l_fin += __shfl_xor_sync(0xffffffffu, l_fin, o);
    l_tot += __shfl_xor_sync(0xffffffffu, l_tot, o);
  }
  if (lane == 0) { s_red[0][warp] = n_fin; s_red[1][warp] = l_fin; s_red[2][warp] = l_tot; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double a = 0.0, b = 0.0, c = 0.0;
    for (int w = 0; w < kLookThreads / 32; ++w) { a += s_red[0][w]; b += s_red[1][w]; c += s_red[2][w]; }
    M[blockIdx.x] = c + ((double)nreq - a) * s_egen - b;
  }
}

}  // namespace spx
