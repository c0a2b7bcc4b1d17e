// Selective speculation support: draft confidence from the logits-row statistics, and the
// batch-level keep-top-(1-alpha) selection.
#pragma once
#include "common.cuh"
#include "sampler.cuh"

namespace spx {

struct ConfParams {
  int32_t batch, total_d, vocab, nsub;
  int64_t row_stride;
  const void *draft;
  const int32_t *draft_ids;   // optional
  const int32_t *q_indptr;
  const float2 *seg_stats;    // [TD][nsub] from the statistics pass over the draft rows
  float *conf_max;            // [TD]
  float *conf_tok;            // [TD], optional
  float *req_conf;            // [B]
  int32_t *dev_status;
};

__device__ __forceinline__ int warp_sum_int(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// One warp per request, lane = draft position.  Top-1 probability = 1 / sum_v 2^(x_v - M) (the
// largest term of the sum is exactly 1), merged from the sub-segment pairs in float64.
template <typename T>
__global__ void __launch_bounds__(128) confidence_kernel(ConfParams p) {
  const int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (r >= p.batch) return;
  const int t0 = p.q_indptr[r];
  const int k = p.q_indptr[r + 1] - t0 - 1;
  const int d0 = t0 - r;
  const float nanf_ = __int_as_float(0x7fc00000);
  if (k < 0 || k > SPX_MAX_K || d0 < 0 || d0 + k > p.total_d) {
    if (lane == 0) {
      atomicOr(p.dev_status, SPX_DEV_BAD_LEN);
      p.req_conf[r] = nanf_;
    }
    return;
  }
  double cmax = 1.0;
  if (lane < k) {
    const float2 *st = p.seg_stats + (int64_t)(d0 + lane) * p.nsub;
    float M = -INFINITY;
    for (int i = 0; i < p.nsub; ++i) M = fmaxf(M, st[i].x);
    double S = 0.0;
    for (int i = 0; i < p.nsub; ++i) S += (double)(st[i].y * fast_exp2(st[i].x - M));
    cmax = 1.0 / S;
    p.conf_max[d0 + lane] = (float)cmax;
    if (p.conf_tok) {
      const int x = p.draft_ids[d0 + lane];
      if (x < 0 || x >= p.vocab) {
        atomicOr(p.dev_status, SPX_DEV_BAD_TOKEN);
        p.conf_tok[d0 + lane] = nanf_;
      } else {
        const double dx = (double)(ld_as_float(reinterpret_cast<const T *>(p.draft), (int64_t)(d0 + lane) * p.row_stride + x) * kLog2e);
        p.conf_tok[d0 + lane] = (float)(exp2(dx - (double)M) / S);
      }
    }
  }
  // product over the request's drafts (lanes >= k contribute 1)
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) cmax *= __shfl_xor_sync(0xffffffffu, cmax, o);
  if (lane == 0) p.req_conf[r] = (float)cmax;
}

// Total order on fp32 bit patterns: -NaN < -inf < ... < -0 < +0 < ... < +inf < +NaN.
__device__ __forceinline__ uint32_t order_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kSelThreads = 1024;

// One block.  Participants are the requests with k_in > 0 (N of them); the n_drop =
// floor(alpha * N) lowest confidences are dropped (k_out = 0), ties going to the higher index
// first.  The n_drop-th smallest key T is found by a 4-pass byte-wise radix select; a request is
// dropped iff its key is below T, or equals T and fewer than (n_drop - #below) equal keys sit at
// higher indices.
__global__ void __launch_bounds__(kSelThreads) select_kernel(int32_t batch, const float *confidence, const int32_t *k_in,
                                                             double alpha, int32_t *k_out, int32_t *n_drop_out,
                                                             int32_t *dev_status) {
  __shared__ int s_hist[256];
  __shared__ int s_warp[kSelThreads / 32];
  __shared__ int s_N, s_bad, s_running;
  __shared__ uint32_t s_prefix;
  __shared__ int s_rank;  // rank still to find inside the current prefix (1-based)
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { s_N = 0; s_bad = 0; }
  __syncthreads();
  int local_n = 0, local_bad = 0;
  for (int r = tid; r < batch; r += kSelThreads) {
    const int k = k_in[r];
    if (k > 0) ++local_n;
    if (k < 0) local_bad = 1;
  }
  local_n = warp_sum_int(local_n);
  if (lane == 0 && local_n) atomicAdd(&s_N, local_n);
  if (local_bad) s_bad = 1;
  __syncthreads();
  const int N = s_N;
  const int n_drop = (int)floor(alpha * (double)N);
  if (tid == 0) {
    if (n_drop_out) *n_drop_out = n_drop;
    if (s_bad) atomicOr(dev_status, SPX_DEV_BAD_LEN);
    s_prefix = 0;
    s_rank = n_drop;
  }
  if (n_drop == 0) {
    for (int r = tid; r < batch; r += kSelThreads) k_out[r] = k_in[r] > 0 ? k_in[r] : 0;
    return;
  }
  if (batch <= kSelThreads) {
    // small batch: rank by counting.  rank(r) = number of participants that are dropped before r
    // (lower key, or equal key at a higher index); r is dropped iff rank(r) < n_drop.
    __shared__ uint32_t s_key[kSelThreads];
    __shared__ int s_part[kSelThreads];
    int k = 0;
    uint32_t key = 0;
    if (tid < batch) {
      k = k_in[tid];
      if (k > 0) key = order_key(confidence[tid]);
      s_key[tid] = key;
      s_part[tid] = k > 0;
    }
    __syncthreads();
    if (tid < batch) {
      int rank = 0;
      for (int j = 0; j < batch; ++j) rank += (s_part[j] && (s_key[j] < key || (s_key[j] == key && j > tid))) ? 1 : 0;
      k_out[tid] = (k > 0 && rank >= n_drop) ? k : 0;
    }
    return;
  }
  // radix select, most significant byte first
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int i = tid; i < 256; i += kSelThreads) s_hist[i] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const uint32_t mask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
    for (int r = tid; r < batch; r += kSelThreads) {
      if (k_in[r] <= 0) continue;
      const uint32_t key = order_key(confidence[r]);
      if ((key & mask) == prefix) atomicAdd(&s_hist[(key >> shift) & 255], 1);
    }
    __syncthreads();
    if (warp == 0) {
      // lane l owns bins 8l..8l+7: exclusive prefix over lanes, then the owner of the crossing bin walks its 8
      int mine = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) mine += s_hist[8 * lane + j];
      int incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int nb = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += nb;
      }
      const int excl = incl - mine;
      const int rank = s_rank;
      if (rank > excl && rank <= incl) {
        int left = rank - excl, b = 8 * lane;
        while (left > s_hist[b]) { left -= s_hist[b]; ++b; }
        s_prefix = prefix | ((uint32_t)b << shift);
        s_rank = left;
      }
    }
    __syncthreads();
  }
  const uint32_t T = s_prefix;
  const int need = s_rank;  // how many of the keys equal to T are dropped (>= 1)
  // suffix counts of keys equal to T, walking the indices downwards in chunks of one block
  if (tid == 0) s_running = 0;
  __syncthreads();
  const int n_chunks = (batch + kSelThreads - 1) / kSelThreads;
  for (int c = n_chunks - 1; c >= 0; --c) {
    const int r = c * kSelThreads + tid;
    int k = 0;
    uint32_t key = 0;
    if (r < batch) {
      k = k_in[r];
      if (k > 0) key = order_key(confidence[r]);
    }
    const bool eq = k > 0 && key == T;
    const uint32_t bal = __ballot_sync(0xffffffffu, eq);
    const int above_in_warp = __popc(bal & (0xfffffffeu << lane));
    if (lane == 0) s_warp[warp] = __popc(bal);
    __syncthreads();
    int above = s_running + above_in_warp;
    for (int w = warp + 1; w < kSelThreads / 32; ++w) above += s_warp[w];
    if (r < batch) {
      int out = k > 0 ? k : 0;
      if (k > 0 && (key < T || (eq && above < need))) out = 0;
      k_out[r] = out;
    }
    __syncthreads();
    if (tid == 0) {
      int tot = 0;
      for (int w = 0; w < kSelThreads / 32; ++w) tot += s_warp[w];
      s_running += tot;
    }
    __syncthreads();
  }
}

}  // namespace spx
