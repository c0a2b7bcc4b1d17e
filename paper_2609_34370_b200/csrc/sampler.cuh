// Speculative rejection sampling: vocabulary-parallel softmax statistics, sequential accept
// test, residual / bonus inverse-CDF draw.
//
// Every logits row is cut into segments of kSegElems tokens.  Pass 1 (row_stats_kernel, the
// bandwidth-bound kernel) reduces each segment to (max, sum exp(x - max)).  accept_kernel merges
// the segment pairs per row in float64, evaluates p(x)/q(x) for the drafts in order and fixes
// n.  resid_seg_kernel re-reads rows n of the rejecting requests and reduces max(0, p - q) per
// segment.  select_kernel picks the segment by a float64 scan of the segment masses and the
// token by an fp32 scan inside that one segment.
#pragma once
#include "common.cuh"

namespace spx {

constexpr int kSegElems = 8192;       // tokens per segment
constexpr int kSampThreads = 256;
constexpr int kElemsPerThread = kSegElems / kSampThreads;  // 32

struct SampleParams {
  int32_t batch, total_q, total_d, vocab, nseg;
  int64_t row_stride;
  const void *target;
  const void *draft;
  const int32_t *draft_ids;
  const int32_t *q_indptr;
  const float *u_accept;
  const float *u_sample;
  int32_t *accepted_len;
  int32_t *out_tokens;
  float *diag_ratio;
  // workspace
  float2 *seg_stats;   // [(TQ+TD)][nseg]  (max in log2 domain, sum)
  float *seg_resid;    // [B][nseg]        residual mass of each segment of row n (units of 1)
  float4 *req_norm;    // [B]  (Mt, 1/St, Md, 1/Sd) of row n, log2 domain maxima; Md = NaN => bonus
  int32_t *dev_status;
};

// 16-byte vector of logits -> floats, scaled into the log2 domain
template <typename T> struct Vec;
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static __forceinline__ void load(const __nv_bfloat16 *p, float (&f)[8]) {
    const uint4 u = __ldg(reinterpret_cast<const uint4 *>(p));
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16) * kLog2e;
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u) * kLog2e;
    }
  }
};
template <> struct Vec<float> {
  static constexpr int N = 4;
  __device__ static __forceinline__ void load(const float *p, float (&f)[4]) {
    const float4 u = __ldg(reinterpret_cast<const float4 *>(p));
    f[0] = u.x * kLog2e; f[1] = u.y * kLog2e; f[2] = u.z * kLog2e; f[3] = u.w * kLog2e;
  }
};

// Load the kElemsPerThread consecutive tokens [v0, v0+32) of a row that this thread owns into
// x[] (log2 domain); tokens >= vocab become -inf.
template <typename T>
__device__ __forceinline__ void load_thread_span(const T *row, int v0, int vocab, float (&x)[kElemsPerThread]) {
  constexpr int N = Vec<T>::N;
#pragma unroll
  for (int c = 0; c < kElemsPerThread / N; ++c) {
    const int v = v0 + c * N;
    if (v + N <= vocab) {
      float f[N];
      Vec<T>::load(row + v, f);
#pragma unroll
      for (int i = 0; i < N; ++i) x[c * N + i] = f[i];
    } else {
#pragma unroll
      for (int i = 0; i < N; ++i) x[c * N + i] = (v + i < vocab) ? ld_as_float(row, v + i) * kLog2e : -INFINITY;
    }
  }
}

// Merge two (max, sum) pairs.
__device__ __forceinline__ void merge_ms(float &m, float &s, float m2, float s2) {
  const float mn = fmaxf(m, m2);
  if (mn == -INFINITY) { s = 0.f; return; }
  s = s * fast_exp2(m - mn) + s2 * fast_exp2(m2 - mn);
  m = mn;
}

// Pass 1.  grid = (nseg, TQ + TD).  Rows [0,TQ) are target rows, [TQ, TQ+TD) draft rows.
// Threads interleave 16-byte vectors so that a warp reads 512 contiguous bytes per load.
template <typename T>
__global__ void __launch_bounds__(kSampThreads) row_stats_kernel(SampleParams p) {
  constexpr int N = Vec<T>::N;
  constexpr int NV = kElemsPerThread / N;  // vectors per thread
  const int seg = blockIdx.x, row = blockIdx.y;
  const T *base = (row < p.total_q)
                      ? reinterpret_cast<const T *>(p.target) + (int64_t)row * p.row_stride
                      : reinterpret_cast<const T *>(p.draft) + (int64_t)(row - p.total_q) * p.row_stride;
  const int seg0 = seg * kSegElems;
  float x[NV][N];
#pragma unroll
  for (int c = 0; c < NV; ++c) {
    const int v = seg0 + (c * kSampThreads + threadIdx.x) * N;
    if (v + N <= p.vocab) {
      Vec<T>::load(base + v, x[c]);
    } else {
#pragma unroll
      for (int i = 0; i < N; ++i) x[c][i] = (v + i < p.vocab) ? ld_as_float(base, v + i) * kLog2e : -INFINITY;
    }
  }
  float m = -INFINITY;
#pragma unroll
  for (int c = 0; c < NV; ++c)
#pragma unroll
    for (int i = 0; i < N; ++i) m = fmaxf(m, x[c][i]);
  float s = 0.f;
  if (m > -INFINITY) {
#pragma unroll
    for (int c = 0; c < NV; ++c)
#pragma unroll
      for (int i = 0; i < N; ++i) s += fast_exp2(x[c][i] - m);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
    const float s2 = __shfl_xor_sync(0xffffffffu, s, o);
    merge_ms(m, s, m2, s2);
  }
  __shared__ float2 s_w[kSampThreads / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) s_w[warp] = make_float2(m, s);
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < kSampThreads / 32; ++w) merge_ms(m, s, s_w[w].x, s_w[w].y);
    p.seg_stats[(int64_t)row * p.nseg + seg] = make_float2(m, s);
  }
}

// Row normalisers from segment pairs, in float64: returns max M (log2 domain) and S = sum 2^(x-M).
__device__ __forceinline__ void row_norm(const float2 *st, int nseg, float &M, double &S) {
  M = -INFINITY;
  for (int i = 0; i < nseg; ++i) M = fmaxf(M, st[i].x);
  S = 0.0;
  for (int i = 0; i < nseg; ++i) S += (double)st[i].y * exp2((double)st[i].x - (double)M);
}

// One thread per request (the work is k+1 tiny serial steps).  Fixes n, writes accepted_len, the
// accepted ids and the -1 padding; leaves slot n for select_kernel.
template <typename T>
__global__ void accept_kernel(SampleParams p) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= p.batch) return;
  const int t0 = p.q_indptr[r];
  const int k = p.q_indptr[r + 1] - t0 - 1;
  const int d0 = t0 - r;
  const T *target = reinterpret_cast<const T *>(p.target);
  const T *draft = reinterpret_cast<const T *>(p.draft);
  const float nanf_ = __int_as_float(0x7fc00000);
  if (k < 0 || k > SPX_MAX_K || t0 < 0 || t0 + k + 1 > p.total_q) {
    atomicOr(p.dev_status, SPX_DEV_BAD_LEN);
    p.accepted_len[r] = 0;
    p.req_norm[r] = make_float4(nanf_, nanf_, nanf_, -1.f);  // w < 0: skip this request
    return;
  }
  bool bad = false;
  for (int i = 0; i < k; ++i) {
    const int x = p.draft_ids[d0 + i];
    if (x < 0 || x >= p.vocab) bad = true;
    if (p.diag_ratio) p.diag_ratio[d0 + i] = nanf_;
  }
  if (bad) {
    atomicOr(p.dev_status, SPX_DEV_BAD_TOKEN);
    p.accepted_len[r] = 0;
    for (int i = 0; i <= k; ++i) p.out_tokens[t0 + i] = -1;
    p.req_norm[r] = make_float4(nanf_, nanf_, nanf_, -1.f);
    return;
  }
  int n = k;
  float Mt = 0.f, Md = 0.f;
  double St = 1.0, Sd = 1.0;
  for (int i = 0; i < k; ++i) {
    row_norm(p.seg_stats + (int64_t)(t0 + i) * p.nseg, p.nseg, Mt, St);
    row_norm(p.seg_stats + (int64_t)(p.total_q + d0 + i) * p.nseg, p.nseg, Md, Sd);
    const int x = p.draft_ids[d0 + i];
    const double tx = (double)(ld_as_float(target, (int64_t)(t0 + i) * p.row_stride + x) * kLog2e);
    const double dx = (double)(ld_as_float(draft, (int64_t)(d0 + i) * p.row_stride + x) * kLog2e);
    // rho = p(x)/q(x) = 2^(tx-Mt)/St * Sd/2^(dx-Md)
    const double rho = exp2((tx - (double)Mt) - (dx - (double)Md)) * (Sd / St);
    if (p.diag_ratio) p.diag_ratio[d0 + i] = (float)rho;
    if (!((double)p.u_accept[d0 + i] < rho)) { n = i; break; }
  }
  p.accepted_len[r] = n;
  for (int i = 0; i < n; ++i) p.out_tokens[t0 + i] = p.draft_ids[d0 + i];
  for (int i = n + 1; i <= k; ++i) p.out_tokens[t0 + i] = -1;
  if (n < k) {
    p.req_norm[r] = make_float4(Mt, (float)(1.0 / St), Md, (float)(1.0 / Sd));
  } else {
    row_norm(p.seg_stats + (int64_t)(t0 + k) * p.nseg, p.nseg, Mt, St);
    p.req_norm[r] = make_float4(Mt, (float)(1.0 / St), nanf_, 0.f);
  }
}

// Residual mass per segment of row n for rejecting requests.  grid = (nseg, B).
template <typename T>
__global__ void __launch_bounds__(kSampThreads) resid_seg_kernel(SampleParams p) {
  const int seg = blockIdx.x, r = blockIdx.y;
  const float4 nm = p.req_norm[r];
  if (nm.w < 0.f || nm.z != nm.z) return;  // invalid request, or bonus case (segment stats suffice)
  const int t0 = p.q_indptr[r];
  const int n = p.accepted_len[r];
  const T *trow = reinterpret_cast<const T *>(p.target) + (int64_t)(t0 + n) * p.row_stride;
  const T *drow = reinterpret_cast<const T *>(p.draft) + (int64_t)(t0 - r + n) * p.row_stride;
  const int v0 = seg * kSegElems + threadIdx.x * kElemsPerThread;
  float xt[kElemsPerThread], xd[kElemsPerThread];
  load_thread_span(trow, v0, p.vocab, xt);
  load_thread_span(drow, v0, p.vocab, xd);
  float acc = 0.f;
#pragma unroll
  for (int i = 0; i < kElemsPerThread; ++i)
    acc += fmaxf(0.f, fast_exp2(xt[i] - nm.x) * nm.y - fast_exp2(xd[i] - nm.z) * nm.w);
  acc = warp_sum(acc);
  __shared__ float s_w[kSampThreads / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) s_w[warp] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
    for (int w = 0; w < kSampThreads / 32; ++w) tot += s_w[w];
    p.seg_resid[(int64_t)r * p.nseg + seg] = tot;
  }
}

// Final draw.  grid = B, block = 256.  Segment choice in float64, token choice by an fp32 scan of
// the chosen segment (thread t owns tokens [32t, 32t+32) of the segment).
template <typename T>
__global__ void __launch_bounds__(kSampThreads) select_kernel(SampleParams p) {
  const int r = blockIdx.x;
  float4 nm = p.req_norm[r];
  if (nm.w < 0.f) return;
  const bool bonus = (nm.z != nm.z);
  const int t0 = p.q_indptr[r];
  const int n = p.accepted_len[r];
  const float2 *tstats = p.seg_stats + (int64_t)(t0 + n) * p.nseg;
  __shared__ int s_seg;
  __shared__ float s_target;
  __shared__ int s_degenerate;
  __shared__ float s_scan[kSampThreads / 32];
  __shared__ int s_tok;
  if (threadIdx.x == 0) {
    // segment masses (float64), total R, target s*R, first segment whose inclusive sum exceeds it
    double R = 0.0;
    int degenerate = 0;
    if (!bonus) {
      for (int i = 0; i < p.nseg; ++i) R += (double)p.seg_resid[(int64_t)r * p.nseg + i];
      if (!(R > 0.0)) degenerate = 1;
    }
    const bool use_target = bonus || degenerate;
    if (use_target) {
      R = 0.0;
      for (int i = 0; i < p.nseg; ++i) R += (double)tstats[i].y * exp2((double)tstats[i].x - (double)nm.x) * (double)nm.y;
    }
    const double target = (double)p.u_sample[r] * R;
    double cum = 0.0;
    int seg = -1, last_pos = -1;
    double before = 0.0, last_before = 0.0;
    for (int i = 0; i < p.nseg; ++i) {
      const double mass = use_target
                              ? (double)tstats[i].y * exp2((double)tstats[i].x - (double)nm.x) * (double)nm.y
                              : (double)p.seg_resid[(int64_t)r * p.nseg + i];
      if (mass > 0.0) { last_pos = i; last_before = cum; }
      if (cum + mass > target) { seg = i; before = cum; break; }
      cum += mass;
    }
    if (seg < 0) { seg = last_pos; before = last_before; }
    s_seg = seg;
    s_target = (float)(target - before);
    s_degenerate = degenerate;
    if (degenerate) atomicOr(p.dev_status, SPX_DEV_DEGENERATE);
  }
  __syncthreads();
  const int seg = s_seg;
  if (seg < 0) {  // no mass anywhere (cannot happen for finite logits)
    if (threadIdx.x == 0) p.out_tokens[t0 + n] = -1;
    return;
  }
  const bool use_target = bonus || s_degenerate;
  const float target = s_target;
  const T *trow = reinterpret_cast<const T *>(p.target) + (int64_t)(t0 + n) * p.row_stride;
  const T *drow = reinterpret_cast<const T *>(p.draft) + (int64_t)(t0 - r + n) * p.row_stride;
  const int v0 = seg * kSegElems + threadIdx.x * kElemsPerThread;
  float w[kElemsPerThread];
  {
    float xt[kElemsPerThread];
    load_thread_span(trow, v0, p.vocab, xt);
    if (use_target) {
#pragma unroll
      for (int i = 0; i < kElemsPerThread; ++i) w[i] = fast_exp2(xt[i] - nm.x) * nm.y;
    } else {
      float xd[kElemsPerThread];
      load_thread_span(drow, v0, p.vocab, xd);
#pragma unroll
      for (int i = 0; i < kElemsPerThread; ++i)
        w[i] = fmaxf(0.f, fast_exp2(xt[i] - nm.x) * nm.y - fast_exp2(xd[i] - nm.z) * nm.w);
    }
  }
  float tsum = 0.f;
#pragma unroll
  for (int i = 0; i < kElemsPerThread; ++i) tsum += w[i];
  // block exclusive scan of thread sums
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float incl = tsum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const float nb = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += nb;
  }
  if (lane == 31) s_scan[warp] = incl;
  if (threadIdx.x == 0) s_tok = 0x7fffffff;
  __syncthreads();
  float woff = 0.f;
  for (int i = 0; i < warp; ++i) woff += s_scan[i];
  const float excl = woff + incl - tsum;
  // the thread whose span contains the crossing walks it; ties across threads resolve to the
  // smallest token through atomicMin
  if (excl <= target && excl + tsum > target) {
    float cum = excl;
    int tok = -1;
#pragma unroll
    for (int i = 0; i < kElemsPerThread; ++i) {
      cum += w[i];
      if (tok < 0 && cum > target) tok = v0 + i;
    }
    if (tok >= 0) atomicMin(&s_tok, tok);
  }
  __syncthreads();
  if (s_tok == 0x7fffffff) {
    // rounding left no crossing inside the segment: take its last token with positive weight
    __syncthreads();
    if (threadIdx.x == 0) s_tok = -1;
    __syncthreads();
    int last = -1;
#pragma unroll
    for (int i = 0; i < kElemsPerThread; ++i)
      if (w[i] > 0.f) last = v0 + i;
    if (last >= 0) atomicMax(&s_tok, last);
    __syncthreads();
  }
  if (threadIdx.x == 0) p.out_tokens[t0 + n] = s_tok;
}

}  // namespace spx
