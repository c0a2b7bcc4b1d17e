// Cache maintenance around the verify step: append the new positions' K/V into their pages,
// shrink the lengths by the rejected drafts afterwards.
#pragma once
#include "common.cuh"

namespace spx {

constexpr int kRopeMaxHeadDim = 512;  // the rotary path keeps base^(-2i/D) of one head in shared memory

struct KvAppendParams {
  int32_t batch, total_q, Hkv, D, P, log2P, num_pages, max_pages_per_req, elem_size;
  const unsigned char *new_k, *new_v;
  unsigned char *k_cache, *v_cache;
  int64_t stride_page, stride_head, stride_token;  // elements
  const int32_t *block_table, *seq_lens, *q_indptr;
  int32_t *dev_status;
  double rope_base;        // 0: plain copy; > 0: K rows (and q_rows) are rotated to their positions
  unsigned char *q_rows;   // optional [TQ, Hq, D], rotated in place
  int32_t Hq;
};

// Rotary embedding of the pairs (x[i], x[i + D/2]), i = i0 .. i0+N-1, of one head vector at
// absolute position t: angle t * inv_freq[i], inv_freq[i] = base^(-2i/D), in double; results rounded
// double -> binary32 -> element type (round-to-nearest-even each).  lo / hi are the 16-byte vectors
// that hold the pairs' first and second elements.
template <typename T>
__device__ __forceinline__ void rope_vectors(uint4 &lo, uint4 &hi, int i0, int t, const double *inv_freq) {
  constexpr int N = 16 / sizeof(T);
  union U { uint4 q; T e[N]; } a, b;
  a.q = lo; b.q = hi;
#pragma unroll
  for (int u = 0; u < N; ++u) {
    const double ang = (double)t * inv_freq[i0 + u];
    double sn, cs;
    sincos(ang, &sn, &cs);
    const double x0 = (double)ld_as_float(a.e, u), x1 = (double)ld_as_float(b.e, u);
    st_from_float(a.e, u, __double2float_rn(x0 * cs - x1 * sn));
    st_from_float(b.e, u, __double2float_rn(x1 * cs + x0 * sn));
  }
  lo = a.q; hi = b.q;
}

// grid = B, block = 256.  One block copies one request's (k+1) x Hkv rows of D elements, 16 bytes
// per thread and step, K and V.  Pure copy: bound by launch latency at verify-step sizes (a few
// MB), by HBM beyond that.  With a rotary base the K rows (and the caller's query rows, in place)
// are rotated to their absolute positions on the way.
__global__ void __launch_bounds__(256) kv_append_kernel(KvAppendParams p) {
  const int r = blockIdx.x;
  const int q0 = p.q_indptr[r];
  const int m = p.q_indptr[r + 1] - q0;
  const int L = p.seq_lens[r];
  __shared__ int s_page[SPX_MAX_K + 1];
  __shared__ int s_bad;
  if (threadIdx.x == 0) s_bad = 0;
  __syncthreads();
  const bool ok_len = m >= 1 && m <= SPX_MAX_K + 1 && L >= m && q0 >= 0 && q0 + m <= p.total_q &&
                      (((int64_t)L + p.P - 1) >> p.log2P) <= (int64_t)p.max_pages_per_req;
  if (!ok_len) {
    if (threadIdx.x == 0) atomicOr(p.dev_status, SPX_DEV_BAD_LEN);
    return;
  }
  if (threadIdx.x < m) {
    const int t = L - m + threadIdx.x;
    const int page = p.block_table[(int64_t)r * p.max_pages_per_req + (t >> p.log2P)];
    s_page[threadIdx.x] = page;
    if (page < 0 || page >= p.num_pages) s_bad = 1;
  }
  __syncthreads();
  if (s_bad) {
    if (threadIdx.x == 0) atomicOr(p.dev_status, SPX_DEV_BAD_PAGE);
    return;
  }
  const int row_bytes = p.D * p.elem_size;
  const int vec_per_row = row_bytes >> 4;
  const int n_vec = m * p.Hkv * vec_per_row;
  if (p.rope_base > 0.0) {
    __shared__ double s_inv_freq[kRopeMaxHeadDim / 2];
    for (int i = threadIdx.x; i < (p.D >> 1); i += blockDim.x) s_inv_freq[i] = pow(p.rope_base, -2.0 * (double)i / (double)p.D);
    __syncthreads();
    // K: a thread takes one vector of the first half of a head row and its partner in the second
    // half, rotates the pairs and stores both; V is copied; the query rows are rotated in place.
    const int half_vecs = vec_per_row >> 1, elems_per_vec = 16 / p.elem_size;
    const int n_k = m * p.Hkv * half_vecs;
    for (int i = threadIdx.x; i < n_k; i += blockDim.x) {
      const int v = i % half_vecs, jg = i / half_vecs, g = jg % p.Hkv, j = jg / p.Hkv;
      const int t = L - m + j;
      const int64_t src = (((int64_t)(q0 + j) * p.Hkv + g) * p.D) * p.elem_size + (int64_t)v * 16;
      const int64_t dst = ((int64_t)s_page[j] * p.stride_page + (int64_t)g * p.stride_head +
                           (int64_t)(t & (p.P - 1)) * p.stride_token) * p.elem_size + (int64_t)v * 16;
      const int64_t half_bytes = (int64_t)(p.D >> 1) * p.elem_size;
      uint4 lo = __ldg(reinterpret_cast<const uint4 *>(p.new_k + src));
      uint4 hi = __ldg(reinterpret_cast<const uint4 *>(p.new_k + src + half_bytes));
      if (p.elem_size == 2) rope_vectors<__nv_bfloat16>(lo, hi, v * elems_per_vec, t, s_inv_freq);
      else rope_vectors<float>(lo, hi, v * elems_per_vec, t, s_inv_freq);
      *reinterpret_cast<uint4 *>(p.k_cache + dst) = lo;
      *reinterpret_cast<uint4 *>(p.k_cache + dst + half_bytes) = hi;
    }
    for (int i = threadIdx.x; i < n_vec; i += blockDim.x) {
      const int v = i % vec_per_row, jg = i / vec_per_row, g = jg % p.Hkv, j = jg / p.Hkv;
      const int t = L - m + j;
      const int64_t src = (((int64_t)(q0 + j) * p.Hkv + g) * p.D) * p.elem_size + (int64_t)v * 16;
      const int64_t dst = ((int64_t)s_page[j] * p.stride_page + (int64_t)g * p.stride_head +
                           (int64_t)(t & (p.P - 1)) * p.stride_token) * p.elem_size + (int64_t)v * 16;
      *reinterpret_cast<uint4 *>(p.v_cache + dst) = __ldg(reinterpret_cast<const uint4 *>(p.new_v + src));
    }
    if (p.q_rows) {
      const int n_q = m * p.Hq * half_vecs;
      for (int i = threadIdx.x; i < n_q; i += blockDim.x) {
        const int v = i % half_vecs, jh = i / half_vecs, h = jh % p.Hq, j = jh / p.Hq;
        const int t = L - m + j;
        unsigned char *row = p.q_rows + (((int64_t)(q0 + j) * p.Hq + h) * p.D) * p.elem_size + (int64_t)v * 16;
        const int64_t half_bytes = (int64_t)(p.D >> 1) * p.elem_size;
        uint4 lo = *reinterpret_cast<const uint4 *>(row);
        uint4 hi = *reinterpret_cast<const uint4 *>(row + half_bytes);
        if (p.elem_size == 2) rope_vectors<__nv_bfloat16>(lo, hi, v * elems_per_vec, t, s_inv_freq);
        else rope_vectors<float>(lo, hi, v * elems_per_vec, t, s_inv_freq);
        *reinterpret_cast<uint4 *>(row) = lo;
        *reinterpret_cast<uint4 *>(row + half_bytes) = hi;
      }
    }
    return;
  }
  for (int i = threadIdx.x; i < n_vec; i += blockDim.x) {
    const int v = i % vec_per_row, jg = i / vec_per_row, g = jg % p.Hkv, j = jg / p.Hkv;
    const int t = L - m + j;
    const int64_t src = (((int64_t)(q0 + j) * p.Hkv + g) * p.D) * p.elem_size + (int64_t)v * 16;
    const int64_t dst = ((int64_t)s_page[j] * p.stride_page + (int64_t)g * p.stride_head +
                         (int64_t)(t & (p.P - 1)) * p.stride_token) * p.elem_size + (int64_t)v * 16;
    *reinterpret_cast<uint4 *>(p.k_cache + dst) = __ldg(reinterpret_cast<const uint4 *>(p.new_k + src));
    *reinterpret_cast<uint4 *>(p.v_cache + dst) = __ldg(reinterpret_cast<const uint4 *>(p.new_v + src));
  }
}

__global__ void kv_rollback_kernel(int32_t batch, const int32_t *seq_lens, const int32_t *q_indptr,
                                   const int32_t *accepted_len, int32_t *new_seq_lens, int32_t *dev_status) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= batch) return;
  const int k = q_indptr[r + 1] - q_indptr[r] - 1;
  const int n = accepted_len[r];
  const int L = seq_lens[r];
  if (k < 0 || n < 0 || n > k || L < k + 1) {
    atomicOr(dev_status, SPX_DEV_BAD_LEN);
    new_seq_lens[r] = -1;
    return;
  }
  new_seq_lens[r] = L - (k - n);
}

}  // namespace spx
