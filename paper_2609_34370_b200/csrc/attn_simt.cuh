// Verify attention in plain fp32 FMA arithmetic (no tensor cores).
//
// This is the kernel for kv_dtype = F32: tensor-core tf32 would round the operands to 10-bit
// mantissas, which does not meet a 1e-4 absolute tolerance, so the fp32 configuration keeps true
// fp32 products.  It executes the same work plan (chunks of 128-token tiles, partials merged by
// combine_kernel; its blocks take the entries through a shared counter rather than by range) as
// the bf16 tensor-core kernel and also accepts bf16 inputs, which the tests
// use to cross-check the two kernels.
#pragma once
#include "common.cuh"

namespace spx {

constexpr int kSimtThreads = 256;
constexpr int kSimtSub = 32;  // tokens per inner step

struct SimtSmem {
  // byte offsets into dynamic shared memory for R packed rows and head dim D
  int q, o, k, v, s, m, l, alpha, page, total;
  __host__ __device__ SimtSmem(int R, int D) {
    int off = 0;
    q = off; off += R * D * 4;
    o = off; off += R * D * 4;
    k = off; off += kSimtSub * (D + 1) * 4;
    v = off; off += kSimtSub * D * 4;
    s = off; off += R * kSimtSub * 4;
    m = off; off += R * 4;
    l = off; off += R * 4;
    alpha = off; off += R * 4;
    page = off; off += kSimtSub * 4;
    total = off;
  }
};

template <typename T, int D>
__global__ void __launch_bounds__(kSimtThreads) attn_simt_kernel(AttnParams p) {
  SPX_TL_SCOPE(kTlAttention);
  // the combine kernel may take its places now (it reads the planner's list, then waits for this
  // kernel to end): its launch then costs nothing behind the last CTA
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ int s_item;
  const SimtSmem lay(p.rows_cap, D);
  float *sQ = reinterpret_cast<float *>(smem_raw + lay.q);
  float *sO = reinterpret_cast<float *>(smem_raw + lay.o);
  float *sK = reinterpret_cast<float *>(smem_raw + lay.k);
  float *sV = reinterpret_cast<float *>(smem_raw + lay.v);
  float *sS = reinterpret_cast<float *>(smem_raw + lay.s);
  float *sM = reinterpret_cast<float *>(smem_raw + lay.m);
  float *sL = reinterpret_cast<float *>(smem_raw + lay.l);
  float *sAlpha = reinterpret_cast<float *>(smem_raw + lay.alpha);
  int *sPage = reinterpret_cast<int *>(smem_raw + lay.page);

  const T *Q = reinterpret_cast<const T *>(p.q);
  const T *Kc = reinterpret_cast<const T *>(p.k_cache);
  const T *Vc = reinterpret_cast<const T *>(p.v_cache);
  T *out = reinterpret_cast<T *>(p.out);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = p.G;
  if (p.hdr->overflow) return;
  const int n_items = p.hdr->n_work;

  for (;;) {
    __syncthreads();
    if (tid == 0) s_item = atomicAdd(&p.hdr->work_counter, 1);
    __syncthreads();
    const int item = s_item;
    if (item >= n_items) break;
    const WorkEntry we = p.work[item];
    const int g = we.g;
    const int r = we.req;
    const int q0 = p.q_indptr[r];
    const int m = p.q_indptr[r + 1] - q0;
    const int L = p.seq_lens[r];
    const int R = m * G;
    const int t_begin = we.tile_begin * kTileTokens;
    const int t_end = min(we.tile_end * kTileTokens, L);
    const int32_t *bt = p.block_table + (int64_t)r * p.max_pages_per_req;

    // stage Q (pre-scaled into the log2 domain), clear O, m, l
    for (int i = tid; i < R * D; i += kSimtThreads) {
      const int row = i / D, d = i % D, j = row / G, hg = row % G;
      sQ[i] = ld_as_float(Q, ((int64_t)(q0 + j) * p.Hq + g * G + hg) * D + d) * p.scale_log2;
      sO[i] = 0.f;
    }
    for (int i = tid; i < R; i += kSimtThreads) { sM[i] = -INFINITY; sL[i] = 0.f; }

    for (int t0 = t_begin; t0 < t_end; t0 += kSimtSub) {
      __syncthreads();
      if (tid < kSimtSub) {
        const int t = t0 + tid;
        int page = -1;
        if (t < t_end) {
          page = bt[t >> p.log2P];
          if (page < 0 || page >= p.num_pages) { page = -1; atomicOr(p.dev_status, SPX_DEV_BAD_PAGE); }
        }
        sPage[tid] = page;
      }
      __syncthreads();
      for (int i = tid; i < kSimtSub * D; i += kSimtThreads) {
        const int tt = i / D, d = i % D;
        const int page = sPage[tt];
        float kv = 0.f, vv = 0.f;
        if (page >= 0) {
          const int64_t a = (int64_t)page * p.stride_page + (int64_t)g * p.stride_head +
                            (int64_t)((t0 + tt) & (p.P - 1)) * p.stride_token + d;
          kv = ld_as_float(Kc, a);
          vv = ld_as_float(Vc, a);
        }
        sK[tt * (D + 1) + d] = kv;
        sV[tt * D + d] = vv;
      }
      __syncthreads();
      // scores: lane = token, warp strides over rows
      for (int row = warp; row < R; row += kSimtThreads / 32) {
        const float *qr = sQ + row * D;
        const float *kr = sK + lane * (D + 1);
        float acc = 0.f;
#pragma unroll 8
        for (int d = 0; d < D; ++d) acc = fmaf(qr[d], kr[d], acc);
        const int t = t0 + lane;
        const int limit = L - m + row / G;
        const bool vis = (t < t_end) && (t <= limit) && (sPage[lane] >= 0);
        const float s = vis ? acc : -INFINITY;
        // online softmax for this row over the 32 tokens of the step
        const float m_old = sM[row];
        const float m_new = fmaxf(m_old, warp_max(s));
        const float pexp = (m_new == -INFINITY) ? 0.f : fast_exp2(s - m_new);
        const float alpha = (m_new == -INFINITY) ? 1.f : fast_exp2(m_old - m_new);
        const float psum = warp_sum(pexp);
        sS[row * kSimtSub + lane] = pexp;
        if (lane == 0) { sM[row] = m_new; sL[row] = sL[row] * alpha + psum; sAlpha[row] = alpha; }
      }
      __syncthreads();
      // O = O * alpha + P V : thread owns column d of a strided set of rows
      for (int i = tid; i < R * D; i += kSimtThreads) {
        const int row = i / D, d = i % D;
        const float *pr = sS + row * kSimtSub;
        float acc = sO[i] * sAlpha[row];
#pragma unroll 8
        for (int tt = 0; tt < kSimtSub; ++tt) acc = fmaf(pr[tt], sV[tt * D + d], acc);
        sO[i] = acc;
      }
    }
    __syncthreads();
    if (we.part_slot < 0) {
      for (int i = tid; i < R * D; i += kSimtThreads) {
        const int row = i / D, d = i % D, j = row / G, hg = row % G;
        st_from_float(out, ((int64_t)(q0 + j) * p.Hq + g * G + hg) * D + d, sO[i] / sL[row]);
      }
      if (p.lse)
        for (int row = tid; row < R; row += kSimtThreads)
          p.lse[(int64_t)(q0 + row / G) * p.Hq + g * G + row % G] = (sM[row] + log2f(sL[row])) * kLn2;
    } else {
      const int64_t slot = (int64_t)we.part_slot * p.rows_cap;
      for (int i = tid; i < R * D; i += kSimtThreads) p.part_o[slot * D + i] = sO[i];
      for (int row = tid; row < R; row += kSimtThreads) p.part_ml[slot + row] = make_float2(sM[row], sL[row]);
    }
  }
}

}  // namespace spx
