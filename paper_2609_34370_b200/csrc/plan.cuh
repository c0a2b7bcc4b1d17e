// Device-side work planner and split-KV combine for the verify-attention kernels.
#pragma once
#include "common.cuh"

namespace spx {

// Exclusive scan of one int per thread over a 1024-thread block; returns the exclusive prefix and
// writes the block total to *total (shared).  scratch holds 32 ints.
__device__ __forceinline__ int block_exclusive_scan_1024(int v, int *scratch, int *total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  __syncthreads();  // scratch may still be read from a previous call
  if (lane == 31) scratch[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = scratch[lane];
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += n;
    }
    scratch[lane] = wi - w;  // exclusive warp offsets
    if (lane == 31) *total = wi;
  }
  __syncthreads();
  return scratch[warp] + incl - v;
}

// One block.  Validates each request's (k+1, L, page count), sizes the chunks so that roughly
// `target_chunks` (chunk, kv-head) work items exist, lays out partial-result slots for split
// requests and emits the work list ordered by decreasing chunk size.
__global__ void __launch_bounds__(1024) plan_kernel(AttnParams p, int target_chunks) {
  __shared__ int s_scratch[32];
  __shared__ int s_total;
  __shared__ int s_hist[1024];
  __shared__ int s_carry_work, s_carry_part, s_bad;
  const int tid = threadIdx.x;
  if (tid == 0) { s_carry_work = 0; s_carry_part = 0; s_bad = 0; }
  s_hist[tid] = 0;
  __syncthreads();

  // pass 1: validate, tiles per request
  int local_tiles = 0;
  for (int r = tid; r < p.batch; r += 1024) {
    const int m = p.q_indptr[r + 1] - p.q_indptr[r];
    const int L = p.seq_lens[r];
    const bool ok = (m >= 1) && (m <= p.max_q_len) && (L >= m) &&
                    (((int64_t)L + p.P - 1) >> p.log2P) <= (int64_t)p.max_pages_per_req &&
                    (p.q_indptr[r] >= 0) && (p.q_indptr[r + 1] <= p.total_q);
    const int tiles = ok ? (L + kTileTokens - 1) / kTileTokens : 0;
    if (!ok) s_bad = 1;
    p.req_nchunks[r] = tiles;  // tiles for now, chunk count after pass 2
    p.req_bad[r] = 0;
    local_tiles += tiles;
  }
  __syncthreads();
  if (tid == 0 && s_bad) atomicOr(p.dev_status, SPX_DEV_BAD_LEN);
  const int tiles_prefix = block_exclusive_scan_1024(local_tiles, s_scratch, &s_total);
  (void)tiles_prefix;
  const long long total_tiles = s_total;
  int chunk_tiles = (int)((total_tiles * p.Hkv + target_chunks - 1) / target_chunks);
  if (chunk_tiles < 1) chunk_tiles = 1;
  __syncthreads();

  // pass 2: chunk counts, work offsets, partial slots; emit unsorted entries
  int overflow = 0;
  for (int base = 0; base < p.batch; base += 1024) {
    const int r = base + tid;
    const int tiles = (r < p.batch) ? p.req_nchunks[r] : 0;
    const int nch = (tiles + chunk_tiles - 1) / chunk_tiles;
    const int npart = nch > 1 ? nch : 0;
    int tot_w, tot_p;
    const int off_w = block_exclusive_scan_1024(nch, s_scratch, &s_total) + s_carry_work;
    tot_w = s_total;
    const int off_p = block_exclusive_scan_1024(npart, s_scratch, &s_total) + s_carry_part;
    tot_p = s_total;
    if (r < p.batch) {
      p.req_nchunks[r] = nch;
      p.req_part_base[r] = npart ? off_p : -1;
      if (off_w + nch > p.max_work) {
        overflow = 1;
      } else {
        const int q = nch ? tiles / nch : 0, rem = nch ? tiles % nch : 0;
        int tb = 0;
        for (int i = 0; i < nch; ++i) {
          const int sz = q + (i < rem ? 1 : 0);
          WorkEntry e;
          e.req = r; e.tile_begin = tb; e.tile_end = tb + sz; e.part_slot = npart ? off_p + i : -1;
          e.q0 = p.q_indptr[r]; e.m = p.q_indptr[r + 1] - e.q0; e.L = p.seq_lens[r]; e.pad = 0;
          p.work_tmp[off_w + i] = e;
          atomicAdd(&s_hist[1023 - min(sz, 1023)], 1);
          tb += sz;
        }
      }
    }
    __syncthreads();
    if (tid == 0) { s_carry_work += tot_w; s_carry_part += tot_p; }
    __syncthreads();
  }
  if (overflow) s_bad = 2;
  __syncthreads();
  const int n_work = (s_bad == 2) ? 0 : s_carry_work;

  // counting sort by decreasing size
  const int bin_count = s_hist[tid];
  const int bin_off = block_exclusive_scan_1024(bin_count, s_scratch, &s_total);
  s_hist[tid] = bin_off;
  __syncthreads();
  for (int i = tid; i < n_work; i += 1024) {
    const WorkEntry e = p.work_tmp[i];
    const int pos = atomicAdd(&s_hist[1023 - min(e.tile_end - e.tile_begin, 1023)], 1);
    p.work[pos] = e;
  }
  if (tid == 0) {
    p.hdr->n_work = n_work;
    p.hdr->chunk_tiles = chunk_tiles;
    p.hdr->n_part_slots = s_carry_part;
    p.hdr->total_tiles = (int)total_tiles;
    p.hdr->work_counter = 0;
    p.hdr->overflow = (s_bad == 2);
    if (s_bad == 2) atomicOr(p.dev_status, SPX_DEV_BAD_LEN);
  }
}

// Merge the chunk partials of split requests: m* = max_c m_c, l* = sum_c 2^(m_c-m*) l_c,
// O = sum_c 2^(m_c-m*) O_c / l*, LSE = (m* + log2 l*) ln 2.  Also writes the sentinel rows of
// invalid requests.  grid = (B * Hkv, ceil(rows_cap * D/4 / 256)), block = 256: one thread per
// (row, 4 columns), chunks walked four at a time so that their loads are in flight together.
template <typename T>
__global__ void __launch_bounds__(256) combine_kernel(AttnParams p) {
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the attention kernel's partials (no-op without PDL)
  const int r = blockIdx.x / p.Hkv, g = blockIdx.x % p.Hkv;
  const int nch = p.req_nchunks[r];
  const int q0 = p.q_indptr[r];
  int m = p.q_indptr[r + 1] - q0;
  T *out = reinterpret_cast<T *>(p.out);
  const int D = p.D, G = p.G;
  const int vecs = D / 4;
  const int item = blockIdx.y * blockDim.x + threadIdx.x;  // (row, dv)
  if (nch == 0 || p.hdr->overflow || p.req_bad[r]) {
    // invalid request (or unusable plan): zero rows, NaN lse; clamp the row range to the tensor
    if (m < 0) m = 0;
    if (m > p.max_q_len) m = p.max_q_len;
    if (q0 < 0 || q0 + m > p.total_q) return;
    if (item < m * G * vecs) {
      const int row = item / vecs, dv = item % vecs, j = row / G, hg = row % G;
      const int64_t o_idx = ((int64_t)(q0 + j) * p.Hq + g * G + hg) * D + dv * 4;
      for (int i = 0; i < 4; ++i) st_from_float(out, o_idx + i, 0.f);
      if (dv == 0 && p.lse) p.lse[(int64_t)(q0 + j) * p.Hq + g * G + hg] = __int_as_float(0x7fc00000);
    }
    return;
  }
  if (nch == 1) return;  // written directly by the attention kernel
  if (item >= m * G * vecs) return;
  const int row = item / vecs, dv = item % vecs;
  const int64_t slot0 = ((int64_t)p.req_part_base[r] * p.Hkv + g) * p.rows_cap + row;
  const int64_t slot_step = (int64_t)p.Hkv * p.rows_cap;
  float lstar = 0.f, mstar = -INFINITY;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  if (nch <= 4) {
    // the common case: every load of the item is issued at once (one memory round trip)
    float2 ml[4];
    float4 o[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int c = min(u, nch - 1);
      ml[u] = p.part_ml[slot0 + c * slot_step];
      o[u] = *reinterpret_cast<const float4 *>(p.part_o + (slot0 + c * slot_step) * D + dv * 4);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (u < nch) mstar = fmaxf(mstar, ml[u].x);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (u >= nch || ml[u].x == -INFINITY) continue;
      const float w = fast_exp2(ml[u].x - mstar);
      lstar += w * ml[u].y;
      acc.x += w * o[u].x; acc.y += w * o[u].y; acc.z += w * o[u].z; acc.w += w * o[u].w;
    }
  } else {
    for (int c = 0; c < nch; ++c) mstar = fmaxf(mstar, p.part_ml[slot0 + c * slot_step].x);
    for (int c0 = 0; c0 < nch; c0 += 4) {
      float2 ml[4];
      float4 o[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int c = min(c0 + u, nch - 1);
        ml[u] = p.part_ml[slot0 + c * slot_step];
        o[u] = *reinterpret_cast<const float4 *>(p.part_o + (slot0 + c * slot_step) * D + dv * 4);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (c0 + u >= nch || ml[u].x == -INFINITY) continue;
        const float w = fast_exp2(ml[u].x - mstar);
        lstar += w * ml[u].y;
        acc.x += w * o[u].x; acc.y += w * o[u].y; acc.z += w * o[u].z; acc.w += w * o[u].w;
      }
    }
  }
  const float inv = 1.f / lstar;
  const int j = row / G, hg = row % G;
  const int64_t o_idx = ((int64_t)(q0 + j) * p.Hq + g * G + hg) * D + dv * 4;
  st_from_float(out, o_idx + 0, acc.x * inv);
  st_from_float(out, o_idx + 1, acc.y * inv);
  st_from_float(out, o_idx + 2, acc.z * inv);
  st_from_float(out, o_idx + 3, acc.w * inv);
  if (dv == 0 && p.lse) p.lse[(int64_t)(q0 + j) * p.Hq + g * G + hg] = (mstar + log2f(lstar)) * kLn2;
}

}  // namespace spx
