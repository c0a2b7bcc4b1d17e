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

constexpr int kPlanMaxCta = 256;  // ranges the planner can cut the tile axis into
// Cost of a pair on the axis the cuts are placed on, in eighths of a tile: its tiles plus a fixed
// part per work entry (the entry's epilogue and the pipeline's restart on a new set of query rows),
// a little larger for pairs of one or two tiles, which leave nothing to overlap it with.  Fitted
// to per-CTA run times of the attention kernel on the Llama-3-8B, Llama-3-70B and mixed-length
// shapes, whose ranges hold 2 to 32 entries: 1.51 us per tile and 0.65 us per entry on all three
// (0.43 tile times), pairs of one or two tiles 0.3 tile times more.
constexpr int kCostPerTile = 8;
__device__ __forceinline__ int plan_entry_cost(int tiles) { return tiles <= 2 ? 5 : 3; }

// One block.  Validates each request's (k+1, L, page count), cuts the tile axis of the valid
// requests' (request, kv head) pairs into n_cta ranges of equal length, lays out partial-result
// slots for the pairs a cut crosses and emits each range's work entries in axis order.
__global__ void __launch_bounds__(1024) plan_kernel(AttnParams p, int n_cta) {
  SPX_TL_SCOPE(kTlPlan);
  __shared__ int s_scratch[32];
  __shared__ int s_total;
  __shared__ int s_cut[kPlanMaxCta + 1];     // cut c: first tile (axis position) of range c
  __shared__ int s_cut_vq[kPlanMaxCta + 1];  // index, among the valid requests' pairs, of the first pair that ends after cut c
  __shared__ int s_cut_in[kPlanMaxCta + 1];  // 1: cut c lies strictly inside that pair
  __shared__ int s_off[kPlanMaxCta + 1];     // work entries of the ranges before c
  __shared__ int s_carry_t, s_carry_v, s_carry_c, s_carry_p, s_carry_l, s_bad;
  // The prefix sums of a batch of up to kPlanSmemReqs requests stay in shared memory: the searches
  // below would otherwise be chains of global loads, each a memory round trip beside the
  // bandwidth-bound kernel that runs while the plan is made (29 us instead of 6 for 64 requests).
  constexpr int kPlanSmemReqs = 1024;
  __shared__ int s_tp[kPlanSmemReqs + 1], s_vp[kPlanSmemReqs + 1], s_cp[kPlanSmemReqs + 1];
  __shared__ int s_q0[kPlanSmemReqs], s_m[kPlanSmemReqs], s_L[kPlanSmemReqs];
  const bool in_smem = p.batch <= kPlanSmemReqs;
  auto tile_prefix = [&](int i) -> int { return in_smem ? s_tp[i] : p.tile_prefix[i]; };
  auto valid_prefix = [&](int i) -> int { return in_smem ? s_vp[i] : p.valid_prefix[i]; };
  auto cost_prefix = [&](int i) -> int { return in_smem ? s_cp[i] : p.cost_prefix[i]; };  // per kv head
  const int tid = threadIdx.x;
  const int Hkv = p.Hkv;
  if (n_cta > kPlanMaxCta) n_cta = kPlanMaxCta;
  if (tid == 0) { s_carry_t = 0; s_carry_v = 0; s_carry_c = 0; s_carry_p = 0; s_carry_l = 0; s_bad = 0; }
  __syncthreads();

  // pass 1: validate; prefix sums of tiles and of valid requests
  for (int base = 0; base < p.batch; base += 1024) {
    const int r = base + tid;
    int tiles = 0;
    if (r < p.batch) {
      const int m = p.q_indptr[r + 1] - p.q_indptr[r];
      const int L = p.seq_lens[r];
      const bool ok = (m >= 1) && (m <= p.max_q_len) && (L >= m) &&
                      (((int64_t)L + p.P - 1) >> p.log2P) <= (int64_t)p.max_pages_per_req &&
                      (p.q_indptr[r] >= 0) && (p.q_indptr[r + 1] <= p.total_q);
      tiles = ok ? (L + kTileTokens - 1) / kTileTokens : 0;
      if (!ok) s_bad = 1;
      p.req_bad[r] = 0;
      if (in_smem) { s_q0[r] = p.q_indptr[r]; s_m[r] = m; s_L[r] = L; }
    }
    const int off_t = block_exclusive_scan_1024(tiles, s_scratch, &s_total) + s_carry_t;
    const int tot_t = s_total;
    const int off_v = block_exclusive_scan_1024(tiles > 0 ? 1 : 0, s_scratch, &s_total) + s_carry_v;
    const int tot_v = s_total;
    const int cost = tiles > 0 ? kCostPerTile * tiles + plan_entry_cost(tiles) : 0;
    const int off_c = block_exclusive_scan_1024(cost, s_scratch, &s_total) + s_carry_c;
    const int tot_c = s_total;
    if (r < p.batch) {
      if (in_smem) { s_tp[r] = off_t; s_vp[r] = off_v; s_cp[r] = off_c; }
      else { p.tile_prefix[r] = off_t; p.valid_prefix[r] = off_v; p.cost_prefix[r] = off_c; }
    }
    __syncthreads();
    if (tid == 0) { s_carry_t += tot_t; s_carry_v += tot_v; s_carry_c += tot_c; }
    __syncthreads();
  }
  if (tid == 0) {
    if (in_smem) { s_tp[p.batch] = s_carry_t; s_vp[p.batch] = s_carry_v; s_cp[p.batch] = s_carry_c; }
    else { p.tile_prefix[p.batch] = s_carry_t; p.valid_prefix[p.batch] = s_carry_v; p.cost_prefix[p.batch] = s_carry_c; }
    if (s_bad) atomicOr(p.dev_status, SPX_DEV_BAD_LEN);
  }
  __syncthreads();  // the prefix arrays are read back below (same block: visible after the barrier)
  const long long total_tiles = s_carry_t;
  const long long T = total_tiles * Hkv;
  const int n_valid_pairs = s_carry_v * Hkv;
  const long long Tw = (long long)s_carry_c * Hkv;  // length of the cost axis
  const bool too_long = T >= (1ll << 30) || s_carry_c >= (1 << 30) || s_carry_c < 0;
  const bool may_split = T >= 2ll * kSnapTiles * n_cta;  // cuts inside pairs are then distinct

  // pass 2: the cuts.  Thread c places cut c at c*T/n_cta, finds the pair it falls in and moves it
  // onto the pair's boundary if it is close to one (always, when the axis is too short to split).
  if (tid <= n_cta && !too_long) {
    int cut, vq, inside = 0;
    if (tid == 0 || T == 0) {
      cut = tid == 0 ? 0 : (int)T; vq = tid == 0 ? 0 : n_valid_pairs;
    } else if (tid == n_cta) {
      cut = (int)T; vq = n_valid_pairs;
    } else {
      // the cut is placed on the cost axis, so that a range of many short pairs gets fewer tiles
      // than a range inside one long pair
      const long long x = (long long)tid * Tw / n_cta;
      // largest r with Hkv * cost_prefix(r) <= x (a request with tiles, since x < Tw)
      int lo = 0, hi = p.batch - 1;
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if ((long long)cost_prefix(mid) * Hkv <= x) lo = mid; else hi = mid - 1;
      }
      const int r = lo;
      const int tp = tile_prefix(r), tiles = tile_prefix(r + 1) - tp;
      const int pair_cost = cost_prefix(r + 1) - cost_prefix(r);
      const int entry_cost = pair_cost - kCostPerTile * tiles;
      const int rel = (int)(x - (long long)cost_prefix(r) * Hkv);
      int g = rel / pair_cost;
      const int offw = rel - g * pair_cost;
      int off = offw < entry_cost ? 0 : (offw - entry_cost) / kCostPerTile;
      if (!may_split || off < kSnapTiles) off = 0;
      else if (tiles - off < kSnapTiles) { off = 0; ++g; }  // onto the end of the pair = the start of the next
      inside = off > 0;
      cut = tp * Hkv + g * tiles + off;
      vq = valid_prefix(r) * Hkv + g;
    }
    s_cut[tid] = cut; s_cut_vq[tid] = vq; s_cut_in[tid] = inside;
  }
  __syncthreads();

  // pass 3: entries per range -> offsets
  int count = 0;
  if (tid < n_cta && !too_long && s_cut[tid + 1] > s_cut[tid]) {
    const int first = s_cut_vq[tid];
    const int last = s_cut_in[tid + 1] ? s_cut_vq[tid + 1] : s_cut_vq[tid + 1] - 1;
    count = last - first + 1;
  }
  const int my_off = block_exclusive_scan_1024(count, s_scratch, &s_total);
  const int n_work_all = s_total;
  if (tid <= n_cta) s_off[tid] = tid < n_cta ? my_off : n_work_all;
  __syncthreads();
  const bool overflow = too_long || n_work_all > p.max_work;
  if (tid <= n_cta) p.cta_off[tid] = overflow ? 0 : s_off[tid];

  // range that holds axis position x: the largest c with cut[c] <= x (ranges before it that
  // start at the same position are empty)
  auto owner = [&](int x) -> int {
    int lo = 0, hi = n_cta - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (s_cut[mid] <= x) lo = mid; else hi = mid - 1;
    }
    return lo;
  };

  // pass 4: one thread per pair: chunk count, partial slots, entries
  const int n_pairs = p.batch * Hkv;
  for (int base = 0; base < n_pairs; base += 1024) {
    const int pair = base + tid;
    const int r = pair / Hkv, g = pair - r * Hkv;
    int tiles = 0, b = 0, c_first = 0, nch = 0;
    if (pair < n_pairs && !overflow) {
      const int tp = tile_prefix(r);
      tiles = tile_prefix(r + 1) - tp;
      if (tiles > 0) {
        b = tp * Hkv + g * tiles;
        c_first = owner(b);
        nch = owner(b + tiles - 1) - c_first + 1;
      }
    }
    const int part = block_exclusive_scan_1024(nch > 1 ? nch : 0, s_scratch, &s_total) + s_carry_p;
    const int tot_p = s_total;
    // the pairs the combine kernel has work for: split ones, and those of invalid requests (sentinel rows)
    const bool listed = pair < n_pairs && nch != 1;
    const int lpos = block_exclusive_scan_1024(listed ? 1 : 0, s_scratch, &s_total) + s_carry_l;
    const int tot_l = s_total;
    if (listed) {
      CombineEntry ce;
      ce.pair = pair; ce.nch = nch; ce.part_base = (nch > 1 && part + nch <= p.max_part_slots) ? part : -1;
      if (in_smem) { ce.q0 = s_q0[r]; ce.m = s_m[r]; }
      else { ce.q0 = p.q_indptr[r]; ce.m = p.q_indptr[r + 1] - ce.q0; }
      ce.pad[0] = ce.pad[1] = ce.pad[2] = 0;
      p.combine_list[lpos] = ce;
    }
    if (pair < n_pairs) {
      const bool split = nch > 1 && part + nch <= p.max_part_slots;
      if (nch > 1 && !split) s_bad = 2;  // cannot happen: at most n_cta - 1 cuts, two slots each
      p.pair_nchunks[pair] = nch;
      p.pair_part_base[pair] = split ? part : -1;
      if (nch > 0) {
        WorkEntry e;
        e.req = r; e.g = g;
        if (in_smem) { e.q0 = s_q0[r]; e.m = s_m[r]; e.L = s_L[r]; }
        else { e.q0 = p.q_indptr[r]; e.m = p.q_indptr[r + 1] - e.q0; e.L = p.seq_lens[r]; }
        const int vq = valid_prefix(r) * Hkv + g;
        for (int j = 0; j < nch; ++j) {
          const int c = c_first + j;
          e.tile_begin = max(s_cut[c], b) - b;
          e.tile_end = min(s_cut[c + 1], b + tiles) - b;
          e.part_slot = split ? part + j : -1;
          const int pos = s_off[c] + (vq - s_cut_vq[c]);
          if (pos >= 0 && pos < p.max_work) p.work[pos] = e;
        }
      }
    }
    __syncthreads();
    if (tid == 0) { s_carry_p += tot_p; s_carry_l += tot_l; }
    __syncthreads();
  }
  // the combine kernel's blocks read their first entry without knowing how long the list is
  if (tid < kCombineListPad && tid >= s_carry_l) {
    CombineEntry ce;
    ce.pair = -1; ce.nch = 1; ce.part_base = -1; ce.q0 = 0; ce.m = 0; ce.pad[0] = ce.pad[1] = ce.pad[2] = 0;
    p.combine_list[tid] = ce;
  }
  if (tid == 0) {
    const bool bad = overflow || s_bad == 2;
    p.hdr->n_work = bad ? 0 : n_work_all;
    p.hdr->n_cta = n_cta;
    p.hdr->n_part_slots = s_carry_p;
    p.hdr->total_tiles = (int)total_tiles;
    p.hdr->work_counter = 0;
    p.hdr->overflow = bad;
    p.hdr->n_combine = s_carry_l;
    if (bad) atomicOr(p.dev_status, SPX_DEV_BAD_LEN);
  }
}

// Merge the chunk partials of split pairs: m* = max_c m_c, l* = sum_c 2^(m_c-m*) l_c,
// O = sum_c 2^(m_c-m*) O_c / l*, LSE = (m* + log2 l*) ln 2.  Also writes the sentinel rows of
// invalid requests.  The planner lists the pairs with such work (a cut of the tile axis makes at
// most one: a hundred or so of the thousands of pairs of a large batch); blocks (b, y) take
// entries b, b + gridDim.x, ... of the list, thread t of block (b, y) the item (row, 4 columns)
// y * 256 + t of a pair - one item per thread, since the items of a thread would run one after
// the other, a memory round trip each - with the chunks walked four at a time so that their loads
// are in flight together.
constexpr int kCombineThreads = 256;
template <typename T>
__global__ void __launch_bounds__(kCombineThreads) combine_kernel(AttnParams p) {
  SPX_TL_SCOPE(kTlCombine);
  // The attention kernel releases this one as its CTAs start, so the blocks are in place, with what
  // the planner left for them in registers, when the attention kernel ends: the length of the list
  // and the block's first entry are read before the wait, the attention kernel's own outputs (the
  // partials, the "bad page id" flags) after it.
  static_assert(sizeof(CombineEntry) == 32, "read as two 16-byte vectors");
  const int n_list = p.hdr->n_combine;
  const int4 first_a = *reinterpret_cast<const int4 *>(p.combine_list + blockIdx.x);   // blockIdx.x < kCombineListPad: always written
  const int first_m = reinterpret_cast<const int32_t *>(p.combine_list + blockIdx.x)[4];
  asm volatile("griddepcontrol.wait;" ::: "memory");  // (no-op without programmatic launch)
  // every request's "bad page id" flag is looked at by one block (the attention kernel sets it while
  // it runs, so the planner's list cannot know): fetched here, used after the list
  const int bid = blockIdx.y * gridDim.x + blockIdx.x, n_blocks = gridDim.x * gridDim.y;
  const int bad_first = bid < p.batch ? p.req_bad[bid] : 0;
  T *out = reinterpret_cast<T *>(p.out);
  const int D = p.D, G = p.G;
  const int vecs = D / 4;
  for (int li = blockIdx.x; li < kCombineListPad || li < n_list; li += gridDim.x) {
    if (li >= kCombineListPad && li >= n_list) break;
    const bool first = li == (int)blockIdx.x;
    const int4 e0 = first ? first_a : *reinterpret_cast<const int4 *>(p.combine_list + li);
    const int pair = e0.x, nch = e0.y, part_base = e0.z, q0 = e0.w;
    if (pair < 0) break;   // past the end of the list
    int m = first ? first_m : reinterpret_cast<const int32_t *>(p.combine_list + li)[4];
    const int r = pair / p.Hkv, g = pair % p.Hkv;
    const int bad = p.req_bad[r];   // set by the attention kernel (a page id out of range); on its way beside the partials
    if (nch == 0) {
      // invalid request (or unusable plan): zero rows, NaN lse; clamp the row range to the tensor
      if (m < 0) m = 0;
      if (m > p.max_q_len) m = p.max_q_len;
      if (q0 < 0 || q0 + m > p.total_q) continue;
      for (int item = blockIdx.y * blockDim.x + threadIdx.x; item < m * G * vecs; item += gridDim.y * blockDim.x) {
        const int row = item / vecs, dv = item % vecs, j = row / G, hg = row % G;
        const int64_t o_idx = ((int64_t)(q0 + j) * p.Hq + g * G + hg) * D + dv * 4;
        for (int i = 0; i < 4; ++i) st_from_float(out, o_idx + i, 0.f);
        if (dv == 0 && p.lse) p.lse[(int64_t)(q0 + j) * p.Hq + g * G + hg] = __int_as_float(0x7fc00000);
      }
      continue;
    }
    if (nch == 1) continue;  // written directly by the attention kernel (not listed; kept for safety)
    const int64_t slot_base = (int64_t)part_base * p.rows_cap;
    const int64_t slot_step = p.rows_cap;
    for (int item = blockIdx.y * blockDim.x + threadIdx.x; item < m * G * vecs; item += gridDim.y * blockDim.x) {
      const int row = item / vecs, dv = item % vecs;
      const int64_t slot0 = slot_base + row;
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
      // a request the attention kernel found a bad page id in gets the sentinel rows instead
      const float inv = bad ? 0.f : 1.f / lstar;
      const int j = row / G, hg = row % G;
      const int64_t o_idx = ((int64_t)(q0 + j) * p.Hq + g * G + hg) * D + dv * 4;
      st_from_float(out, o_idx + 0, bad ? 0.f : acc.x * inv);
      st_from_float(out, o_idx + 1, bad ? 0.f : acc.y * inv);
      st_from_float(out, o_idx + 2, bad ? 0.f : acc.z * inv);
      st_from_float(out, o_idx + 3, bad ? 0.f : acc.w * inv);
      if (dv == 0 && p.lse)
        p.lse[(int64_t)(q0 + j) * p.Hq + g * G + hg] = bad ? __int_as_float(0x7fc00000) : (mstar + log2f(lstar)) * kLn2;
    }
  }
  // sentinel rows (zero output, NaN lse) for every head of a request with a bad page id, whichever
  // of its pairs were split
  for (int r = bid; r < p.batch; r += n_blocks) {
    if (!(r == bid ? bad_first : p.req_bad[r])) continue;
    const int q0 = p.q_indptr[r];
    int m = p.q_indptr[r + 1] - q0;
    if (m < 0) m = 0;
    if (m > p.max_q_len) m = p.max_q_len;
    if (q0 < 0 || q0 + m > p.total_q) continue;
    const int64_t n = (int64_t)m * p.Hq * D, base = (int64_t)q0 * p.Hq * D;
    for (int64_t i = threadIdx.x; i < n; i += blockDim.x) st_from_float(out, base + i, 0.f);
    if (p.lse)
      for (int i = threadIdx.x; i < m * p.Hq; i += blockDim.x) p.lse[(int64_t)q0 * p.Hq + i] = __int_as_float(0x7fc00000);
  }
}

}  // namespace spx
