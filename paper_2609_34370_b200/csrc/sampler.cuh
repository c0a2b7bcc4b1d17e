// Speculative rejection sampling: vocabulary-parallel softmax statistics, sequential accept
// test, residual / bonus inverse-CDF draw.
//
// Every logits row is cut into sub-segments of kSubElems tokens, four of which make a segment of
// kSegElems.  Pass 1 (row_stats_kernel, the bandwidth-bound kernel: persistent warps, each with
// the loads of its next sub-segment in flight while it reduces the current one, no block-level
// synchronisation) reduces each sub-segment to (max, sum exp(x - max)).  accept_kernel (one warp per
// request, one lane per row) merges the segment pairs per row, evaluates p(x)/q(x) for the
// drafts in float64 and fixes n.  resid_mass_kernel re-reads rows n of the rejecting requests and
// reduces max(0, p - q) per segment; resid_pick_kernel (one block per request) picks the segment
// by a float64 scan of the segment masses and the token by an fp32 scan inside it.
#pragma once
#include "common.cuh"

namespace spx {

constexpr int kSegElems = 8192;       // tokens per segment (residual pass, final draw)
#ifndef SPX_SUB_ELEMS
#define SPX_SUB_ELEMS 2048
#endif
constexpr int kSubElems = SPX_SUB_ELEMS;  // tokens per sub-segment (statistics pass)
constexpr int kSubPerSeg = kSegElems / kSubElems;
constexpr int kSampThreads = 256;
constexpr int kResidThreads = 256;   // residual kernels
constexpr int kElemsPerThread = kSegElems / kResidThreads;  // 32

struct SampleParams {
  int32_t batch, total_q, total_d, vocab, nseg, nsub;
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
  float2 *seg_stats;   // [(TQ+TD)][nsub]  per sub-segment (max in log2 domain, sum)
  float *seg_resid;    // [B][nseg]        residual mass of each segment of row n (units of 1); kMassPending until its block has written it
  float4 *req_norm;    // [B]  (Mt, 1/St, Md, 1/Sd) of row n, log2 domain maxima; Md = NaN => bonus
  int32_t *dev_status;
  // verification variants (both NULL: temperature 1 everywhere)
  const float *temperature;  // [B]  > 0: sample at that temperature; 0: greedy (NULL with filters: 1)
  float *row_scale;          // [(TQ+TD)] workspace: log2(e)/tau of the row's request; 0 = row not needed
  // top-k / top-p filtering (all NULL unless one of top_k / top_p is given)
  const int32_t *top_k;      // [B]  < 1 or >= vocab: off
  const float *top_p;        // [B]  1: off
  int32_t *row_req;          // [(TQ+TD)] request whose filter applies to the row, -1 = none
  uint32_t *row_thresh;      // [(TQ+TD)] order key of the lowest kept logit (0 = everything kept)
  double *row_z;             // [(TQ+TD)] kept mass sum 2^(x*scale - M); < 0 = unfiltered, use the statistics
  int32_t first_row;         // statistics pass: rows below this one already have their statistics (LM-head epilogue)
  uint2 *req_thresh;         // [B]  thresholds of rows n (target, draft)
  float *seg_pmass;          // [B][nseg] kept target mass of each segment of row n
};

// 16-byte vector of logits -> floats, scaled into the log2 domain
template <typename T> struct Vec;
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static __forceinline__ void load(const __nv_bfloat16 *p, float (&f)[8], float c) {
    const uint4 u = __ldg(reinterpret_cast<const uint4 *>(p));
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16) * c;
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u) * c;
    }
  }
};
template <> struct Vec<float> {
  static constexpr int N = 4;
  __device__ static __forceinline__ void load(const float *p, float (&f)[4], float c) {
    const float4 u = __ldg(reinterpret_cast<const float4 *>(p));
    f[0] = u.x * c; f[1] = u.y * c; f[2] = u.z * c; f[3] = u.w * c;
  }
};

// Element j of a raw 16-byte vector of logits, times scale.
template <typename T>
__device__ __forceinline__ float raw_elem(const uint4 &u, int j, float scale) {
  const int k = sizeof(T) == 2 ? j >> 1 : j;
  const uint32_t w = k == 0 ? u.x : k == 1 ? u.y : k == 2 ? u.z : u.w;
  if (sizeof(T) == 2) return __uint_as_float((j & 1) ? (w & 0xffff0000u) : (w << 16)) * scale;
  return __uint_as_float(w) * scale;
}

// 16-byte asynchronous copy global -> shared.  Used for data only the copying thread reads back:
// cp.async.wait_all orders it, no barrier is needed.
__device__ __forceinline__ void cp_async16(void *smem, const void *gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem) : "memory");
}

// The kElemsPerThread consecutive tokens [v0, v0+32) of a row that a thread owns, kept as raw
// 16-byte vectors and converted token by token (for bf16 logits half the registers of the converted
// values).  get(i, scale) is token v0+i in the log2 domain (logit * scale, scale = log2(e) /
// temperature, or the stored logit with scale 1); tokens >= vocab read as -inf.
template <typename T>
struct RawSpan {
  static constexpr int N = Vec<T>::N, NV = kElemsPerThread / N;
  uint4 raw[NV];
  __device__ __forceinline__ void issue(const T *row, int v0, int vocab) {
#pragma unroll
    for (int c = 0; c < NV; ++c) {
      const int v = v0 + c * N;
      if (v + N <= vocab) {
        raw[c] = __ldg(reinterpret_cast<const uint4 *>(row + v));
      } else {
        union { uint4 u; T e[N]; } tmp;
#pragma unroll
        for (int i = 0; i < N; ++i) {
          if (v + i < vocab) tmp.e[i] = row[v + i];
          else st_from_float(tmp.e, i, -INFINITY);
        }
        raw[c] = tmp.u;
      }
    }
  }
  __device__ __forceinline__ float get(int i, float scale) const { return raw_elem<T>(raw[i / N], i % N, scale); }
};

// Merge two (max, sum) pairs.
__device__ __forceinline__ void merge_ms(float &m, float &s, float m2, float s2) {
  const float mn = fmaxf(m, m2);
  if (mn == -INFINITY) { s = 0.f; return; }
  s = s * fast_exp2(m - mn) + s2 * fast_exp2(m2 - mn);
  m = mn;
}

// The kSubElems / 32 tokens of a sub-segment that a lane owns, as raw 16-byte vectors interleaved
// across the warp (a warp reads 512 contiguous bytes per load).  Vectors that straddle the end of
// the vocabulary are assembled element by element with -inf padding.
template <typename T>
struct SubSlice {
  static constexpr int N = Vec<T>::N;                 // elements per 16-byte vector
  static constexpr int NV = kSubElems / 32 / N;       // vectors per lane
  uint4 raw[NV];
  __device__ __forceinline__ void issue(const T *row_base, int sub, int vocab, int lane) {
#pragma unroll
    for (int c = 0; c < NV; ++c) {
      const int v = sub * kSubElems + (c * 32 + lane) * N;
      if (v + N <= vocab) {
        raw[c] = __ldg(reinterpret_cast<const uint4 *>(row_base + v));
      } else {
        union { uint4 u; T e[N]; } tmp;
#pragma unroll
        for (int i = 0; i < N; ++i) {
          if (v + i < vocab) tmp.e[i] = row_base[v + i];
          else st_from_float(tmp.e, i, -INFINITY);
        }
        raw[c] = tmp.u;
      }
    }
  }
};

// thread-local (max, sum 2^(x*log2e - max)) of a slice; the maximum is returned in the log2 domain.
// Four independent maxima and four independent partial sums keep the dependency chains short
// (the reduction order is fixed, so results do not depend on scheduling).
__device__ __forceinline__ void slice_stats(const SubSlice<__nv_bfloat16> &sl, float &m, float &s, float scale) {
  constexpr int NV = SubSlice<__nv_bfloat16>::NV;
  // packed bf16 maximum: one instruction per two tokens
  __nv_bfloat162 mx[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) mx[i] = *reinterpret_cast<const __nv_bfloat162 *>(&sl.raw[0].x);
#pragma unroll
  for (int c = 0; c < NV; ++c) {
    const uint32_t w[4] = {sl.raw[c].x, sl.raw[c].y, sl.raw[c].z, sl.raw[c].w};
#pragma unroll
    for (int i = 0; i < 4; ++i) mx[i] = __hmax2(mx[i], *reinterpret_cast<const __nv_bfloat162 *>(&w[i]));
  }
  const __nv_bfloat162 mm = __hmax2(__hmax2(mx[0], mx[1]), __hmax2(mx[2], mx[3]));
  m = fmaxf(__low2float(mm), __high2float(mm)) * scale;
  s = 0.f;
  if (m == -INFINITY) return;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int c = 0; c < NV; ++c) {
    const uint32_t w[4] = {sl.raw[c].x, sl.raw[c].y, sl.raw[c].z, sl.raw[c].w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      acc[i] += fast_exp2(fmaf(__uint_as_float(w[i] << 16), scale, -m));
      acc[i] += fast_exp2(fmaf(__uint_as_float(w[i] & 0xffff0000u), scale, -m));
    }
  }
  s = (acc[0] + acc[1]) + (acc[2] + acc[3]);
}
__device__ __forceinline__ void slice_stats(const SubSlice<float> &sl, float &m, float &s, float scale) {
  constexpr int NV = SubSlice<float>::NV;
  float mx = -INFINITY;
#pragma unroll
  for (int c = 0; c < NV; ++c)
    mx = fmaxf(fmaxf(mx, fmaxf(__uint_as_float(sl.raw[c].x), __uint_as_float(sl.raw[c].y))),
               fmaxf(__uint_as_float(sl.raw[c].z), __uint_as_float(sl.raw[c].w)));
  m = mx * scale;
  s = 0.f;
  if (m == -INFINITY) return;
#pragma unroll
  for (int c = 0; c < NV; ++c) {
    s += fast_exp2(fmaf(__uint_as_float(sl.raw[c].x), scale, -m));
    s += fast_exp2(fmaf(__uint_as_float(sl.raw[c].y), scale, -m));
    s += fast_exp2(fmaf(__uint_as_float(sl.raw[c].z), scale, -m));
    s += fast_exp2(fmaf(__uint_as_float(sl.raw[c].w), scale, -m));
  }
}

// Pass 1.  Persistent warps; unit u = row * nsub + sub, rows [0,TQ) target, [TQ,TQ+TD) draft.
// (Skipping the rows after a request's first rejection inside this pass was tried - rows walked
// position-major, completion counters, a steering accept test - and measured slower: the
// bookkeeping cost more than the 22 % of bytes it saved.)
template <typename T, bool kScaled>
__global__ void __launch_bounds__(kSampThreads) row_stats_kernel(SampleParams p, int n_units) {
  SPX_TL_SCOPE(kTlLogitStats);
  const int lane = threadIdx.x & 31;
  const int warp_global = (blockIdx.x * kSampThreads + threadIdx.x) >> 5;
  const int n_warps = (gridDim.x * kSampThreads) >> 5;
  auto row_base = [&](int u) -> const T * {
    const int row = u / p.nsub;
    return (row < p.total_q) ? reinterpret_cast<const T *>(p.target) + (int64_t)row * p.row_stride
                             : reinterpret_cast<const T *>(p.draft) + (int64_t)(row - p.total_q) * p.row_stride;
  };
  // per-row scale of the variants; a scale of 0 marks a row nobody will read (draft rows of greedy
  // requests, rows of requests with an invalid temperature)
  auto row_scale = [&](int u) -> float { return kScaled ? p.row_scale[u / p.nsub] : kLog2e; };
  SubSlice<T> cur, nxt;
  int u = warp_global;
  float sc_cur = kLog2e, sc_nxt = kLog2e;
  if (u < n_units) {
    sc_cur = row_scale(u);
    if (sc_cur != 0.f) cur.issue(row_base(u), u % p.nsub, p.vocab, lane);
  }
  for (; u < n_units; u += n_warps) {
    const int un = u + n_warps;
    if (un < n_units) {
      sc_nxt = row_scale(un);
      if (sc_nxt != 0.f) nxt.issue(row_base(un), un % p.nsub, p.vocab, lane);
    }
    if (sc_cur != 0.f) {
      float m, s;
      slice_stats(cur, m, s, sc_cur);
      // warp merge: one exponential per lane (rescale to the warp maximum), then a plain sum
      const float M = warp_max(m);
      if (M > -INFINITY) s *= fast_exp2(m - M);
      const float S = warp_sum(s);
      if (lane == 0) p.seg_stats[u] = make_float2(M, S);
    }
    cur = nxt;
    sc_cur = sc_nxt;
  }
}

// Pass 1 for bf16 logits, fed by bulk asynchronous copies.  One CTA per SM: a producer thread
// streams 32 KB chunks of logits rows (16384 tokens = 8 sub-segments) into a ring of shared-memory
// stages with cp.async.bulk; eight consumer warps each reduce one sub-segment of every stage.
// 192 KB are in flight per SM whatever the consumers are doing, which the register-prefetching
// kernel above cannot offer (its loads in flight are bounded by its registers).  Same outputs
// (seg_stats layout and values) as row_stats_kernel.
constexpr int kRingStageElems = 16384;
constexpr int kRingStages = 6;
constexpr int kRingConsumerWarps = kRingStageElems / kSubElems;  // 8 warps reduce one stage
#ifndef SPX_RING_GROUPS
#define SPX_RING_GROUPS 3
#endif
constexpr int kRingGroups = SPX_RING_GROUPS;                     // groups of 8 warps, each takes every kRingGroups-th stage
constexpr int kRingThreads = (kRingGroups * kRingConsumerWarps + 1) * 32;
constexpr int kRingSmemBytes = kRingStages * kRingStageElems * 2 + 1024 + 256;
// A stage must always be consumed by the same group: a group then never waits for a phase of a
// stage's barrier that is two phases ahead of the one in flight (a parity wait cannot tell those apart).
static_assert(kRingStages % kRingGroups == 0, "stages per group must be whole");

__device__ __forceinline__ bool ring_wait(uint64_t *bar, uint32_t parity, volatile int *abort, int32_t *dev_status) {
  const uint32_t addr = (uint32_t)__cvta_generic_to_shared(bar);
  const long long t0 = clock64();
  for (;;) {
    for (int i = 0; i < 64; ++i) {
      uint32_t ok;
      asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                   : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
      if (ok) return true;
    }
    if (*abort) return false;
    if (clock64() - t0 > kWaitLimitCycles) {  // about a second: give up, report, let the others leave too
      *abort = 1;
      atomicOr(dev_status, SPX_DEV_TIMEOUT);
      return false;
    }
  }
}

template <bool kScaled>
__global__ void __launch_bounds__(kRingThreads, 1) row_stats_ring_kernel(SampleParams p, int chunks_per_row, int n_chunks) {
  SPX_TL_SCOPE(kTlLogitStats);
  extern __shared__ __align__(1024) unsigned char ring_smem[];
  unsigned char *stages = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(ring_smem) + 1023) & ~uintptr_t(1023));
  uint64_t *full = reinterpret_cast<uint64_t *>(stages + kRingStages * kRingStageElems * 2);
  uint64_t *empty = full + kRingStages;
  volatile int *abort = reinterpret_cast<volatile int *>(empty + kRingStages);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kRingStages; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(&full[s])), "r"(1));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(&empty[s])), "r"(kRingConsumerWarps));
    }
    *abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const __nv_bfloat16 *target = reinterpret_cast<const __nv_bfloat16 *>(p.target);
  const __nv_bfloat16 *draft = reinterpret_cast<const __nv_bfloat16 *>(p.draft);
  auto chunk_src = [&](int g, int &row, int &e0) -> const __nv_bfloat16 * {
    row = p.first_row + g / chunks_per_row;
    e0 = (g % chunks_per_row) * kRingStageElems;
    const __nv_bfloat16 *base = row < p.total_q ? target + (int64_t)row * p.row_stride
                                                : draft + (int64_t)(row - p.total_q) * p.row_stride;
    return base + e0;
  };
  if (warp == kRingGroups * kRingConsumerWarps) {
    // ---- producer (one thread)
    if (lane == 0) {
      int i = 0;
      // the scale of the next chunk's row is fetched one iteration ahead, off the issue path
      float sc_next = (kScaled && (int)blockIdx.x < n_chunks) ? p.row_scale[p.first_row + blockIdx.x / chunks_per_row] : 1.f;
      for (int g = blockIdx.x; g < n_chunks; g += gridDim.x, ++i) {
        const float sc = sc_next;
        if (kScaled && g + (int)gridDim.x < n_chunks) sc_next = p.row_scale[p.first_row + (g + gridDim.x) / chunks_per_row];
        const int s = i % kRingStages;
        if (i >= kRingStages && !ring_wait(&empty[s], ((i / kRingStages) - 1) & 1, abort, p.dev_status)) break;
        int row, e0;
        const __nv_bfloat16 *src = chunk_src(g, row, e0);
        const int elems = min(kRingStageElems, p.vocab - e0);
        const uint32_t bytes = (uint32_t)((elems * 2 + 15) & ~15);  // stays inside the row: its stride is a multiple of 16 bytes
        const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&full[s]);
        if (kScaled && sc == 0.f) {
          // a row nobody will read: hand the stage over empty, the consumers release it at once
          asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
          continue;
        }
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"((uint32_t)__cvta_generic_to_shared(stages + (size_t)s * kRingStageElems * 2)), "l"(src), "r"(bytes), "r"(bar)
                     : "memory");
      }
    }
  } else {
    // ---- consumers: group `grp` takes chunks grp, grp + kRingGroups, ...; its warp w reduces
    // sub-segment w of each of them
    const int grp = warp / kRingConsumerWarps;
    const int wsub = warp % kRingConsumerWarps;
    int i = grp;
    for (int g = blockIdx.x + grp * gridDim.x; g < n_chunks; g += kRingGroups * gridDim.x, i += kRingGroups) {
      const int s = i % kRingStages;
      int row, e0;
      chunk_src(g, row, e0);
      const float scale = kScaled ? p.row_scale[row] : kLog2e;  // in flight while the stage fills
      const bool ok = __all_sync(0xffffffffu, ring_wait(&full[s], (i / kRingStages) & 1, abort, p.dev_status));
      if (!ok) break;
      const int v_sub = e0 + wsub * kSubElems;  // first token of this warp's sub-segment
      if (v_sub < p.vocab && scale != 0.f) {
        SubSlice<__nv_bfloat16> sl;
        const uint4 *src = reinterpret_cast<const uint4 *>(stages + (size_t)s * kRingStageElems * 2 + (size_t)wsub * kSubElems * 2);
#pragma unroll
        for (int c = 0; c < SubSlice<__nv_bfloat16>::NV; ++c) {
          uint4 v = src[c * 32 + lane];
          const int tok = v_sub + (c * 32 + lane) * 8;
          if (tok + 8 > p.vocab) {
            // tokens past the vocabulary (never copied, or the row's padding): -inf
            uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              if (tok + 2 * j >= p.vocab) w[j] = (w[j] & 0xffff0000u) | 0xff80u;
              if (tok + 2 * j + 1 >= p.vocab) w[j] = (w[j] & 0x0000ffffu) | 0xff800000u;
            }
            v = make_uint4(w[0], w[1], w[2], w[3]);
          }
          sl.raw[c] = v;
        }
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"((uint32_t)__cvta_generic_to_shared(&empty[s])) : "memory");
        float m, sum;
        slice_stats(sl, m, sum, scale);
        const float M = warp_max(m);
        if (M > -INFINITY) sum *= fast_exp2(m - M);
        const float S = warp_sum(sum);
        if (lane == 0) p.seg_stats[(int64_t)row * p.nsub + (v_sub / kSubElems)] = make_float2(M, S);
      } else {
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"((uint32_t)__cvta_generic_to_shared(&empty[s])) : "memory");
      }
    }
  }
}

// Total order on fp32 bit patterns, as an unsigned key (larger logit -> larger key).
__device__ __forceinline__ uint32_t order_key32(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// top-k / top-p thresholds of one logits row per block (kFilterThreads threads).
//
// bf16 rows are settled by one histogram of counts over their exact 16-bit keys (see the kernel);
// what follows is the general way, which fp32 rows take, and bf16 rows with values outside that
// histogram's range.
//
// The kept set is {v : key(x_v) >= T}.  T is found by a descent from the top, level by level; each
// level is a 256-bin histogram (count, mass) of the elements still in play, and warp 0 picks the
// bin where the running count reaches top_k, or the running mass reaches top_p times the survivors'
// mass.
//   Level 0 sweeps the whole row and bins every element by its distance below the row maximum in
//   logit units, 1/8 unit per bin (bin = 255 - min(255, floor(8 (max - x))), monotone in x).  The
//   leading byte of a float is the same for almost every logit of a row, so a histogram on key
//   bytes would serialise the shared-memory atomics on a handful of addresses; the distance spreads
//   a row over dozens of bins, and every lane of a warp owns its own copy of the histogram
//   (hist[bin][lane]: one bank per lane, no replays inside a warp).  A mass is added as three
//   15-bit pieces with 32-bit atomics (a copy sees at most vocab/32 elements, no piece overflows;
//   64-bit shared-memory atomics are far slower).  Counts are kept only for a top-k descent,
//   masses only for a top-p descent.
//   One more sweep collects the elements of the chosen level-0 bin (a few hundred, typically) into
//   shared memory, and the remaining levels walk their exact key bytes (2 for bf16, 4 for fp32)
//   over that list.  A bin too crowded for the list (a row of equal values, a mass of masked
//   tokens in the last bin) is walked with sweeps over the row instead: slower, same result.
// Masses are sums of 2^(x*scale - M) in 2^-44 fixed point: integer arithmetic makes every sum exact
// and independent of the order of arrival, so the result is reproducible and the cumulative mass
// at the top-k threshold equals the survivors' mass bit for bit.  After the first sweep the row
// comes out of L2.
constexpr int kFilterThreads = 1024;
constexpr int kFilterUnroll = 4;   // 16-byte loads in flight per thread: one block per SM has to cover the latency alone
constexpr int kFilterWarps = kFilterThreads / 32;
constexpr int kFilterListCap = 12288;
constexpr float kMassScale = 17592186044416.f;  // 2^44
constexpr int kFilterSmemBytes = 4 * 256 * 32 * 4 + 256 * (8 + 4) * 2 + kFilterListCap * 4 + 64;
constexpr int kExactUnroll = 4;                                   // 16-byte loads per thread and round
constexpr int kExactPerThread = 35;                               // odd: a thread's run of counters starts in its own bank
constexpr int kExactBins = kFilterThreads * kExactPerThread;      // counters of the exact-value histogram (bf16 rows)
constexpr int kExactListCap = (kFilterSmemBytes - (kExactBins + 32) * 4) / 2;   // 16-bit distances of the occupied counters
static_assert(kExactBins <= 65536 && kExactListCap >= 16384, "the exact-value histogram and its list reuse the general path's shared memory");

// Calls f(x) for every element of a row; the block's threads stride over 16-byte vectors and keep
// kFilterUnroll of them in flight.
template <typename T, int kThreads = kFilterThreads, typename F>
__device__ __forceinline__ void sweep_row(const T *base, int vocab, int tid, F f) {
  constexpr int N = Vec<T>::N;
  constexpr int stride = kThreads * N;
  int v = tid * N;
  for (; v + (kFilterUnroll - 1) * stride + N <= vocab; v += kFilterUnroll * stride) {
    uint4 raw[kFilterUnroll];
#pragma unroll
    for (int u = 0; u < kFilterUnroll; ++u) raw[u] = __ldg(reinterpret_cast<const uint4 *>(base + v + u * stride));
#pragma unroll
    for (int u = 0; u < kFilterUnroll; ++u) {
      union { uint4 q; T e[N]; } tmp;
      tmp.q = raw[u];
#pragma unroll
      for (int i = 0; i < N; ++i) f(ld_as_float(tmp.e, i));
    }
  }
  for (; v < vocab; v += stride) {
    if (v + N <= vocab) {
      union { uint4 q; T e[N]; } tmp;
      tmp.q = __ldg(reinterpret_cast<const uint4 *>(base + v));
#pragma unroll
      for (int i = 0; i < N; ++i) f(ld_as_float(tmp.e, i));
    } else {
      for (int i = 0; i < N && v + i < vocab; ++i) f(ld_as_float(base, v + i));
    }
  }
}

// Calls f_vec(v) for every aligned group of eight bf16 logits of a row (one 16-byte vector, the
// element of the lowest index in the low half of v.x) and f_one(x) for the elements of a ragged
// end.  Rounds of kUnroll 16-byte loads per thread, predicated at the end of the row; the loads of
// the next round are in flight while a round is processed (two register buffers in turn).
template <int kUnroll, int kThreads, typename F, typename G>
__device__ __forceinline__ void sweep_row_vecs(const __nv_bfloat16 *base, int vocab, int tid, F f_vec, G f_one) {
  const int n_vec = vocab >> 3;
  const uint4 *b4 = reinterpret_cast<const uint4 *>(base);
  constexpr int kRound = kUnroll * kThreads;
  auto load = [&](uint4 (&raw)[kUnroll], int v0) {
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
      if (v0 + u * kThreads < n_vec) raw[u] = __ldg(b4 + v0 + u * kThreads);
  };
  auto work = [&](const uint4 (&raw)[kUnroll], int v0) {
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
      if (v0 + u * kThreads < n_vec) f_vec(raw[u]);
  };
  uint4 ra[kUnroll], rb[kUnroll];
  load(ra, tid);
  for (int v0 = tid; v0 < n_vec; v0 += 2 * kRound) {
    load(rb, v0 + kRound);
    work(ra, v0);
    load(ra, v0 + 2 * kRound);
    work(rb, v0 + kRound);
  }
  for (int i = (n_vec << 3) + tid; i < vocab; i += kThreads) f_one(__bfloat162float(base[i]));
}
// The same, word by word: f_pair(w) for every aligned pair of logits.
template <int kUnroll, int kThreads, typename F, typename G>
__device__ __forceinline__ void sweep_row_pairs(const __nv_bfloat16 *base, int vocab, int tid, F f_pair, G f_one) {
  sweep_row_vecs<kUnroll, kThreads>(base, vocab, tid, [&](const uint4 &v) { f_pair(v.x); f_pair(v.y); f_pair(v.z); f_pair(v.w); }, f_one);
}

// top-k (optionally with top-p on top) of one row per block for K no larger than the number of
// sub-segments of the row: the K-th largest of the sub-segment maxima (left by the statistics
// pass) is a lower bound of the K-th largest logit, so one compare-only sweep finds every
// candidate (a few hundred logits for K = 50 on a 128k vocabulary).  256 threads and a few KB of
// shared memory per row, so all the rows of a batch are resident at once and the kernel runs at
// the rate the logits arrive.
//   bf16 rows: the candidates lie within a few dozen 16-bit keys of the row maximum, so they are
//   counted per exact value in a window of kTopkWindow keys below it (mass of a key = count times
//   the mass of its value), and one scan over the window gives both thresholds; no list, so a
//   block of equal logits at the cut costs nothing.
//   fp32 rows: the candidates are listed and ranked by counting - thread i sums count and mass of
//   the keys above and at-or-above its own; no histogram, no atomics on the masses.
// Rows it cannot take (K larger than that, top-p alone, candidates beyond the window or the list)
// are left marked pending (row_z = NaN, set by row_scale_kernel) for filter_rows_kernel.
constexpr int kTopkThreads = 256;
constexpr int kTopkListCap = 1024;
constexpr int kTopkWindow = 1024;   // keys below the row maximum counted by the bf16 path (four per thread)
template <typename T>
__global__ void __launch_bounds__(kTopkThreads, 5) topk_list_kernel(SampleParams p) {
  __shared__ float s_list[kTopkListCap];
  __shared__ uint32_t s_key[kTopkListCap];
  __shared__ unsigned long long s_m[kTopkListCap];
  __shared__ uint32_t s_n, s_Tk, s_Tf;
  __shared__ unsigned long long s_Zk, s_Zf;
  __shared__ int s_found;
  __shared__ float s_bound;
  const int row = blockIdx.x, tid = threadIdx.x;
  const int r = p.row_req[row];
  if (r < 0) {
    if (tid == 0) { p.row_thresh[row] = 0; p.row_z[row] = -1.0; }
    return;
  }
  const int tk_raw = p.top_k ? p.top_k[r] : 0;
  const bool use_k = tk_raw >= 1 && tk_raw < p.vocab;
  const float tp = p.top_p ? p.top_p[r] : 1.f;
  const bool use_p = tp < 1.f;
  if (!use_k || tk_raw > p.nsub || p.nsub > kTopkThreads) return;
  const float scale = p.row_scale[row];
  const T *base = row < p.total_q ? reinterpret_cast<const T *>(p.target) + (int64_t)row * p.row_stride
                                  : reinterpret_cast<const T *>(p.draft) + (int64_t)(row - p.total_q) * p.row_stride;
  // the sub-segment maxima, once from memory (one per thread), then out of shared memory
  __shared__ float s_max[kTopkThreads];
  const float2 *st = p.seg_stats + (int64_t)row * p.nsub;
  if (tid < p.nsub) s_max[tid] = st[tid].x;
  if (tid == 0) { s_n = 0; s_found = 0; }
  __syncthreads();
  float M = -INFINITY;
  for (int j = 0; j < p.nsub; ++j) M = fmaxf(M, s_max[j]);
  auto mass_of = [&](float x) -> unsigned long long { return __float2ull_rn(fast_exp2(fmaf(x, scale, -M)) * kMassScale); };
  if (tid < p.nsub) {
    const float mine = s_max[tid];
    int rank = 0;
    for (int j = 0; j < p.nsub; ++j) {
      const float o = s_max[j];
      rank += (o > mine || (o == mine && j < tid)) ? 1 : 0;
    }
    if (rank == tk_raw - 1) s_bound = mine;
  }
  __syncthreads();
  const float bound = s_bound - (fabsf(s_bound) * 1e-6f + 1e-6f);  // in the scaled (log2) domain, like the statistics
  if constexpr (sizeof(T) == 2) {
    __shared__ uint32_t s_hist[kTopkWindow];
    __shared__ uint32_t s_wc[kTopkThreads / 32], s_dk, s_df;
    __shared__ unsigned long long s_wm[kTopkThreads / 32], s_zk, s_zf;
    const int lane = tid & 31, warp = tid >> 5;
    // keys: the reference one step above a bf16 value at or above the row maximum, the bound one
    // step below a bf16 value at or below the bound (in logit units)
    uint32_t key_ref, key_lo;
    {
      float xub = M / scale;
      xub = xub >= 0.f ? xub * (1.f + 0x1p-20f) : xub * (1.f - 0x1p-20f);
      const uint32_t fu = __float_as_uint(xub);
      const uint32_t bu = (fu & 0x80000000u) ? (fu >> 16) : ((fu + 0xffffu) >> 16);   // towards +inf
      const uint32_t ku = order_key32(__uint_as_float(bu << 16)) >> 16;
      key_ref = ku < 0xffffu ? ku + 1u : ku;
      const uint32_t fl = __float_as_uint(bound / scale);
      const uint32_t bl = (fl & 0x80000000u) ? ((fl + 0xffffu) >> 16) : (fl >> 16);   // towards -inf
      const uint32_t kl = order_key32(__uint_as_float(bl << 16)) >> 16;
      key_lo = kl > 0u ? kl - 1u : kl;
    }
    if (key_lo > key_ref || key_ref - key_lo >= (uint32_t)kTopkWindow) return;   // (uniform) the general kernel takes the row
#pragma unroll
    for (int i = 0; i < kTopkWindow / kTopkThreads; ++i) s_hist[tid + i * kTopkThreads] = 0;
    __syncthreads();
    bool above = false;
    auto take = [&](uint32_t k) {
      if (k >= key_lo) {
        const uint32_t d = key_ref - k;
        if (d < (uint32_t)kTopkWindow) atomicAdd(&s_hist[d], 1u); else above = true;   // above the reference: never with sound statistics
      }
    };
    // eight logits per test: their maximum by packed bf16 instructions against the bound as a value
    // (a superset of the key test: -0 and +0 compare equal); the rare vector that passes is taken
    // apart key by key
    const float x_lo = __uint_as_float(((key_lo & 0x8000u) ? (key_lo & 0x7fffu) : (~key_lo & 0xffffu)) << 16);
    sweep_row_vecs<kFilterUnroll, kTopkThreads>(reinterpret_cast<const __nv_bfloat16 *>(base), p.vocab, tid,
        [&](const uint4 &v) {
          auto b2 = [](uint32_t w) { return *reinterpret_cast<const __nv_bfloat162 *>(&w); };
          const __nv_bfloat162 m2 = __hmax2(__hmax2(b2(v.x), b2(v.y)), __hmax2(b2(v.z), b2(v.w)));
          if (fmaxf(__low2float(m2), __high2float(m2)) >= x_lo) {
            const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              uint32_t sm;
              asm("prmt.b32 %0, %1, 0, 0xBB99;" : "=r"(sm) : "r"(w4[i]));
              const uint32_t k2 = w4[i] ^ (sm | 0x80008000u);
              take(k2 & 0xffffu);
              take(k2 >> 16);
            }
          }
        },
        [&](float x) { take(order_key32(x) >> 16); });
    if (__syncthreads_or(above)) return;
    auto value_of = [&](uint32_t d) -> float {
      const uint32_t k = key_ref - d;
      const uint32_t b16 = (k & 0x8000u) ? (k & 0x7fffu) : (~k & 0xffffu);
      return __uint_as_float(b16 << 16);
    };
    // every thread takes four consecutive keys of the window (descending), then a block scan
    constexpr int kPerT = kTopkWindow / kTopkThreads;
    const uint32_t d0 = (uint32_t)tid * kPerT;
    uint32_t cb[kPerT], c_t = 0;
    unsigned long long mb[kPerT], m_t = 0ull;
#pragma unroll
    for (int j = 0; j < kPerT; ++j) {
      cb[j] = s_hist[d0 + j];
      mb[j] = cb[j] ? (unsigned long long)cb[j] * mass_of(value_of(d0 + j)) : 0ull;
      c_t += cb[j];
      m_t += mb[j];
    }
    uint32_t ci = c_t;
    unsigned long long mi = m_t;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t cn = __shfl_up_sync(0xffffffffu, ci, o);
      const unsigned long long mn = __shfl_up_sync(0xffffffffu, mi, o);
      if (lane >= o) { ci += cn; mi += mn; }
    }
    if (lane == 31) { s_wc[warp] = ci; s_wm[warp] = mi; }
    __syncthreads();
    uint32_t ce = ci - c_t, total_c = 0;   // counts / masses of the keys above this thread's four
    unsigned long long me = mi - m_t;
#pragma unroll
    for (int w = 0; w < kTopkThreads / 32; ++w) {
      if (w < warp) { ce += s_wc[w]; me += s_wm[w]; }
      total_c += s_wc[w];
    }
    if (total_c < (uint32_t)tk_raw) return;   // (uniform; cannot happen: the K largest sub-segment maxima are candidates)
    if (ce < (uint32_t)tk_raw && ce + c_t >= (uint32_t)tk_raw) {   // exactly one thread
      uint32_t cc = ce;
      unsigned long long mm = me;
#pragma unroll
      for (int j = 0; j < kPerT; ++j) {
        cc += cb[j];
        mm += mb[j];
        if (cb[j] && cc >= (uint32_t)tk_raw) { s_dk = d0 + j; s_zk = mm; s_df = d0 + j; s_zf = mm; break; }
      }
    }
    __syncthreads();
    const unsigned long long Zk = s_zk;
    if (use_p) {
      // the highest key with mass(key >= T) >= P * kept mass: at or above the top-k cut, where the
      // running mass equals the kept mass
      const double need_mass = (double)tp * (double)Zk;
      if (!((double)me >= need_mass) && (double)(me + m_t) >= need_mass) {   // exactly one thread
        unsigned long long mm = me;
#pragma unroll
        for (int j = 0; j < kPerT; ++j) {
          mm += mb[j];
          if (cb[j] && (double)mm >= need_mass) { s_df = d0 + j; s_zf = mm; break; }
        }
      }
      __syncthreads();
    }
    if (tid == 0) {
      p.row_thresh[row] = order_key32(value_of(s_df));
      p.row_z[row] = (double)s_zf / (double)kMassScale;
    }
    return;
  }
  sweep_row<T, kTopkThreads>(base, p.vocab, tid, [&](float x) {
    if (x * scale >= bound) {
      const uint32_t i = atomicAdd(&s_n, 1u);
      if (i < (uint32_t)kTopkListCap) s_list[i] = x;
    }
  });
  __syncthreads();
  const uint32_t n = s_n;
  if (n > (uint32_t)kTopkListCap) return;   // too many equal logits at the cut: the general kernel takes the row
  for (uint32_t i = tid; i < n; i += kTopkThreads) { s_key[i] = order_key32(s_list[i]); s_m[i] = mass_of(s_list[i]); }
  __syncthreads();
  // the highest key T with count(key >= T) >= K; then, with top-p, the highest key with
  // mass(key >= T) >= P * kept mass (never below the top-k cut)
  constexpr int kPer = kTopkListCap / kTopkThreads;
  uint32_t key[kPer], cnt_ge[kPer];
  unsigned long long m_gt[kPer], m_ge[kPer];
#pragma unroll
  for (int q = 0; q < kPer; ++q) {
    const uint32_t i = tid + q * kTopkThreads;
    key[q] = 0; cnt_ge[q] = 0; m_gt[q] = 0ull; m_ge[q] = 0ull;
    if (i < n) {
      const uint32_t ki = s_key[i];
      uint32_t c_gt = 0, c_ge = 0;
      unsigned long long a_gt = 0ull, a_ge = 0ull;
      for (uint32_t j = 0; j < n; ++j) {
        const uint32_t kj = s_key[j];
        const unsigned long long mj = s_m[j];
        if (kj > ki) { ++c_gt; a_gt += mj; }
        if (kj >= ki) { ++c_ge; a_ge += mj; }
      }
      key[q] = ki; cnt_ge[q] = c_ge; m_gt[q] = a_gt; m_ge[q] = a_ge;
      if (c_gt < (uint32_t)tk_raw && c_ge >= (uint32_t)tk_raw) { s_Tk = ki; s_Zk = a_ge; }  // equal keys write equal values
    }
  }
  __syncthreads();
  const uint32_t Tk = s_Tk;
  const unsigned long long Zk = s_Zk;
  uint32_t Tf = Tk;
  unsigned long long Zf = Zk;
  if (use_p) {
    const double need_mass = (double)tp * (double)Zk;
#pragma unroll
    for (int q = 0; q < kPer; ++q)
      if (tid + q * kTopkThreads < (int)n && (double)m_gt[q] < need_mass && (double)m_ge[q] >= need_mass) {
        s_Tf = key[q]; s_Zf = m_ge[q]; s_found = 1;
      }
    __syncthreads();
    if (!s_found) {  // rounding left the criterion unmet even at the lowest key: take it
#pragma unroll
      for (int q = 0; q < kPer; ++q)
        if (tid + q * kTopkThreads < (int)n && cnt_ge[q] == n) { s_Tf = key[q]; s_Zf = m_ge[q]; }
      __syncthreads();
    }
    Tf = s_Tf; Zf = s_Zf;
    if (Tf < Tk) { Tf = Tk; Zf = Zk; }
  }
  if (tid == 0) {
    p.row_thresh[row] = Tf;
    p.row_z[row] = (double)Zf / (double)kMassScale;
  }
}

template <typename T>
__global__ void __launch_bounds__(kFilterThreads, 1) filter_rows_kernel(SampleParams p) {
  extern __shared__ __align__(16) unsigned char fsm[];
  unsigned long long *s_mass = reinterpret_cast<unsigned long long *>(fsm);                    // [256] level sums
  unsigned long long *s_mass1 = s_mass + 256;                                                  // [256] level-0 copy
  uint32_t *h_cnt = reinterpret_cast<uint32_t *>(s_mass1 + 256);                               // [256][lane]
  uint32_t *h_m0 = h_cnt + 256 * 32;                                                           // mass bits 0..14
  uint32_t *h_m1 = h_m0 + 256 * 32;                                                            // mass bits 15..29
  uint32_t *h_m2 = h_m1 + 256 * 32;                                                            // mass bits 30..44
  uint32_t *s_cnt = h_m2 + 256 * 32;
  uint32_t *s_cnt1 = s_cnt + 256;
  float *s_list = reinterpret_cast<float *>(s_cnt1 + 256);                                     // [kFilterListCap]
  __shared__ uint32_t s_bin, s_above_cnt, s_list_n;
  __shared__ unsigned long long s_above_mass, s_bin_mass;
  const int row = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // what the block needs of the row, fetched in two round trips instead of a chain of five: the
  // loads that do not depend on the request first, all at once
  const float2 *st = p.seg_stats + (int64_t)row * p.nsub;
  const double z_in = __ldg(p.row_z + row);
  const int r = __ldg(p.row_req + row);
  const float scale = __ldg(p.row_scale + row);
  if (z_in == z_in) return;   // not pending (NaN): topk_list_kernel has settled this row
  if (r < 0) {
    if (tid == 0) { p.row_thresh[row] = 0; p.row_z[row] = -1.0; }
    return;
  }
  float M = -INFINITY;   // the row maximum (scaled) out of the sub-segment statistics: every warp reduces them for itself
  for (int j = lane; j < p.nsub; j += 32) M = fmaxf(M, __ldg(&st[j].x));
  constexpr int kLevels = sizeof(T) == 2 ? 2 : 4;      // exact key bytes after level 0
  constexpr int kKeyShift = sizeof(T) == 2 ? 16 : 0;   // bf16: the low 16 bits of the fp32 key carry nothing
  const int tk_raw = p.top_k ? __ldg(p.top_k + r) : 0;
  const float tp = p.top_p ? __ldg(p.top_p + r) : 1.f;
  if constexpr (sizeof(T) == 2) {
    // the exact-value histogram below is cleared while those two are on their way
    uint32_t *h = reinterpret_cast<uint32_t *>(fsm);
    for (int i = tid; i < kExactBins + 32; i += kFilterThreads) h[i] = 0;
  }
  const bool use_k = tk_raw >= 1 && tk_raw < p.vocab;
  const bool use_p = tp < 1.f;
  const float inv_w = 8.f / scale;   // distance in log2 units -> eighths of a logit unit
  const T *base = row < p.total_q ? reinterpret_cast<const T *>(p.target) + (int64_t)row * p.row_stride
                                  : reinterpret_cast<const T *>(p.draft) + (int64_t)(row - p.total_q) * p.row_stride;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  auto bin0_of = [&](float x) -> uint32_t {
    const float d = fmaxf(fmaf(x, -scale, M), 0.f) * inv_w;
    return 255u - (uint32_t)fminf(d, 255.f);
  };
  auto mass_of = [&](float x) -> unsigned long long { return __float2ull_rn(fast_exp2(fmaf(x, scale, -M)) * kMassScale); };

  // bf16 rows: one histogram of COUNTS over the exact values.  A bf16 logit has a 16-bit key, and the
  // keys of a row lie within a few ten thousand steps below the key of its maximum (128 per binade:
  // from 16 down through zero to -16 are 34 k keys), so one counter per key fits in shared memory.
  // Equal values have equal masses, so the mass of a key is its count times the mass of its value -
  // the same integer as the sum over its elements - and the thresholds follow from one scan over the
  // occupied counters in descending key order: no masses are added per element, no second sweep,
  // no further levels.  What bounds the sweep are the shared-memory atomics: 32 random counters per
  // instruction meet in about four bank conflicts.  Values below the counters are tolerated while
  // they carry no mass (masked tokens at -inf) and no threshold falls among them; any other row
  // with values outside the counters' range takes the general path below.
  if constexpr (sizeof(T) == 2) {
    uint32_t *h = reinterpret_cast<uint32_t *>(fsm);   // [kExactBins], index = key distance below the reference
    uint16_t *nzl = reinterpret_cast<uint16_t *>(fsm + (kExactBins + 32) * 4);   // [kExactListCap] distances of the occupied counters
    __shared__ uint32_t s_over, s_tail, s_dk, s_df, s_found, s_nn, s_tc, s_wc[kFilterWarps];
    __shared__ unsigned long long s_wm[kFilterWarps], s_zk, s_zf, s_tm;
    if (tid == 0) { s_over = 0; s_tail = 0; s_found = 0; }
    // reference: a bf16 value at or above every value of the row (the maximum of the statistics is
    // the row's largest logit times the scale, rounded)
    uint32_t key_ref;
    {
      float xub = M / scale;
      xub = xub >= 0.f ? xub * (1.f + 0x1p-20f) : xub * (1.f - 0x1p-20f);
      const uint32_t fb = __float_as_uint(xub);
      const uint32_t b16 = (fb & 0x80000000u) ? (fb >> 16) : ((fb + 0xffffu) >> 16);   // towards +inf
      const uint32_t k = order_key32(__uint_as_float(b16 << 16)) >> 16;
      key_ref = k < 0xffffu ? k + 1u : k;
    }
    __syncthreads();
    // Two logits per step of integer arithmetic: the sign of each half spread over the half (one
    // byte permute), the order key of both (one logic operation), both distances by one
    // subtraction - the reference is at or above every value, so no half borrows from the other.
    // A value below the counters is counted in one of 32 spare counters behind them (the lane's own:
    // a row full of masked tokens must not queue up on one address), so the loop has no branch.
    const uint32_t ref2 = key_ref * 0x10001u;
    const uint32_t spare = (uint32_t)kExactBins + (uint32_t)lane;
    sweep_row_pairs<kExactUnroll, kFilterThreads>(reinterpret_cast<const __nv_bfloat16 *>(base), p.vocab, tid,
        [&](uint32_t w) {
          uint32_t sm;
          asm("prmt.b32 %0, %1, 0, 0xBB99;" : "=r"(sm) : "r"(w));
          const uint32_t d2 = ref2 - (w ^ (sm | 0x80008000u));
          atomicAdd(&h[min(d2 & 0xffffu, spare)], 1u);
          atomicAdd(&h[min(d2 >> 16, spare)], 1u);
        },
        [&](float x) { atomicAdd(&h[min(key_ref - (order_key32(x) >> 16), spare)], 1u); });
    __syncthreads();
    const bool outside = tid < 32 && h[kExactBins + tid] != 0u;
    if (__syncthreads_or(outside)) {
      // Values below the counters (masked tokens at -inf, typically) are harmless while they carry
      // no mass and no threshold falls among them: one more sweep tells which kind they are.
      sweep_row<T>(base, p.vocab, tid, [&](float x) {
        const uint32_t k = order_key32(x) >> 16;
        if (k > key_ref || key_ref - k >= (uint32_t)kExactBins) {
          const bool massless = k <= key_ref && mass_of(x) == 0ull;
          const uint32_t act = __activemask();
          const uint32_t zl = __ballot_sync(act, massless);
          if (lane == __ffs(act) - 1) {   // the lanes that got here together add once
            if (zl) atomicAdd(&s_tail, (uint32_t)__popc(zl));
            if (zl != act) atomicAdd(&s_over, (uint32_t)__popc(act & ~zl));
          }
        }
      });
      __syncthreads();
    }
    if (s_over == 0) {
      auto value_of = [&](uint32_t d) -> float {
        const uint32_t k = key_ref - d;
        const uint32_t b16 = (k & 0x8000u) ? (k & 0x7fffu) : (~k & 0xffffu);
        return __uint_as_float(b16 << 16);
      };
      // The occupied counters lie in two or three dense stretches of the key axis, so their keys
      // are first written out as a list (descending): every thread counts the occupied counters
      // of its own run, a scan gives it its place in the list, and then every thread takes an
      // equal share of the LIST - masses are evaluated three or so per thread instead of a
      // whole run by the few threads whose runs are occupied.
      const uint32_t d0 = (uint32_t)tid * kExactPerThread;
      static_assert(kExactPerThread % 5 == 0, "runs are read five counters at a time");
      uint32_t nz_t = 0;
#pragma unroll
      for (int j = 0; j < kExactPerThread; ++j) nz_t += h[d0 + j] != 0u ? 1u : 0u;
      // exclusive scan over the block: within the warps, then warp 0 over the warps' totals
      uint32_t nzi = nz_t;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, nzi, o);
        if (lane >= o) nzi += v;
      }
      if (lane == 31) s_wc[warp] = nzi;
      __syncthreads();
      if (warp == 0) {
        const uint32_t v = s_wc[lane];
        uint32_t vi = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t x = __shfl_up_sync(0xffffffffu, vi, o);
          if (lane >= o) vi += x;
        }
        s_wc[lane] = vi - v;
        if (lane == 31) s_nn = vi;
      }
      __syncthreads();
      const uint32_t n_nz = s_nn;
      if (n_nz >= 1u && n_nz <= (uint32_t)kExactListCap) {
        uint32_t off = nzi - nz_t + s_wc[warp];
        for (int j = 0; j < kExactPerThread; ++j)
          if (h[d0 + j]) nzl[off++] = (uint16_t)(d0 + j);
        __syncthreads();
        const uint32_t per = (n_nz + kFilterThreads - 1) / kFilterThreads;
        const uint32_t e0 = min((uint32_t)tid * per, n_nz), e1 = min(e0 + per, n_nz);
        uint32_t c_t = 0;
        unsigned long long m_t = 0ull;
        for (uint32_t e = e0; e < e1; ++e) {
          const uint32_t d = nzl[e], c = h[d];
          c_t += c;
          m_t += (unsigned long long)c * mass_of(value_of(d));
        }
        uint32_t ci = c_t;
        unsigned long long mi = m_t;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t cn = __shfl_up_sync(0xffffffffu, ci, o);
          const unsigned long long mn = __shfl_up_sync(0xffffffffu, mi, o);
          if (lane >= o) { ci += cn; mi += mn; }
        }
        if (lane == 31) { s_wc[warp] = ci; s_wm[warp] = mi; }
        __syncthreads();
        if (warp == 0) {
          const uint32_t v = s_wc[lane];
          const unsigned long long w = s_wm[lane];
          uint32_t vi = v;
          unsigned long long wi = w;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const uint32_t x = __shfl_up_sync(0xffffffffu, vi, o);
            const unsigned long long y = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) { vi += x; wi += y; }
          }
          s_wc[lane] = vi - v;
          s_wm[lane] = wi - w;
          if (lane == 31) { s_tc = vi; s_tm = wi; }
        }
        __syncthreads();
        const uint32_t ce = ci - c_t + s_wc[warp], total_c = s_tc;   // counts / masses of the keys above this thread's share
        const unsigned long long me = mi - m_t + s_wm[warp], total = s_tm;
        // a top-k cut among the tokens below the counters is left to the general path
        if (!use_k || total_c >= (uint32_t)tk_raw) {
          unsigned long long Zk = total;
          if (use_k) {
            if (ce < (uint32_t)tk_raw && ce + c_t >= (uint32_t)tk_raw) {   // exactly one thread
              uint32_t cc = ce;
              unsigned long long mm = me;
              for (uint32_t e = e0; e < e1; ++e) {
                const uint32_t d = nzl[e], c = h[d];
                cc += c;
                mm += (unsigned long long)c * mass_of(value_of(d));
                if (cc >= (uint32_t)tk_raw) { s_dk = d; s_zk = mm; break; }
              }
            }
            __syncthreads();
            Zk = s_zk;
          }
          if (use_p) {
            const double need_mass = (double)tp * (double)Zk;
            if (!((double)me >= need_mass) && (double)(me + m_t) >= need_mass) {   // at most one thread
              unsigned long long mm = me;
              for (uint32_t e = e0; e < e1; ++e) {
                const uint32_t d = nzl[e];
                mm += (unsigned long long)h[d] * mass_of(value_of(d));
                if ((double)mm >= need_mass) { s_df = d; s_zf = mm; s_found = 1; break; }
              }
            }
            __syncthreads();
          }
          // rounding can leave the mass criterion unmet even at the lowest key, which is then taken:
          // with tokens below the counters that key is not known here
          if (!use_p || s_found || s_tail == 0) {
            if (tid == 0) {
              uint32_t d_f;
              unsigned long long Zf;
              if (use_p) {
                if (s_found) { d_f = s_df; Zf = s_zf; } else { d_f = nzl[n_nz - 1]; Zf = total; }
                if (use_k && d_f > s_dk) { d_f = s_dk; Zf = s_zk; }   // the sets stay nested
              } else {
                d_f = s_dk; Zf = s_zk;
              }
              p.row_thresh[row] = order_key32(value_of(d_f));
              p.row_z[row] = (double)Zf / (double)kMassScale;
            }
            return;
          }
        }
      }
    }
    __syncthreads();
  }

  // warp 0: the highest bin b such that (count or mass of bins >= b, plus what lies above the
  // prefix) reaches the target; leaves the bin, and count / mass of the bins above it, in shared memory
  auto pick = [&](bool by_count, uint32_t need_cnt, double need_mass, unsigned long long mass_above_prefix) {
    if (warp == 0) {
      // lane l owns bins 255-8l .. 248-8l (descending)
      uint32_t c8 = 0;
      unsigned long long m8 = 0ull;
#pragma unroll
      for (int j = 0; j < 8; ++j) { c8 += s_cnt[255 - 8 * lane - j]; m8 += s_mass[255 - 8 * lane - j]; }
      uint32_t ci = c8;
      unsigned long long mi = m8;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t cn = __shfl_up_sync(0xffffffffu, ci, o);
        const unsigned long long mn = __shfl_up_sync(0xffffffffu, mi, o);
        if (lane >= o) { ci += cn; mi += mn; }
      }
      const bool reached = by_count ? (ci >= need_cnt) : ((double)(mass_above_prefix + mi) >= need_mass);
      const uint32_t bal = __ballot_sync(0xffffffffu, reached);
      // rounding could leave the mass criterion unmet even at the last bin: take the lowest occupied bin then
      const int owner = bal ? __ffs(bal) - 1 : 31;
      if (lane == owner) {
        uint32_t cc = ci - c8;
        unsigned long long mm = mi - m8;
        int b = 255 - 8 * lane, chosen = -1;
        for (int j = 0; j < 8; ++j, --b) {
          const bool hit = by_count ? (cc + s_cnt[b] >= need_cnt) : ((double)(mass_above_prefix + mm + s_mass[b]) >= need_mass);
          if (hit) { chosen = b; break; }
          cc += s_cnt[b];
          mm += s_mass[b];
        }
        if (chosen < 0) {  // only without a crossing: lowest occupied bin of the whole level
          cc = 0; mm = 0ull; chosen = 0;
          for (int bb = 255; bb >= 0; --bb) if (s_cnt[bb] || s_mass[bb]) chosen = bb;
          for (int bb = 255; bb > chosen; --bb) { cc += s_cnt[bb]; mm += s_mass[bb]; }
        }
        s_bin = (uint32_t)chosen;
        s_above_cnt = cc;
        s_above_mass = mm;
        s_bin_mass = s_mass[chosen];
      }
    }
    __syncthreads();
  };

  // One level's histogram (count, mass per key byte) of the listed logits that match the prefix.
  // The listed logits lie within a fraction of a logit unit of each other, so at the first levels
  // all of them fall into one bin and at the later ones into a few dozen: 64-bit shared-memory
  // atomics (a compare-and-swap loop) on so few addresses queue up for hundreds of cycles each.  The
  // masses are therefore added as three 15-bit pieces with native 32-bit atomics (a list holds at
  // most kFilterListCap logits: no piece overflows), into the first rows of the per-lane arrays,
  // which are idle here; and a warp whose lanes all agree on the bin adds its 32 masses up with
  // shuffles and issues one set of atomics.
  auto level_hist_of_list = [&](int level, int shift, uint32_t prefix, uint32_t n_list) {
    if (tid < 256) { s_cnt[tid] = 0; h_m0[tid] = 0; h_m1[tid] = 0; h_m2[tid] = 0; }
    __syncthreads();
    for (uint32_t i0 = (uint32_t)(tid & ~31); i0 < n_list; i0 += kFilterThreads) {   // warp-uniform bounds
      const uint32_t i = i0 + lane;
      bool use = i < n_list;
      float x = 0.f;
      uint32_t key = 0;
      if (use) {
        x = s_list[i];
        key = order_key32(x);
        use = level == 1 || (key >> (shift + 8)) == (prefix >> (shift + 8));
      }
      const uint32_t bin = use ? ((key >> shift) & 255u) : 0xffffffffu;
      unsigned long long m = use ? mass_of(x) : 0ull;
      uint32_t c = use ? 1u : 0u;
      int same = 0;
      __match_all_sync(0xffffffffu, bin, &same);
      if (same) {
        if (bin == 0xffffffffu) continue;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          m += __shfl_xor_sync(0xffffffffu, m, o);
          c += __shfl_xor_sync(0xffffffffu, c, o);
        }
        if (lane == 0) {   // up to 32 masses: the pieces are cut from the sum, 20 bits suffice for the top one
          atomicAdd(&s_cnt[bin], c);
          atomicAdd(&h_m0[bin], (uint32_t)(m & 0x7fffull));
          atomicAdd(&h_m1[bin], (uint32_t)((m >> 15) & 0x7fffull));
          atomicAdd(&h_m2[bin], (uint32_t)(m >> 30));
        }
      } else if (use) {
        atomicAdd(&s_cnt[bin], 1u);
        atomicAdd(&h_m0[bin], (uint32_t)(m & 0x7fffull));
        atomicAdd(&h_m1[bin], (uint32_t)((m >> 15) & 0x7fffull));
        atomicAdd(&h_m2[bin], (uint32_t)(m >> 30));
      }
    }
    __syncthreads();
    if (tid < 256)
      s_mass[tid] = (unsigned long long)h_m0[tid] + ((unsigned long long)h_m1[tid] << 15) + ((unsigned long long)h_m2[tid] << 30);
  };

  // Exact key-byte levels over the n_list logits in s_list (every level narrows the key by one
  // byte; after the last the key is complete).  Returns the threshold key, *Z the mass at or above it.
  auto levels_over_list = [&](bool by_count, uint32_t need, double need_mass, uint32_t n_list, unsigned long long *Z) -> uint32_t {
    uint32_t prefix = 0;
    unsigned long long above = 0ull;
    for (int level = 1; level <= kLevels; ++level) {
      const int shift = kKeyShift + 8 * (kLevels - level);
      if (tid < 256) { s_cnt[tid] = 0; s_mass[tid] = 0ull; }
      __syncthreads();
      level_hist_of_list(level, shift, prefix, n_list);
      __syncthreads();
      pick(by_count, need, need_mass, above);
      prefix |= s_bin << shift;
      need -= s_above_cnt;
      above += s_above_mass;
      if (level == kLevels) *Z = above + s_bin_mass;
      __syncthreads();
    }
    return prefix;
  };

  // top-k with K no larger than the number of sub-segments of the row, for the rows that
  // topk_list_kernel left (more candidates than its list holds, or more sub-segments than it has
  // threads): the same lower bound and compare-only sweep into the larger list here, then the
  // exact key-byte levels over that list.  A list that overflows even here (many equal logits)
  // falls back to the histogram path below.
  if (use_k && tk_raw <= p.nsub && p.nsub <= kFilterThreads) {
    __shared__ float s_bound;
    const float2 *st = p.seg_stats + (int64_t)row * p.nsub;
    if (tid < p.nsub) {
      const float mine = st[tid].x;
      int rank = 0;
      for (int j = 0; j < p.nsub; ++j) {
        const float o = st[j].x;
        rank += (o > mine || (o == mine && j < tid)) ? 1 : 0;
      }
      if (rank == tk_raw - 1) s_bound = mine;
    }
    if (tid == 0) s_list_n = 0;
    __syncthreads();
    const float bound = s_bound - (fabsf(s_bound) * 1e-6f + 1e-6f);  // in the scaled (log2) domain, like the statistics
    sweep_row<T>(base, p.vocab, tid, [&](float x) {
      if (x * scale >= bound) {
        const uint32_t i = atomicAdd(&s_list_n, 1u);
        if (i < (uint32_t)kFilterListCap) s_list[i] = x;
      }
    });
    __syncthreads();
    const uint32_t n_list = s_list_n;
    if (n_list <= (uint32_t)kFilterListCap) {
      unsigned long long Zk = 0ull, Zf = 0ull;
      const uint32_t Tk = levels_over_list(true, (uint32_t)tk_raw, 0.0, n_list, &Zk);
      uint32_t Tf = Tk;
      Zf = Zk;
      if (use_p) {
        Tf = levels_over_list(false, 0u, (double)tp * (double)Zk, n_list, &Zf);
        if (Tf < Tk) { Tf = Tk; Zf = Zk; }
      }
      if (tid == 0) {
        p.row_thresh[row] = Tf;
        p.row_z[row] = (double)Zf / (double)kMassScale;
      }
      return;
    }
    __syncthreads();
  }

  // level 0: the whole row into the per-lane copies, then their sums into s_cnt / s_mass
  for (int i = tid; i < 4 * 256 * 32; i += kFilterThreads) h_cnt[i] = 0;   // the four arrays are contiguous
  __syncthreads();
  sweep_row<T>(base, p.vocab, tid, [&](float x) {
    const uint32_t slot = bin0_of(x) * 32 + lane;
    if (use_k) atomicAdd(&h_cnt[slot], 1u);
    if (use_p) {
      const unsigned long long m = mass_of(x);
      atomicAdd(&h_m0[slot], (uint32_t)(m & 0x7fffull));
      atomicAdd(&h_m1[slot], (uint32_t)((m >> 15) & 0x7fffull));
      atomicAdd(&h_m2[slot], (uint32_t)(m >> 30));
    }
  });
  __syncthreads();
  if (tid < 256) {
    uint32_t c = 0;
    unsigned long long m = 0ull;
    for (int j = 0; j < 32; ++j) {
      const int slot = tid * 32 + ((j + tid) & 31);
      c += h_cnt[slot];
      m += (unsigned long long)h_m0[slot] + ((unsigned long long)h_m1[slot] << 15) + ((unsigned long long)h_m2[slot] << 30);
    }
    s_cnt[tid] = s_cnt1[tid] = c;
    s_mass[tid] = s_mass1[tid] = m;
  }
  __syncthreads();
  unsigned long long total = 0ull;
  for (int b = 0; b < 256; ++b) total += s_mass1[b];   // every thread: 256 broadcast reads

  // One descent.  On entry s_cnt / s_mass hold level 0.  Returns the threshold key; *Z receives the
  // mass at or above it (meaningful only when masses were kept at level 0, i.e. use_p).
  unsigned long long mass_above_bin = 0ull;  // top-k alone: this thread's share of the mass in the bins above the chosen one
  bool list_ok = false;
  uint32_t list_len = 0;
  auto descend = [&](bool by_count, uint32_t need, double need_mass, unsigned long long *Z) -> uint32_t {
    pick(by_count, need, need_mass, 0ull);
    const uint32_t b0 = s_bin;
    need -= s_above_cnt;
    unsigned long long above = s_above_mass;
    __syncthreads();
    // the elements of bin b0, into shared memory if they fit
    if (tid == 0) s_list_n = 0;
    __syncthreads();
    const bool sum_above = by_count && !use_p;  // no masses were kept at level 0: add up what lies above the bin here
    sweep_row<T>(base, p.vocab, tid, [&](float x) {
      const uint32_t bx = bin0_of(x);
      if (sum_above && bx > b0) mass_above_bin += mass_of(x);
      if (bx != b0) return;
      const uint32_t i = atomicAdd(&s_list_n, 1u);
      if (i < (uint32_t)kFilterListCap) s_list[i] = x;
    });
    __syncthreads();
    const uint32_t n_list = s_list_n;
    const bool listed = n_list <= (uint32_t)kFilterListCap;
    list_ok = listed;
    list_len = n_list;
    uint32_t prefix = 0;
    for (int level = 1; level <= kLevels; ++level) {
      const int shift = kKeyShift + 8 * (kLevels - level);
      if (tid < 256) { s_cnt[tid] = 0; s_mass[tid] = 0ull; }
      __syncthreads();
      auto add = [&](float x) {
        const uint32_t key = order_key32(x);
        if (level > 1 && (key >> (shift + 8)) != (prefix >> (shift + 8))) return;
        const uint32_t bin = (key >> shift) & 255u;
        atomicAdd(&s_cnt[bin], 1u);
        atomicAdd(&s_mass[bin], mass_of(x));
      };
      if (listed) {
        level_hist_of_list(level, shift, prefix, n_list);
      } else {
        sweep_row<T>(base, p.vocab, tid, [&](float x) { if (bin0_of(x) == b0) add(x); });
      }
      __syncthreads();
      pick(by_count, need, need_mass, above);
      prefix |= s_bin << shift;
      need -= s_above_cnt;
      above += s_above_mass;
      if (level == kLevels) *Z = above + s_bin_mass;
      __syncthreads();
    }
    return prefix;
  };

  uint32_t Tk = 0;
  unsigned long long Zk = total;
  if (use_k) Tk = descend(true, (uint32_t)tk_raw, 0.0, &Zk);
  uint32_t Tf = Tk;
  unsigned long long Zf = Zk;
  if (use_p) {
    if (use_k) {  // level 0 again (the top-k descent reused the arrays)
      if (tid < 256) { s_cnt[tid] = s_cnt1[tid]; s_mass[tid] = s_mass1[tid]; }
      __syncthreads();
    }
    Tf = descend(false, 0u, (double)tp * (double)Zk, &Zf);
    if (Tf < Tk) { Tf = Tk; Zf = Zk; }  // cannot happen with exact sums; keeps the sets nested regardless
  } else {
    // top-k alone kept only counts at level 0.  The kept mass is what lay above the chosen bin (added up
    // during the collecting sweep) plus the listed elements at or above the threshold; a bin too
    // crowded for the list costs one more sweep instead.
    unsigned long long acc = 0ull;
    if (list_ok) {
      acc = mass_above_bin;
      for (uint32_t i = tid; i < list_len; i += kFilterThreads)
        if (order_key32(s_list[i]) >= Tf) acc += mass_of(s_list[i]);
    } else {
      sweep_row<T>(base, p.vocab, tid, [&](float x) { if (order_key32(x) >= Tf) acc += mass_of(x); });
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    __syncthreads();
    if (lane == 0) s_mass[warp] = acc;
    __syncthreads();
    Zf = 0ull;
    for (int w = 0; w < kFilterWarps; ++w) Zf += s_mass[w];
  }
  if (tid == 0) {
    p.row_thresh[row] = Tf;
    p.row_z[row] = (double)Zf / (double)kMassScale;
  }
}

// Verification variants, step 0: the scale log2(e)/tau of every logits row.  One thread per request.
// Greedy requests (tau = 0) need only the maxima of their target rows (scale log2(e)); their draft
// rows, and every row of a request whose temperature is not one, are marked 0 = skip.
__global__ void row_scale_kernel(SampleParams p) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= p.batch) return;
  const int t0 = p.q_indptr[r];
  const int k = p.q_indptr[r + 1] - t0 - 1;
  if (k < 0 || k > SPX_MAX_K || t0 < 0 || t0 + k + 1 > p.total_q) return;  // reported by accept_kernel
  const float tau = p.temperature ? p.temperature[r] : 1.f;
  const float tp = p.top_p ? p.top_p[r] : 1.f;
  const int tk = p.top_k ? p.top_k[r] : 0;
  const bool valid = tau >= 0.f && tau != INFINITY && tp > 0.f && tp <= 1.f;
  const float st = !valid ? 0.f : (tau == 0.f ? kLog2e : kLog2e / tau);
  const float sd = (valid && tau > 0.f) ? st : 0.f;
  for (int i = 0; i <= k; ++i) p.row_scale[t0 + i] = st;
  for (int i = 0; i < k; ++i) p.row_scale[p.total_q + t0 - r + i] = sd;
  if (p.row_req) {
    const bool filtered = valid && tau > 0.f && ((tk >= 1 && tk < p.vocab) || tp < 1.f);
    const double pending = __longlong_as_double(0x7ff8000000000000ll);  // NaN: no threshold yet
    for (int i = 0; i <= k; ++i) { p.row_req[t0 + i] = filtered ? r : -1; p.row_z[t0 + i] = pending; }
    for (int i = 0; i < k; ++i) { p.row_req[p.total_q + t0 - r + i] = filtered ? r : -1; p.row_z[p.total_q + t0 - r + i] = pending; }
  }
}

// Greedy verification (tau = 0) of one request by one block: a warp finds the greedy choice of a
// target row - the lowest token id that attains the row maximum, compared on the stored values -
// from the sub-segment maxima of the statistics pass (scaling is monotone, so the row maximum lies
// in a sub-segment whose scaled maximum equals the row's) and one scan of those sub-segments.
// Thread 0 then accepts drafts while they equal the greedy choice and emits the choice of row n.
// Requests that are not greedy, or that the accept test reports as invalid, are left alone.
template <typename T>
__device__ __forceinline__ void greedy_request(const SampleParams &p, int r) {
  if (!p.temperature || !(p.temperature[r] == 0.f)) return;
  const int t0 = p.q_indptr[r];
  const int k = p.q_indptr[r + 1] - t0 - 1;
  if (k < 0 || k > SPX_MAX_K || t0 < 0 || t0 + k + 1 > p.total_q) return;
  const int d0 = t0 - r;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  __shared__ int s_arg[SPX_MAX_K + 1];
  __shared__ int s_bad;
  if (threadIdx.x == 0) s_bad = 0;
  __syncthreads();
  if ((int)threadIdx.x < k) {
    const int x = p.draft_ids[d0 + threadIdx.x];
    if (x < 0 || x >= p.vocab) s_bad = 1;
  }
  __syncthreads();
  if (s_bad) return;
  for (int i = warp; i <= k; i += n_warps) {
    constexpr int N = Vec<T>::N;
    const float2 *st = p.seg_stats + (int64_t)(t0 + i) * p.nsub;
    const T *row = reinterpret_cast<const T *>(p.target) + (int64_t)(t0 + i) * p.row_stride;
    float M = -INFINITY;
    for (int j = lane; j < p.nsub; j += 32) M = fmaxf(M, st[j].x);
    M = warp_max(M);
    float best = -INFINITY;
    int best_i = 0x7fffffff;
    auto consider = [&](float v, int idx) {
      if (v > best || (v == best && idx < best_i)) { best = v; best_i = idx; }
    };
    for (int j0 = 0; j0 < p.nsub; j0 += 32) {
      const int j = j0 + lane;
      uint32_t cand = __ballot_sync(0xffffffffu, j < p.nsub && st[j].x == M);
      while (cand) {
        const int sub = j0 + __ffs(cand) - 1;
        cand &= cand - 1;
#pragma unroll
        for (int c = 0; c < kSubElems / 32 / N; ++c) {
          const int v = sub * kSubElems + (c * 32 + lane) * N;
          if (v + N <= p.vocab) {
            union { uint4 u; T e[N]; } tmp;
            tmp.u = __ldg(reinterpret_cast<const uint4 *>(row + v));
#pragma unroll
            for (int e = 0; e < N; ++e) consider(ld_as_float(tmp.e, e), v + e);
          } else {
            for (int e = 0; e < N && v + e < p.vocab; ++e) consider(ld_as_float(row, v + e), v + e);
          }
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
      consider(ov, oi);
    }
    if (lane == 0) s_arg[i] = best_i;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int n = k;
    for (int i = 0; i < k; ++i)
      if (p.draft_ids[d0 + i] != s_arg[i]) { n = i; break; }
    p.accepted_len[r] = n;
    for (int i = 0; i < n; ++i) p.out_tokens[t0 + i] = s_arg[i];
    p.out_tokens[t0 + n] = s_arg[n] == 0x7fffffff ? -1 : s_arg[n];
    for (int i = n + 1; i <= k; ++i) p.out_tokens[t0 + i] = -1;
  }
}

// A segment mass that its block has not written yet: a NaN with a payload no arithmetic produces.  The
// accept kernel fills a request's masses with it, the draw kernel waits for it to go away.
constexpr uint32_t kMassPending = 0x7fc0dead;

// One warp per request, lane = row (lanes 0..k: target rows, lanes k+1..2k: draft rows).  Each lane
// merges its row's segment pairs (fp32 exponentials, float64 sum); the accept ratios of all
// drafts are evaluated in parallel in float64 and the first failure fixes n.  Writes
// accepted_len, the accepted ids and the -1 padding; slot n is left for resid_pick_kernel.
template <typename T, bool kScaled, bool kFiltered>
__global__ void __launch_bounds__(128) accept_kernel(SampleParams p, int accept_blocks) {
  SPX_TL_SCOPE(kTlAccept);
  if (kScaled && (int)blockIdx.x >= accept_blocks) {  // variants: one extra block per request for the greedy ones
    greedy_request<T>(p, blockIdx.x - accept_blocks);
    return;
  }
  const int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (r >= p.batch) return;
  for (int i = lane; i < p.nseg; i += 32) p.seg_resid[(int64_t)r * p.nseg + i] = __uint_as_float(kMassPending);
  const int t0 = p.q_indptr[r];
  const int k = p.q_indptr[r + 1] - t0 - 1;
  const int d0 = t0 - r;
  const T *target = reinterpret_cast<const T *>(p.target);
  const T *draft = reinterpret_cast<const T *>(p.draft);
  const float nanf_ = __int_as_float(0x7fc00000);
  if (k < 0 || k > SPX_MAX_K || t0 < 0 || t0 + k + 1 > p.total_q) {
    if (lane == 0) {
      atomicOr(p.dev_status, SPX_DEV_BAD_LEN);
      p.accepted_len[r] = 0;
      p.req_norm[r] = make_float4(nanf_, nanf_, nanf_, -1.f);  // w < 0: skip this request
    }
    return;
  }
  int x = 0;
  bool bad = false;
  if (lane < k) {
    x = p.draft_ids[d0 + lane];
    bad = x < 0 || x >= p.vocab;
    if (p.diag_ratio) p.diag_ratio[d0 + lane] = nanf_;
  }
  if (__any_sync(0xffffffffu, bad)) {
    if (lane == 0) {
      atomicOr(p.dev_status, SPX_DEV_BAD_TOKEN);
      p.accepted_len[r] = 0;
      p.req_norm[r] = make_float4(nanf_, nanf_, nanf_, -1.f);
    }
    if (lane <= k) p.out_tokens[t0 + lane] = -1;
    return;
  }
  double scale = (double)kLog2e;
  if (kScaled) {
    const float tau = p.temperature ? p.temperature[r] : 1.f;
    const float tp = (kFiltered && p.top_p) ? p.top_p[r] : 1.f;
    if (!(tau >= 0.f) || tau == INFINITY || !(tp > 0.f && tp <= 1.f)) {
      if (lane == 0) {
        atomicOr(p.dev_status, SPX_DEV_BAD_PARAM);
        p.accepted_len[r] = 0;
        p.req_norm[r] = make_float4(nanf_, nanf_, nanf_, -1.f);
      }
      if (lane <= k) p.out_tokens[t0 + lane] = -1;
      return;
    }
    if (tau == 0.f) {  // greedy: decided by this launch's extra blocks, nothing for the residual pass
      if (lane == 0) p.req_norm[r] = make_float4(nanf_, nanf_, nanf_, -1.f);
      return;
    }
    scale = (double)p.row_scale[t0];
  }
  // row normalisers: M (log2 domain) and S = sum 2^(x - M)
  float M = -INFINITY;
  double S = 0.0;
  uint32_t thr = 0;  // filtering: order key of the row's lowest kept logit
  if (lane < 2 * k + 1) {
    const int row = lane <= k ? t0 + lane : p.total_q + d0 + (lane - k - 1);
    const float2 *st = p.seg_stats + (int64_t)row * p.nsub;
    for (int i = 0; i < p.nsub; ++i) M = fmaxf(M, st[i].x);
    for (int i = 0; i < p.nsub; ++i) S += (double)(st[i].y * fast_exp2(st[i].x - M));
    if (kFiltered) {
      const double z = p.row_z[row];
      if (z >= 0.0) { S = z; thr = p.row_thresh[row]; }
    }
  }
  // lane i < k pairs target row i (its own) with draft row i (lane k+1+i)
  const float Md = __shfl_sync(0xffffffffu, M, (k + 1 + lane) & 31);
  const double Sd = __shfl_sync(0xffffffffu, S, (k + 1 + lane) & 31);
  const uint32_t thr_d = __shfl_sync(0xffffffffu, thr, (k + 1 + lane) & 31);
  bool reject = false;
  if (lane < k) {
    double tx, dx;
    if (kScaled) {
      tx = (double)ld_as_float(target, (int64_t)(t0 + lane) * p.row_stride + x) * scale;
      dx = (double)ld_as_float(draft, (int64_t)(d0 + lane) * p.row_stride + x) * scale;
    } else {
      tx = (double)(ld_as_float(target, (int64_t)(t0 + lane) * p.row_stride + x) * kLog2e);
      dx = (double)(ld_as_float(draft, (int64_t)(d0 + lane) * p.row_stride + x) * kLog2e);
    }
    // rho = p(x)/q(x) = 2^(tx-Mt)/St * Sd/2^(dx-Md)
    double rho = exp2((tx - (double)M) - (dx - (double)Md)) * (Sd / S);
    if (kFiltered) {
      // a drafted token outside the target's kept set is rejected; one outside the draft's own kept
      // set (it cannot have been drafted) is accepted when the target keeps it
      const bool p_in = order_key32(ld_as_float(target, (int64_t)(t0 + lane) * p.row_stride + x)) >= thr;
      const bool q_in = order_key32(ld_as_float(draft, (int64_t)(d0 + lane) * p.row_stride + x)) >= thr_d;
      if (!p_in) rho = 0.0;
      else if (!q_in) rho = (double)INFINITY;
    }
    reject = !((double)p.u_accept[d0 + lane] < rho);
    if (p.diag_ratio) p.diag_ratio[d0 + lane] = (float)rho;
  }
  const uint32_t rej_mask = __ballot_sync(0xffffffffu, reject);
  const int n = rej_mask ? __ffs(rej_mask) - 1 : k;
  if (p.diag_ratio && lane < k && lane > n) p.diag_ratio[d0 + lane] = nanf_;  // rows after n are not consulted
  if (lane == 0) p.accepted_len[r] = n;
  if (lane < n) p.out_tokens[t0 + lane] = x;
  if (lane > n && lane <= k) p.out_tokens[t0 + lane] = -1;
  // normalisers of row n for the residual pass (target: lane n; draft: lane k+1+n)
  const float Mt_n = __shfl_sync(0xffffffffu, M, n);
  const double St_n = __shfl_sync(0xffffffffu, S, n);
  const float Md_n = __shfl_sync(0xffffffffu, M, (k + 1 + n) & 31);
  const double Sd_n = __shfl_sync(0xffffffffu, S, (k + 1 + n) & 31);
  if (lane == 0) {
    if (n < k) p.req_norm[r] = make_float4(Mt_n, (float)(1.0 / St_n), Md_n, (float)(1.0 / Sd_n));
    else p.req_norm[r] = make_float4(Mt_n, (float)(1.0 / St_n), nanf_, 0.f);
  }
  if (kFiltered) {
    const uint32_t tt = __shfl_sync(0xffffffffu, thr, n);
    const uint32_t td = __shfl_sync(0xffffffffu, thr, (k + 1 + n) & 31);
    if (lane == 0) p.req_thresh[r] = make_uint2(tt, n < k ? td : 0u);
  }
}

// What the two residual kernels need to know about request r: the normalisers of rows n, the
// filter thresholds, the row pointers and the probability terms of one token.
template <typename T, bool kScaled, bool kFiltered>
struct ResidCtx {
  float4 nm;        // (Mt, 1/St, Md, 1/Sd) of rows n; Md = NaN: bonus draw
  uint2 thr;        // order keys of the lowest kept logit of rows n (target, draft); 0 = unfiltered
  bool bonus, masked;
  int t0, n;
  float scale;      // log2(e)/tau of the request (variants), log2(e) otherwise
  const T *trow, *drow;
  static constexpr float kLoadScale = kScaled ? 1.f : kLog2e;

  // false: nothing to draw (an invalid request, or a greedy one decided beside the accept test)
  __device__ __forceinline__ bool init(const SampleParams &p, int r) {
    nm = p.req_norm[r];
    if (nm.w < 0.f) return false;
    bonus = (nm.z != nm.z);
    // filtering: tokens below the row's threshold carry no mass.  A masked request always takes
    // the full pass (the statistics of the unfiltered row are of no use to it), a bonus draw as a
    // residual against a draft term of zero.
    thr = make_uint2(0u, 0u);
    if (kFiltered) thr = p.req_thresh[r];
    masked = kFiltered && (thr.x != 0u || thr.y != 0u);
    t0 = p.q_indptr[r];
    n = p.accepted_len[r];
    // the variants keep the stored logit and scale it inside one fused multiply-add with the
    // maximum (a separately rounded product would cost |x * scale| * 2^-24 of relative accuracy,
    // which matters at low temperature); the base rule scales at load time
    scale = kScaled ? p.row_scale[t0] : kLog2e;
    trow = reinterpret_cast<const T *>(p.target) + (int64_t)(t0 + n) * p.row_stride;
    drow = reinterpret_cast<const T *>(p.draft) + (int64_t)(t0 - r + n) * p.row_stride;
    return true;
  }
  __device__ __forceinline__ bool full_pass() const { return !bonus || masked; }
  __device__ __forceinline__ float ex(float x, float M) const {
    return kScaled ? fast_exp2(fmaf(x, scale, -M)) : fast_exp2(x - M);
  }
  // probability terms of one token (xt, xd are stored logits whenever kFiltered)
  __device__ __forceinline__ float pt_of(float xt) const {
    const float v = ex(xt, nm.x) * nm.y;
    return (kFiltered && order_key32(xt) < thr.x) ? 0.f : v;
  }
  __device__ __forceinline__ float qd_of(float xd) const {
    if (kFiltered && (bonus || order_key32(xd) < thr.y)) return 0.f;
    return ex(xd, nm.z) * nm.w;
  }
  // residual weight max(0, p - q) of one token
  __device__ __forceinline__ float resid_of(float xt, float xd) const {
    if (kFiltered) return fmaxf(0.f, pt_of(xt) - qd_of(xd));
    return fmaxf(0.f, ex(xt, nm.x) * nm.y - ex(xd, nm.z) * nm.w);
  }
};

// Residual mass max(0, p - q) of each segment of rows n (and the kept target mass under
// filters).  grid = (nseg, B); bonus requests without a mask need no pass.  The masses are plain
// stores: the draw runs as the next kernel of the stream, so no fence or counter sits between a
// block's loads and its exit (with a last-block-done counter every block paid two more memory
// round trips, and the step's tail is made of these).
constexpr int kResidStageBytes = 2 * kSegElems * 2;  // bf16 logits: the block's segment of both rows
template <typename T, bool kScaled, bool kFiltered>
__global__ void __launch_bounds__(kResidThreads, sizeof(T) == 2 ? 6 : 1) resid_mass_kernel(SampleParams p) {
  SPX_TL_SCOPE(kTlResidMass);
  // the draw kernel may start once every block of this one runs: it waits for its own request's masses
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int seg_mine = blockIdx.x, r = blockIdx.y;
  ResidCtx<T, kScaled, kFiltered> c;
  if (!c.init(p, r) || !c.full_pass()) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __shared__ float s_w[kResidThreads / 32];
  __shared__ float s_wp[kResidThreads / 32];
  float acc = 0.f, accp = 0.f;
  if constexpr (sizeof(T) == 2) {
    // bf16 logits: each thread parks its vectors in shared memory with asynchronous copies and
    // reads them back itself (vector (c, thread) of a row holds tokens (c*256 + thread)*8 ..+8 of
    // the segment: every copy instruction of a warp covers 512 contiguous bytes).  Nothing of the
    // segment sits in registers while it is in flight, so six blocks share an SM and the pass
    // needs about one wave of blocks instead of two.
    extern __shared__ __align__(16) unsigned char resid_stage[];
    constexpr int N = 8, NV = kSegElems / N / kResidThreads;
    uint4 *stg = reinterpret_cast<uint4 *>(resid_stage);  // [row][vector][thread]
    auto park = [&](const T *row, int which) {
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        const int e0 = seg_mine * kSegElems + (v * kResidThreads + (int)threadIdx.x) * N;
        uint4 *dst = stg + (which * NV + v) * kResidThreads + threadIdx.x;
        if (e0 + N <= p.vocab) {
          cp_async16(dst, row + e0);
        } else {
          union { uint4 u; T e[N]; } tmp;
#pragma unroll
          for (int i = 0; i < N; ++i) {
            if (e0 + i < p.vocab) tmp.e[i] = row[e0 + i];
            else st_from_float(tmp.e, i, -INFINITY);
          }
          *dst = tmp.u;
        }
      }
    };
    park(c.trow, 0);
    if (!c.bonus) park(c.drow, 1);
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const uint4 ut = stg[v * kResidThreads + threadIdx.x];
      // a bonus request has no draft row: qd_of() is zero for it whatever is passed
      const uint4 ud = c.bonus ? ut : stg[(NV + v) * kResidThreads + threadIdx.x];
#pragma unroll
      for (int i = 0; i < N; ++i) {
        const float xt = raw_elem<T>(ut, i, c.kLoadScale), xd = raw_elem<T>(ud, i, c.kLoadScale);
        acc += c.resid_of(xt, xd);
        if (kFiltered) accp += c.pt_of(xt);
      }
    }
  } else {
    const int v0 = seg_mine * kSegElems + threadIdx.x * kElemsPerThread;
    RawSpan<T> st, sd;
    st.issue(c.trow, v0, p.vocab);
    if (!c.bonus) sd.issue(c.drow, v0, p.vocab);
    else sd = st;  // never read as a draft row: qd_of() is zero for a bonus request
#pragma unroll
    for (int i = 0; i < kElemsPerThread; ++i) {
      const float xt = st.get(i, c.kLoadScale), xd = sd.get(i, c.kLoadScale);
      acc += c.resid_of(xt, xd);
      if (kFiltered) accp += c.pt_of(xt);
    }
  }
  acc = warp_sum(acc);
  if (kFiltered) accp = warp_sum(accp);
  if (lane == 0) { s_w[warp] = acc; if (kFiltered) s_wp[warp] = accp; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
    for (int w = 0; w < kResidThreads / 32; ++w) tot += s_w[w];
    if (kFiltered) {
      float totp = 0.f;
      for (int w = 0; w < kResidThreads / 32; ++w) totp += s_wp[w];
      p.seg_pmass[(int64_t)r * p.nseg + seg_mine] = totp;
      __threadfence();   // the draw kernel reads it once it has seen the residual mass below
    }
    p.seg_resid[(int64_t)r * p.nseg + seg_mine] = tot;
  }
}

// The final draw of request r = blockIdx.x: segment choice in float64 over the segment masses,
// token choice by an fp32 scan of the chosen segment (thread t owns tokens [32t, 32t+32) of it).
// Launched with programmatic stream serialization behind resid_mass_kernel, whose blocks release it
// as they start: what the accept kernel left is read at once, the masses of the request's own
// segments as their blocks write them.
template <typename T, bool kScaled, bool kFiltered>
__global__ void __launch_bounds__(kResidThreads, sizeof(T) == 2 ? 4 : 1) resid_pick_kernel(SampleParams p) {
  SPX_TL_SCOPE(kTlResidPick);
  const int r = blockIdx.x;
  ResidCtx<T, kScaled, kFiltered> c;
  const bool live = c.init(p, r);
  const float u = p.u_sample[r];
  if (!live) return;
  const bool bonus = c.bonus, masked = c.masked;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float2 *tstats = p.seg_stats + (int64_t)(c.t0 + c.n) * p.nsub;
  // probability mass of segment i of the target row, from its sub-segment statistics
  auto target_mass = [&](int i) -> double {
    if (masked) return (double)p.seg_pmass[(int64_t)r * p.nseg + i];
    double acc = 0.0;
    for (int j = i * kSubPerSeg; j < min((i + 1) * kSubPerSeg, p.nsub); ++j)
      acc += (double)(tstats[j].y * fast_exp2(tstats[j].x - c.nm.x));
    return acc * (double)c.nm.y;
  };
  // The segment masses are fetched by one thread each before the scan (one memory round trip for
  // the lot; a scan that loads as it goes pays one round trip per segment, 10 us on a 128k
  // vocabulary).  Segments beyond the staging array, if any, are read in place.
  constexpr int kStageSegs = 128;
  __shared__ double s_mass[kStageSegs];
  __shared__ int s_seg;
  __shared__ float s_target;
  __shared__ int s_degenerate;
  __shared__ float s_scan[kResidThreads / 32];
  __shared__ int s_tok;
  const float *resid = p.seg_resid + (int64_t)r * p.nseg;
  auto stage = [&](bool from_target) {
    for (int i = threadIdx.x; i < min(p.nseg, kStageSegs); i += kResidThreads)
      s_mass[i] = from_target ? target_mass(i) : (double)resid[i];
    __syncthreads();
  };
  auto mass_at = [&](int i, bool from_target) -> double {
    return i < kStageSegs ? s_mass[i] : from_target ? target_mass(i) : (double)resid[i];
  };
  bool use_target = bonus && !masked;
  if (use_target) {
    stage(true);
  } else {
    // The residual masses of this request's segments.  The draw is launched while the mass blocks
    // still run (every one of them is resident or done by then, so waiting for them cannot starve
    // them): each thread waits for one mass to appear - with a limit, like every wait of the
    // library - and has it in hand when it does, so the masses cost no round trip of their own.
    for (int i = threadIdx.x; i < p.nseg; i += kResidThreads) {
      const long long t_start = clock64();
      uint32_t bits;
      for (;;) {
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(bits) : "l"(resid + i) : "memory");
        if (bits != kMassPending) break;
        if (clock64() - t_start > kWaitLimitCycles) { atomicOr(p.dev_status, SPX_DEV_TIMEOUT); bits = 0u; break; }
        __nanosleep(32);
      }
      if (i < kStageSegs) s_mass[i] = (double)__uint_as_float(bits);
    }
    __syncthreads();
  }
  // Total mass R, target u * R, first segment whose inclusive sum exceeds it (float64).  Up to 32
  // segments (a vocabulary of 262144) are scanned by warp 0 with shuffles - a thread that walks
  // them alone pays a shared-memory latency and a float64 add per segment, three times over, on
  // the step's critical path; more segments are walked by one thread.
  const bool by_warp = p.nseg <= 32;
  auto warp_pick = [&](bool from_target) -> double {   // warp 0; returns R, leaves s_seg / s_target
    const double m = lane < p.nseg ? s_mass[lane] : 0.0;
    double incl = m;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double nb = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += nb;
    }
    const double R = __shfl_sync(0xffffffffu, incl, 31);
    const double target = (double)u * R;
    const uint32_t over = __ballot_sync(0xffffffffu, lane < p.nseg && incl > target);
    const uint32_t pos = __ballot_sync(0xffffffffu, m > 0.0);
    // rounding can leave the target unreached at the end: the last segment with mass takes it
    const int seg = over ? __ffs(over) - 1 : pos ? 31 - __clz(pos) : -1;
    if (lane == (seg < 0 ? 0 : seg)) {
      s_seg = seg;
      s_target = (float)(target - (incl - m));
      s_tok = 0x7fffffff;
    }
    (void)from_target;
    return R;
  };
  if (by_warp) {
    if (warp == 0) {
      const double R = warp_pick(use_target);
      if (lane == 0) s_degenerate = !use_target && !(R > 0.0);
    }
  } else if (threadIdx.x == 0) {
    double R = 0.0;
    for (int i = 0; i < p.nseg; ++i) R += mass_at(i, use_target);
    s_degenerate = !use_target && !(R > 0.0);
  }
  __syncthreads();
  if (s_degenerate) {  // the residual is identically zero: draw from the target row instead
    use_target = true;
    stage(true);
    if (threadIdx.x == 0) atomicOr(p.dev_status, SPX_DEV_DEGENERATE);
    if (by_warp) {
      if (warp == 0) warp_pick(true);
      __syncthreads();
    }
  }
  if (!by_warp) {
    if (threadIdx.x == 0) {
      double R = 0.0;
      for (int i = 0; i < p.nseg; ++i) R += mass_at(i, use_target);
      const double target = (double)u * R;
      double cum = 0.0;
      int seg = -1, last_pos = -1;
      double before = 0.0, last_before = 0.0;
      for (int i = 0; i < p.nseg; ++i) {
        const double mass = mass_at(i, use_target);
        if (mass > 0.0) { last_pos = i; last_before = cum; }
        if (cum + mass > target) { seg = i; before = cum; break; }
        cum += mass;
      }
      if (seg < 0) { seg = last_pos; before = last_before; }
      s_seg = seg;
      s_target = (float)(target - before);
      s_tok = 0x7fffffff;
    }
    __syncthreads();
  }
  const int seg = s_seg;
  if (seg < 0) {  // no mass anywhere (cannot happen for finite logits)
    if (threadIdx.x == 0) p.out_tokens[c.t0 + c.n] = -1;
    return;
  }
  const float target = s_target;
  const int v0 = seg * kSegElems + threadIdx.x * kElemsPerThread;
  float w[kElemsPerThread];
  {
    RawSpan<T> st;
    st.issue(c.trow, v0, p.vocab);
    if (use_target || (kFiltered && bonus)) {
#pragma unroll
      for (int i = 0; i < kElemsPerThread; ++i) {
        const float xt = st.get(i, c.kLoadScale);
        w[i] = kFiltered ? c.pt_of(xt) : c.ex(xt, c.nm.x) * c.nm.y;
      }
    } else {
      RawSpan<T> sd;
      sd.issue(c.drow, v0, p.vocab);
#pragma unroll
      for (int i = 0; i < kElemsPerThread; ++i) w[i] = c.resid_of(st.get(i, c.kLoadScale), sd.get(i, c.kLoadScale));
    }
  }
  float tsum = 0.f;
#pragma unroll
  for (int i = 0; i < kElemsPerThread; ++i) tsum += w[i];
  // block exclusive scan of thread sums
  float incl = tsum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const float nb = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += nb;
  }
  if (lane == 31) s_scan[warp] = incl;
  __syncthreads();
  float woff = 0.f;
  for (int i = 0; i < warp; ++i) woff += s_scan[i];
  const float excl = woff + incl - tsum;
  // the thread whose span contains the crossing walks it; if rounding leaves its running sum
  // short of the target it takes its last token with positive weight
  if (excl <= target && excl + tsum > target) {
    float cum = excl;
    int tok = -1, last = -1;
#pragma unroll
    for (int i = 0; i < kElemsPerThread; ++i) {
      cum += w[i];
      if (w[i] > 0.f) last = v0 + i;
      if (tok < 0 && cum > target) tok = v0 + i;
    }
    if (tok < 0) tok = last;
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
  if (threadIdx.x == 0) p.out_tokens[c.t0 + c.n] = s_tok;
}

}  // namespace spx
