// Shared device helpers for the verify-step kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "spx.h"

namespace spx {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kTileTokens = 128;   // KV tokens per attention tile (both attention kernels plan in this unit)

// ------------------------------------------------------------------------------------------
// Timeline builds (-DSPX_TIMELINE=1; see build.py and `bench.py --timeline`): every kernel of the
// step stamps %globaltimer per CTA at entry and exit into a device array that
// spx_debug_timeline copies out: slot [kernel][cta] = {start ns, end ns, SM id, 0}.  The end is
// the latest exit of the CTA's warps.  Costs about 1.5 us per step; compiled out otherwise.
// ------------------------------------------------------------------------------------------
#ifndef SPX_TIMELINE
#define SPX_TIMELINE 0
#endif
constexpr int kTlKernels = 8;        // plan, attention, combine, logits statistics, accept, residual masses, draw, spare
constexpr int kTlCtas = 4096;        // CTAs recorded per kernel
#if SPX_TIMELINE
__device__ unsigned long long g_timeline[kTlKernels * kTlCtas * 4];
struct TlScope {
  unsigned long long *slot;
  __device__ __forceinline__ static unsigned long long now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
  }
  __device__ __forceinline__ explicit TlScope(int kernel_id) : slot(nullptr) {
    const int cta = blockIdx.x + blockIdx.y * gridDim.x;
    if (cta < kTlCtas) {
      slot = g_timeline + ((size_t)kernel_id * kTlCtas + cta) * 4;
      if (threadIdx.x == 0) {
        unsigned sm;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
        slot[0] = now();
        slot[2] = sm;
      }
    }
  }
  __device__ __forceinline__ ~TlScope() {
    if (slot && (threadIdx.x & 31) == 0) atomicMax(slot + 1, now());
  }
};
#define SPX_TL_SCOPE(id) TlScope spx_tl_scope_(id)
#else
#define SPX_TL_SCOPE(id) do { } while (0)
#endif
enum { kTlPlan = 0, kTlAttention = 1, kTlCombine = 2, kTlLogitStats = 3, kTlAccept = 4, kTlResidMass = 5, kTlResidPick = 6 };

__device__ __forceinline__ float ld_as_float(const float *p, int64_t i) { return p[i]; }
__device__ __forceinline__ float ld_as_float(const __nv_bfloat16 *p, int64_t i) { return __bfloat162float(p[i]); }

__device__ __forceinline__ void st_from_float(float *p, int64_t i, float v) { p[i] = v; }
__device__ __forceinline__ void st_from_float(__nv_bfloat16 *p, int64_t i, float v) { p[i] = __float2bfloat16_rn(v); }

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ------------------------------------------------------------------------------------------
// Work plan shared by the attention kernels.  Built on the device by plan_kernel so that no
// host copy of seq_lens is needed.
//
// A pair is one (request, kv head); its KV range is tiles_r tiles of kTileTokens tokens.  The
// pairs of the valid requests, in (request, head) order, form one tile axis of length T, which is
// cut into n_cta contiguous ranges of equal cost (tiles plus a fixed cost per pair); CTA c of a
// persistent kernel executes range c (entries cta_off[c] .. cta_off[c+1] of the work list, in
// axis order).  A cut within kSnapTiles
// of a pair boundary moves onto it, so most pairs stay whole; a pair that k cuts cross has k+1
// chunks, whose partial results the combine kernel merges.  At most n_cta - 1 pairs are split,
// whatever the length mix.
// ------------------------------------------------------------------------------------------
constexpr int kSnapTiles = 2;   // a cut this close to a pair boundary is moved onto the boundary
struct PlanHeader {
  int32_t n_work;        // number of work entries
  int32_t n_cta;         // ranges the tile axis was cut into
  int32_t n_part_slots;  // partial-result slots in use (chunks of split pairs)
  int32_t total_tiles;   // sum over requests of tiles (one kv-head)
  int32_t work_counter;  // dynamic scheduler cursor (SIMT kernel), zeroed by the planner
  int32_t overflow;      // 1 if the plan did not fit the workspace (nothing is executed then)
  int32_t n_combine;     // pairs the combine kernel has work for (split pairs, pairs of invalid requests)
  int32_t pad[1];
};

// What the combine kernel needs to know of a pair, in one load.
struct __align__(16) CombineEntry {
  int32_t pair;       // request * Hkv + kv head; -1: past the end of the list
  int32_t nch;        // chunks of the pair (0: invalid request, sentinel rows)
  int32_t part_base;  // first partial slot
  int32_t q0, m;      // first query row and number of query rows of the request
  int32_t pad[3];
};
constexpr int kCombineListPad = 148;   // entries the planner always writes (the combine kernel's blocks read their first entry unconditionally)

struct __align__(16) WorkEntry {
  int32_t req;         // request index
  int32_t tile_begin;  // first tile of the chunk
  int32_t tile_end;    // one past the last tile
  int32_t part_slot;   // partial slot, or -1 when the pair is not split (direct output)
  int32_t q0;          // q_indptr[req]: first query row of the request
  int32_t m;           // k+1 query positions
  int32_t L;           // seq_lens[req]
  int32_t g;           // kv head
};

struct AttnParams {
  int32_t batch, total_q, max_q_len, Hq, Hkv, G, D, P, log2P, num_pages, max_pages_per_req;
  float scale_log2;  // sm_scale * log2(e)
  const void *q;
  const void *k_cache;
  const void *v_cache;
  int64_t stride_page, stride_head, stride_token;
  const int32_t *block_table;
  const int32_t *seq_lens;
  const int32_t *q_indptr;
  void *out;
  float *lse;
  // plan + partials (workspace)
  PlanHeader *hdr;
  int32_t *pair_nchunks;   // [B*Hkv]  chunks of the pair, 0 = invalid request
  int32_t *pair_part_base; // [B*Hkv]  first partial slot of a split pair
  CombineEntry *combine_list;  // [max(B*Hkv, kCombineListPad)]  the pairs the combine kernel has work for: n_combine entries, then pair = -1
  int32_t *tile_prefix;    // [B+1]  tiles of the requests before r (one kv head)
  int32_t *valid_prefix;   // [B+1]  valid requests before r
  int32_t *cost_prefix;    // [B+1]  planning cost (one kv head) of the requests before r
  int32_t *cta_off;        // [n_cta+1]  work entries of the CTAs before c
  int32_t *req_bad;        // [B]  set when a needed page id was out of range
  int32_t head_inner;      // tensor-map dimension order: 1 = (d, head, token, page), 0 = (d, token, head, page)
  WorkEntry *work;         // [max_work]
  int32_t max_work;
  int32_t max_part_slots;
  float *part_o;           // [slot][rows_cap][D]
  float2 *part_ml;         // [slot][rows_cap]  (m in log2 domain, l)
  int32_t rows_cap;        // G * max_q_len
  int32_t q_box_rows;      // query positions one Q box of the tensor-core kernel fetches (<= max_q_len)
  int32_t *dev_status;
  long long *prof;         // optional per-CTA cycle counters (profiling builds only), else NULL
};

// Every spin on a barrier in this library gives up after this many clock cycles (about a second at
// the default), raises SPX_DEV_TIMEOUT and makes the other roles of its CTA leave too.  The
// wait-test build (build.py: build_wait_test) compiles a limit of some tens of microseconds and a
// small kernel that lets each of the wait helpers run out on purpose (spx_debug_wait_expiry).
#ifndef SPX_WAIT_LIMIT_CYCLES
#define SPX_WAIT_LIMIT_CYCLES (1ll << 31)
#endif
constexpr long long kWaitLimitCycles = SPX_WAIT_LIMIT_CYCLES;
#ifndef SPX_WAIT_TEST
#define SPX_WAIT_TEST 0
#endif

#ifndef SPX_PROFILE
#define SPX_PROFILE 0
#endif
constexpr bool kProfile = SPX_PROFILE != 0;
constexpr int kProfSlots = 16;

}  // namespace spx
