// Verify attention on the 5th-generation tensor cores (tcgen05 + TMEM) fed by TMA page gathers.
//
// One persistent CTA per SM, warp-specialised:
//   warp 0      producer: reads the block table and issues one TMA box per (page, 64-column half)
//               for K and for V into a ring of shared-memory stages (128-byte swizzle);
//   warp 1      MMA issuer (one lane): S = Q K^T into one of two TMEM score buffers, O += P V with
//               P read from TMEM and V as an MN-major shared-memory operand;
//   warps 2-5   softmax: thread = packed query row (TMEM lane).  Online softmax in the log2
//               domain with lazy rescaling of the TMEM-resident O (only when the running maximum
//               grows by more than 2^8), P written back over the score buffer as bf16, epilogue.
// The G*(k+1) query rows that share a kv-head are packed into the M dimension of one tile, so each
// K/V byte is fetched once for all of them.  Work items come from the plan (chunks of 128-token
// tiles of one (request, kv head) pair; CTA c walks its own range of the list); the chunks of a
// split pair write fp32 partials that combine_kernel merges.
//
// Every wait is bounded: on expiry the CTA raises SPX_DEV_TIMEOUT, all roles leave their loops,
// pending copies get time to land and TMEM is released.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace spx {

constexpr int kTcThreads = 192;
#ifndef SPX_RESCALE_THRESHOLD
#define SPX_RESCALE_THRESHOLD 8.f
#endif
constexpr float kRescaleThreshold = SPX_RESCALE_THRESHOLD;  // log2 units

template <int D, int QROWS>
struct TcCfg {
  static constexpr int kHalves = D / 64;                   // 64-element (128-byte) column halves
  static constexpr int kHalfBytes = kTileTokens * 128;     // one half of a K or V tile
  static constexpr int kTileBytes = kHalves * kHalfBytes;  // K or V tile
  static constexpr int kQHalfBytes = QROWS * 128;
  static constexpr int kQBytes = kHalves * kQHalfBytes;
  static constexpr int kBarBytes = 1024;
  static constexpr int kBudget = 232448 - 1024 - kBarBytes - 2 * kQBytes;
  static constexpr int kStagesRaw = kBudget / (2 * kTileBytes);
  static constexpr int kStages = kStagesRaw > 4 ? 4 : kStagesRaw;
  static constexpr int kSmemBytes = 1024 + 2 * kQBytes + kStages * 2 * kTileBytes + kBarBytes;
  static constexpr int kTmemCols = 512;
  static constexpr int kColS0 = 0, kColS1 = 128, kColO = 256;
  static_assert(kStages >= 2, "need at least two stages");
};

struct TcBarriers {
  uint64_t k_full[4], v_full[4], k_empty[4], v_empty[4];
  uint64_t s_full[2], p_full[2], q_full[2], q_empty[2];
  uint64_t pv_done[2], o_free, o_free2[2], e_bar;  // pv_done alternates per tile: a waiter may lag the MMA by two tiles
  uint32_t tmem_base;
  volatile int32_t abort;
};

namespace tc {

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t *b, uint32_t cnt) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(cnt));
}
__device__ __forceinline__ void mbar_arrive(uint64_t *b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *b, uint32_t parity) {
  uint32_t ok;
  asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
               : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: gives up after kWaitLimitCycles (about a second) or when another role aborted.
__device__ __forceinline__ bool mbar_wait(uint64_t *b, uint32_t parity, TcBarriers *bars, int32_t *dev_status) {
  if (mbar_try_wait(b, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(b, parity)) return true;
    if (bars->abort) return false;
    if (clock64() - t0 > kWaitLimitCycles) {
      bars->abort = 1;
      atomicOr(dev_status, SPX_DEV_TIMEOUT);
      return false;
    }
  }
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
// shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr >> 4) & 0x3fff) | ((uint64_t)((lbo_bytes >> 4) & 0x3fff) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3fff) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p; }"
               ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p; }"
               ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]),
        "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]),
        "r"(r[30]), "r"(r[31]) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t *>(&b);
}

// instruction descriptor: D fp32, A/B bf16, M = 128; b_major = 1 for the MN-major V operand
__host__ __device__ constexpr uint32_t idesc(uint32_t n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

struct ItemInfo {
  int req, g, q0, m, L, R, tile_begin, tile_end, part_slot, t_end;
};

}  // namespace tc

template <int D, int QROWS>
__global__ void __launch_bounds__(kTcThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap, AttnParams p) {
  SPX_TL_SCOPE(kTlAttention);
  // the combine kernel may take its places now (it reads the planner's list, then waits for this
  // kernel to end): its launch then costs nothing behind the last CTA
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  using Cfg = TcCfg<D, QROWS>;
  using namespace tc;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char *sQ = smem;                                 // two Q buffers
  unsigned char *sK = smem + 2 * Cfg::kQBytes;              // kStages K tiles
  unsigned char *sV = sK + Cfg::kStages * Cfg::kTileBytes;  // kStages V tiles
  TcBarriers *bars = reinterpret_cast<TcBarriers *>(sV + Cfg::kStages * Cfg::kTileBytes);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < 4; ++s) { mbar_init(&bars->k_full[s], 1); mbar_init(&bars->v_full[s], 1); mbar_init(&bars->k_empty[s], 1); mbar_init(&bars->v_empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&bars->s_full[b], 1); mbar_init(&bars->p_full[b], 4); mbar_init(&bars->q_full[b], 4); mbar_init(&bars->q_empty[b], 1); }
    mbar_init(&bars->pv_done[0], 1);
    mbar_init(&bars->pv_done[1], 1);
    mbar_init(&bars->o_free, 4);
    bars->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "n"(Cfg::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem = bars->tmem_base;
  // the plan is read from here on: under programmatic dependent launch, wait for the planner
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // this CTA's range of the plan: entries cta_off[c] .. cta_off[c+1] of the work list, in order
  const bool planned = !p.hdr->overflow && (int)blockIdx.x < p.hdr->n_cta;
  const int item_begin = planned ? p.cta_off[blockIdx.x] : 0;
  const int item_end = planned ? p.cta_off[blockIdx.x + 1] : 0;
  auto item_index = [&](int it) -> int { return item_begin + it < item_end ? item_begin + it : -1; };
  auto load_item = [&](int idx, ItemInfo &I) {
    const WorkEntry we = p.work[idx];
    I.req = we.req; I.g = we.g; I.tile_begin = we.tile_begin; I.tile_end = we.tile_end; I.part_slot = we.part_slot;
    I.q0 = p.q_indptr[we.req];
    I.m = p.q_indptr[we.req + 1] - I.q0;
    I.L = p.seq_lens[we.req];
    I.R = I.m * p.G;
    I.t_end = min(we.tile_end * kTileTokens, I.L);
  };
  const int pages_per_tile = kTileTokens >> p.log2P;
  // warp-uniform bounded wait (all lanes poll; the outcome is shared so that the warp never
  // diverges around the .sync.aligned tensor-memory instructions)
  auto warp_wait = [&](uint64_t *bar, uint32_t parity) -> bool {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, bars, p.dev_status));
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    uint32_t tc_ = 0;
    for (int it = 0;; ++it) {
      const int idx = item_index(it);
      if (idx < 0 || bars->abort) break;
      ItemInfo I;
      load_item(idx, I);
      const int32_t *bt = p.block_table + (int64_t)I.req * p.max_pages_per_req;
      bool ok = true;
      for (int tile = I.tile_begin; tile < I.tile_end && ok; ++tile, ++tc_) {
        const int slot = tc_ % Cfg::kStages;
        const uint32_t ph = (tc_ / Cfg::kStages) & 1;
        const int ntok = min(kTileTokens, I.t_end - tile * kTileTokens);
        const int npages = (ntok + p.P - 1) >> p.log2P;
        int page = 0;
        if (lane < npages) {
          page = bt[tile * pages_per_tile + lane];
          if (page < 0 || page >= p.num_pages) {
            page = 0;  // keep the copy in bounds; the request is flagged and its rows are voided
            atomicOr(p.dev_status, SPX_DEV_BAD_PAGE);
            p.req_bad[I.req] = 1;
          }
        }
        const uint32_t bytes = (uint32_t)npages * p.P * D * 2;
        ok = warp_wait(&bars->k_empty[slot], ph ^ 1);
        if (!ok) break;
        if (lane == 0) mbar_expect_tx(&bars->k_full[slot], bytes);
        if (lane < npages) {
#pragma unroll
          for (int h = 0; h < Cfg::kHalves; ++h)
            tma_load_4d(smem_u32(sK + slot * Cfg::kTileBytes + h * Cfg::kHalfBytes + lane * p.P * 128), &kmap,
                        &bars->k_full[slot], h * 64, p.head_inner ? I.g : 0, p.head_inner ? 0 : I.g, page);
        }
        ok = warp_wait(&bars->v_empty[slot], ph ^ 1);
        if (!ok) break;
        if (lane == 0) mbar_expect_tx(&bars->v_full[slot], bytes);
        if (lane < npages) {
#pragma unroll
          for (int h = 0; h < Cfg::kHalves; ++h)
            tma_load_4d(smem_u32(sV + slot * Cfg::kTileBytes + h * Cfg::kHalfBytes + lane * p.P * 128), &vmap,
                        &bars->v_full[slot], h * 64, p.head_inner ? I.g : 0, p.head_inner ? 0 : I.g, page);
        }
      }
      if (!ok) break;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t kIdescQK = idesc(kTileTokens, false);
      constexpr uint32_t kIdescPV = idesc(D, true);
      uint32_t tc_ = 0, qc = 0;
      bool ok = true;
      auto issue_qk = [&](uint32_t t, uint32_t qb) -> bool {
        const int slot = t % Cfg::kStages;
        if (!mbar_wait(&bars->k_full[slot], (t / Cfg::kStages) & 1, bars, p.dev_status)) return false;
        fence_after();
        const uint32_t qa = smem_u32(sQ + qb * Cfg::kQBytes), ka = smem_u32(sK + slot * Cfg::kTileBytes);
        const uint32_t ts = tmem + ((t & 1) ? Cfg::kColS1 : Cfg::kColS0);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t qoff = (k / 4) * Cfg::kQHalfBytes + (k % 4) * 32;
          const uint32_t koff = (k / 4) * Cfg::kHalfBytes + (k % 4) * 32;
          mma_ss(ts, smem_desc(qa + qoff, 16, 1024), smem_desc(ka + koff, 16, 1024), kIdescQK, k > 0);
        }
        mma_commit(&bars->s_full[t & 1]);
        mma_commit(&bars->k_empty[slot]);
        return true;
      };
      for (int it = 0; ok; ++it, ++qc) {
        const int idx = item_index(it);
        if (idx < 0 || bars->abort) break;
        const WorkEntry we = p.work[idx];
        const int n_tiles = we.tile_end - we.tile_begin;
        const uint32_t qb = qc & 1;
        ok = mbar_wait(&bars->q_full[qb], (qc >> 1) & 1, bars, p.dev_status);
        if (!ok) break;
        for (int i = 0; i < n_tiles && ok; ++i, ++tc_) {
          if (i == 0) ok = issue_qk(tc_, qb);
          if (ok && i + 1 < n_tiles) ok = issue_qk(tc_ + 1, qb);
          if (ok && i + 1 >= n_tiles) mma_commit(&bars->q_empty[qb]);  // last QK of the item has been issued
          if (!ok) break;
          ok = mbar_wait(&bars->p_full[tc_ & 1], (tc_ >> 1) & 1, bars, p.dev_status);
          if (ok && i == 0 && qc > 0) ok = mbar_wait(&bars->o_free, (qc - 1) & 1, bars, p.dev_status);
          const int slot = tc_ % Cfg::kStages;
          if (ok) ok = mbar_wait(&bars->v_full[slot], (tc_ / Cfg::kStages) & 1, bars, p.dev_status);
          if (!ok) break;
          fence_after();
          const uint32_t va = smem_u32(sV + slot * Cfg::kTileBytes);
          const uint32_t tp = tmem + ((tc_ & 1) ? Cfg::kColS1 : Cfg::kColS0);
#pragma unroll
          for (int k = 0; k < kTileTokens / 16; ++k)
            mma_ts(tmem + Cfg::kColO, tp + k * 8, smem_desc(va + k * 2 * 1024, Cfg::kHalfBytes, 1024), kIdescPV, (i > 0) || (k > 0));
          mma_commit(&bars->v_empty[slot]);
          mma_commit(&bars->pv_done[tc_ & 1]);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax / epilogue
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const int sm_tid = tid - 64;  // 0..127 among the softmax threads
    const __nv_bfloat16 *Qg = reinterpret_cast<const __nv_bfloat16 *>(p.q);
    __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(p.out);
    constexpr int kChunksPerRow = D / 8;  // 16-byte chunks per Q row

    // Q rows of an item -> shared memory, K-major with the 128-byte swizzle the MMA expects
    auto stage_q = [&](const ItemInfo &I, uint32_t qb) {
      unsigned char *dst = sQ + qb * Cfg::kQBytes;
      for (int i = sm_tid; i < I.R * kChunksPerRow; i += 128) {
        const int r = i / kChunksPerRow, c16 = i % kChunksPerRow, h = c16 >> 3, c = c16 & 7;
        const int j = r / p.G, hg = r % p.G;
        const uint4 v = *reinterpret_cast<const uint4 *>(Qg + ((int64_t)(I.q0 + j) * p.Hq + I.g * p.G + hg) * D + c16 * 8);
        *reinterpret_cast<uint4 *>(dst + h * Cfg::kQHalfBytes + (r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4)) = v;
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->q_full[qb]);
    };

    uint32_t tc_ = 0, qc = 0;
    bool ok = true;
    ItemInfo I, Inext;
    int idx = item_index(0);
    if (idx >= 0) { load_item(idx, I); stage_q(I, 0); }
    for (int it = 0; idx >= 0 && ok; ++it, ++qc) {
      if (bars->abort) break;
      // stage the next item's Q while this item streams
      const int idx_next = item_index(it + 1);
      if (idx_next >= 0) {
        load_item(idx_next, Inext);
        const uint32_t nb = (qc + 1) & 1;
        if (qc >= 1) ok = warp_wait(&bars->q_empty[nb], ((qc - 1) >> 1) & 1);
        if (!ok) break;
        stage_q(Inext, nb);
      }
      const bool active = quad * 32 < I.R;
      float m_ref = -INFINITY, l_sum = 0.f;
      const int limit = I.L - I.m + row / p.G;  // last visible token of this row
      for (int tile = I.tile_begin; tile < I.tile_end && ok; ++tile, ++tc_) {
        const uint32_t b = tc_ & 1;
        const uint32_t ts = tmem + (b ? Cfg::kColS1 : Cfg::kColS0) + lane_addr;
        const int t0 = tile * kTileTokens;
        const bool mask_tile = t0 + kTileTokens - 1 > I.L - I.m;
        ok = warp_wait(&bars->s_full[b], (tc_ >> 1) & 1);
        if (!ok) break;
        fence_after();
        if (active) {
          // pass 1: row maximum of this tile
          float mx = -INFINITY;
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld32(ts + c * 32, r);
            wait_ld();
            if (mask_tile) {
#pragma unroll
              for (int i = 0; i < 32; ++i) mx = fmaxf(mx, (t0 + c * 32 + i <= limit) ? __uint_as_float(r[i]) : -INFINITY);
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(r[i]));
            }
          }
          mx *= p.scale_log2;
          // lazy rescale: move the reference maximum only when it would grow by more than 2^8.
          // A row that has seen no visible token yet adopts the tile maximum for free (its O is
          // exactly zero so far, or about to be overwritten by the first PV of the item).
          const bool valid_row = row < I.R;
          float alpha = 1.f;
          bool need_scale = false;
          if (valid_row) {
            if (m_ref == -INFINITY) {
              m_ref = mx;
            } else if (mx > m_ref + kRescaleThreshold) {
              alpha = fast_exp2(m_ref - mx);
              m_ref = mx;
              l_sum *= alpha;
              need_scale = true;
            }
          }
          if (__any_sync(0xffffffffu, need_scale)) {
            // O holds contributions of earlier tiles: wait for the last PV, then scale the rows
            ok = warp_wait(&bars->pv_done[(tc_ - 1) & 1], ((tc_ - 1) >> 1) & 1);
            if (!ok) break;
            fence_after();
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
              uint32_t r[32];
              tmem_ld32(tmem + Cfg::kColO + lane_addr + c * 32, r);
              wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
              tmem_st32(tmem + Cfg::kColO + lane_addr + c * 32, r);
            }
          }
          // pass 2: P = 2^(s*scale - m_ref) as bf16 over the score buffer, row sum in fp32
          const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
          float sum = 0.f;
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld32(ts + c * 32, r);
            wait_ld();
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              float s0 = __uint_as_float(r[2 * i]), s1 = __uint_as_float(r[2 * i + 1]);
              if (mask_tile) {
                s0 = (t0 + c * 32 + 2 * i <= limit) ? s0 : -INFINITY;
                s1 = (t0 + c * 32 + 2 * i + 1 <= limit) ? s1 : -INFINITY;
              }
              const float p0 = fast_exp2(fmaf(s0, p.scale_log2, -m_use));
              const float p1 = fast_exp2(fmaf(s1, p.scale_log2, -m_use));
              sum += p0 + p1;
              pk[i] = pack_bf16(p0, p1);
            }
            tmem_st16(ts + c * 16, pk);
          }
          l_sum += sum;
          wait_st();
        }
        // the last tile of a request may end inside the tile: rows of V past the end must be zero
        // (their weights are zero, but stale or uninitialised bytes could be NaN/Inf)
        const int ntok = min(kTileTokens, I.t_end - t0);
        if (ntok < kTileTokens) {
          const int slot = tc_ % Cfg::kStages;
          ok = warp_wait(&bars->v_full[slot], (tc_ / Cfg::kStages) & 1);
          if (!ok) break;
          unsigned char *vt = sV + slot * Cfg::kTileBytes;
          const int n_chunks = (kTileTokens - ntok) * 8 * Cfg::kHalves;  // 16-byte chunks to clear
          for (int i = sm_tid; i < n_chunks; i += 128) {
            const int h = i / ((kTileTokens - ntok) * 8), rem = i % ((kTileTokens - ntok) * 8);
            const int tok = ntok + rem / 8, c = rem % 8;
            *reinterpret_cast<uint4 *>(vt + (tok >> 3) * 1024 + h * Cfg::kHalfBytes + (tok & 7) * 128 + c * 16) = make_uint4(0, 0, 0, 0);
          }
          fence_async_smem();
        }
        fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->p_full[b]);
      }
      if (!ok) break;
      // epilogue: wait for the last PV of the item, normalise and store
      ok = warp_wait(&bars->pv_done[(tc_ - 1) & 1], ((tc_ - 1) >> 1) & 1);
      if (!ok) break;
      fence_after();
      if (active) {
        const bool valid_row = row < I.R;
        const int j = row / p.G, hg = row % p.G;
        if (I.part_slot < 0) {
          const float inv = 1.f / l_sum;
          __nv_bfloat16 *dst = out + ((int64_t)(I.q0 + j) * p.Hq + I.g * p.G + hg) * D;
#pragma unroll 1
          for (int c = 0; c < D / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(tmem + Cfg::kColO + lane_addr + c * 32, r);
            wait_ld();
            if (valid_row) {
#pragma unroll
              for (int v = 0; v < 4; ++v) {
                uint4 o;
                o.x = pack_bf16(__uint_as_float(r[8 * v + 0]) * inv, __uint_as_float(r[8 * v + 1]) * inv);
                o.y = pack_bf16(__uint_as_float(r[8 * v + 2]) * inv, __uint_as_float(r[8 * v + 3]) * inv);
                o.z = pack_bf16(__uint_as_float(r[8 * v + 4]) * inv, __uint_as_float(r[8 * v + 5]) * inv);
                o.w = pack_bf16(__uint_as_float(r[8 * v + 6]) * inv, __uint_as_float(r[8 * v + 7]) * inv);
                *reinterpret_cast<uint4 *>(dst + c * 32 + v * 8) = o;
              }
            }
          }
          if (valid_row && p.lse) p.lse[(int64_t)(I.q0 + j) * p.Hq + I.g * p.G + hg] = (m_ref + log2f(l_sum)) * kLn2;
        } else {
          const int64_t slot = (int64_t)I.part_slot * p.rows_cap + row;
          float *dst = p.part_o + slot * D;
#pragma unroll 1
          for (int c = 0; c < D / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(tmem + Cfg::kColO + lane_addr + c * 32, r);
            wait_ld();
            if (valid_row) {
#pragma unroll
              for (int v = 0; v < 8; ++v)
                *reinterpret_cast<uint4 *>(dst + c * 32 + v * 4) = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
            }
          }
          if (valid_row) p.part_ml[slot] = make_float2(m_ref, l_sum);
        }
      }
      fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->o_free);
      idx = idx_next;
      I = Inext;
    }
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();
  if (bars->abort) {
    // give copies that are still in flight time to land before shared memory is released
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);
  }
  fence_before();
  __syncthreads();
  if (warp == 1) {
    fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(Cfg::kTmemCols) : "memory");
  }
}

}  // namespace spx
