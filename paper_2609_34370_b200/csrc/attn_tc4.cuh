// Verify attention for at most 64 packed query rows per kv-head: column-split softmax.
//
// With G*(k+1) <= 64 a 128-lane tensor-memory tile would leave half or three quarters of the lane
// quadrants (and with them the SM's sub-partitions, each with its own issue slot and exponential
// unit) idle.  This kernel splits every 128-token tile by columns instead (MROWS = 32: four
// blocks of 32 tokens; MROWS = 64: two blocks of 64 tokens for each of two row groups):
//   * S = Q K^T is a weight-stationary MMA with M = MROWS, whose accumulator layout spreads the
//     tokens of every query row over the lane quadrants;
//   * each softmax warp owns one (row group, token block).  The warps that share a row agree on the
//     row maximum of the tile through shared memory (one bounded barrier per tile), so that all of
//     them use the same reference maximum, and write P as bf16 into a swizzled shared-memory tile
//     (one tile: it is rewritten as soon as the previous value MMA has consumed it);
//   * O += P V is again a weight-stationary M = MROWS MMA (P from shared memory, V MN-major), so O
//     comes out column-split the same way: each thread holds D/4 (or D/2) columns of one row,
//     complete, and the epilogue is one tensor-memory load and one store per thread.
// Producer, stage ring, work plan, bounded waits and partial/direct output are those of
// attn_tc_kernel.
#pragma once
#include "attn_tc.cuh"

namespace spx {

template <int D, int MROWS>
struct Tc4Cfg {
  static_assert(MROWS == 32 || MROWS == 64, "MROWS is 32 or 64");
  static constexpr int kSplit = 128 / MROWS;               // token blocks per tile: 4 or 2
  static constexpr int kTokPerThread = kTileTokens / kSplit;  // 32 or 64 score columns per thread
  static constexpr int kHalves = D / 64;
  static constexpr int kHalfBytes = kTileTokens * 128;
  static constexpr int kTileBytes = kHalves * kHalfBytes;
  static constexpr int kQHalfBytes = MROWS * 128;
  static constexpr int kQBytes = kHalves * kQHalfBytes;
  static constexpr int kQBufs = MROWS == 32 ? 2 : 1;       // the 64-row tile leaves room for one Q buffer only
  static constexpr int kPHalfBytes = MROWS * 128;          // P tile: MROWS rows x 128 tokens bf16, two 64-token halves
  static constexpr int kPBytes = 2 * kPHalfBytes;
  static constexpr int kBarBytes = 2304;         // barriers (256) + row maxima (1024) + row sums (1024)
  static constexpr int kSlack = 512;             // room to round the dynamic shared base up to 1024 bytes
  // With 32 rows 8 KB are left unused on purpose: with them (and the 1 KB the hardware reserves
  // per block) the short sampling kernels, which need about 2 KB of shared memory, can share an SM
  // with this CTA.
  static constexpr int kFree = MROWS == 32 ? 8192 : 0;
  static constexpr int kBudget = 232448 - kFree - kSlack - kBarBytes - kQBufs * kQBytes - kPBytes;
  static constexpr int kStagesRaw = kBudget / (2 * kTileBytes);
  static constexpr int kStages = kStagesRaw > 4 ? 4 : kStagesRaw;
  static constexpr int kSmemBytes = kSlack + kQBufs * kQBytes + kStages * 2 * kTileBytes + kPBytes + kBarBytes;
  static constexpr int kColBlock = D / kSplit;   // output columns held by one thread
  static constexpr int kColS0 = 0, kColS1 = kTokPerThread, kColO = 2 * kTokPerThread;  // + two O buffers of kColBlock
  static constexpr int kTmemCols = (2 * kTokPerThread + 2 * kColBlock) <= 128 ? 128 : 256;
  static_assert(kStages >= 2, "need at least two stages");
};

namespace tc {
__device__ __forceinline__ void mma_ws_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.ws.cta_group::1.kind::f16 [%0], %1, %2, %3, p; }"
               ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
template <int N>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, uint32_t (&r)[N]) {
  if constexpr (N == 64) {
    tmem_ld32(taddr, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
    tmem_ld32(taddr + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[32]));
  } else if constexpr (N == 32) {
    tmem_ld32(taddr, r);
  } else {
    tmem_ld16(taddr, r);
  }
}
template <int N>
__device__ __forceinline__ void tmem_st(uint32_t taddr, const uint32_t (&r)[N]) {
  if constexpr (N == 64) {
    tmem_st32(taddr, *reinterpret_cast<const uint32_t(*)[32]>(&r[0]));
    tmem_st32(taddr + 32, *reinterpret_cast<const uint32_t(*)[32]>(&r[32]));
  } else if constexpr (N == 32) {
    tmem_st32(taddr, r);
  } else {
    tmem_st16(taddr, r);
  }
}
// weight-stationary instruction descriptor: D fp32, A/B bf16, A K-major, M = 32 or 64
__host__ __device__ constexpr uint32_t idesc_ws(uint32_t m, uint32_t n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) | ((n >> 3) << 17) | ((m >> 4) << 24);
}
}  // namespace tc

template <int D, int MROWS>
__global__ void __launch_bounds__(kTcThreads, 1)
attn_tc4_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap,
                const __grid_constant__ CUtensorMap qmap, AttnParams p) {
  SPX_TL_SCOPE(kTlAttention);
  // the combine kernel may take its places now (it reads the planner's list, then waits for this
  // kernel to end): its launch then costs nothing behind the last CTA
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  using Cfg = Tc4Cfg<D, MROWS>;
  using namespace tc;
  constexpr int kSplit = Cfg::kSplit, TPT = Cfg::kTokPerThread;
  extern __shared__ __align__(1024) unsigned char smem_dyn[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  if (smem - smem_dyn > Cfg::kSlack) {  // cannot happen with the declared alignment; never run past the allocation
    if (threadIdx.x == 0) atomicOr(p.dev_status, SPX_DEV_TIMEOUT);
    return;
  }
  unsigned char *sQ = smem;
  unsigned char *sK = smem + Cfg::kQBufs * Cfg::kQBytes;
  unsigned char *sV = sK + Cfg::kStages * Cfg::kTileBytes;
  unsigned char *sP = sV + Cfg::kStages * Cfg::kTileBytes;  // one P tile
  TcBarriers *bars = reinterpret_cast<TcBarriers *>(sP + Cfg::kPBytes);
  float *sMx = reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(bars) + 256);  // [2 tiles][kSplit][MROWS]
  float *sL = sMx + 2 * 128;                                                             // [2 items][kSplit][MROWS]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  long long prof_g0 = 0;
  if (kProfile) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(prof_g0));
  if (tid == 0) {
    for (int s = 0; s < 4; ++s) { mbar_init(&bars->k_full[s], 1); mbar_init(&bars->v_full[s], 1); mbar_init(&bars->k_empty[s], 1); mbar_init(&bars->v_empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&bars->s_full[b], 1); mbar_init(&bars->p_full[b], 4); mbar_init(&bars->q_full[b], 1); mbar_init(&bars->q_empty[b], 1); }
    mbar_init(&bars->pv_done[0], 1);
    mbar_init(&bars->pv_done[1], 1);
    mbar_init(&bars->o_free2[0], 4);
    mbar_init(&bars->o_free2[1], 4);
    mbar_init(&bars->e_bar, 4);
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
  // Everything above touched only this CTA's own resources; the plan is read from here on.  Under
  // programmatic dependent launch this is where the kernel waits for the planner to finish.
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // this CTA's range of the plan: entries cta_off[c] .. cta_off[c+1] of the work list, in order
  const bool planned = !p.hdr->overflow && (int)blockIdx.x < p.hdr->n_cta;
  const int item_begin = planned ? p.cta_off[blockIdx.x] : 0;
  const int item_end = planned ? p.cta_off[blockIdx.x + 1] : 0;
  auto item_index = [&](int it) -> int { return item_begin + it < item_end ? item_begin + it : -1; };
  // Work entries carry everything a role needs about the request (one 32-byte load).
  auto entry_of = [&](int idx) -> WorkEntry { return p.work[idx]; };
  auto make_item = [&](const WorkEntry &we, int idx) -> ItemInfo {
    ItemInfo I;
    I.req = we.req; I.g = we.g; I.tile_begin = we.tile_begin; I.tile_end = we.tile_end; I.part_slot = we.part_slot;
    I.q0 = we.q0; I.m = we.m; I.L = we.L;
    I.R = I.m * p.G;
    I.t_end = min(we.tile_end * kTileTokens, I.L);
    return I;
  };
  const int pages_per_tile = kTileTokens >> p.log2P;
  long long prof_acc[4] = {0, 0, 0, 0};
  long long prof_x[3] = {0, 0, 0};
  const long long prof_t0 = kProfile ? clock64() : 0;
  auto warp_wait = [&](uint64_t *bar, uint32_t parity, int slot = 3) -> bool {
    const long long t0 = kProfile ? clock64() : 0;
    const bool r = __all_sync(0xffffffffu, mbar_wait(bar, parity, bars, p.dev_status));
    if (kProfile) prof_acc[slot] += clock64() - t0;
    return r;
  };
  auto lane_wait = [&](uint64_t *bar, uint32_t parity, int slot) -> bool {
    const long long t0 = kProfile ? clock64() : 0;
    const bool r = mbar_wait(bar, parity, bars, p.dev_status);
    if (kProfile) prof_acc[slot] += clock64() - t0;
    return r;
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    // Tiles are walked in groups of 32/pages_per_tile tiles so that every lane owns one page of
    // the group: one coalesced block-table read per group, issued one group ahead of the copies
    // (and the next item's work entry one item ahead) so that no load latency sits between two
    // tiles.
    const int tiles_per_group = 32 / pages_per_tile;
    const int my_tile = lane / pages_per_tile, my_page = lane % pages_per_tile;
    struct GCursor { int it, idx, tile0; WorkEntry e, e_next; bool valid; };
    auto open = [&](GCursor &c, int it) {
      c.it = it;
      c.idx = item_index(it);
      c.valid = c.idx >= 0;
      if (c.valid) {
        c.tile0 = c.e.tile_begin;
        const int idx_next = item_index(it + 1);
        if (idx_next >= 0) c.e_next = entry_of(idx_next);  // in flight until the next item opens
      }
    };
    auto advance = [&](GCursor &c) {
      c.tile0 += tiles_per_group;
      if (c.tile0 >= c.e.tile_end) { c.e = c.e_next; open(c, c.it + 1); }
    };
    // page id of this lane's (tile, page) in the cursor's group; -1 if the lane has none
    auto load_page = [&](const GCursor &c) -> int {
      const int tile = c.tile0 + my_tile;
      if (!c.valid || tile >= c.e.tile_end) return -1;
      const int t_end = min(c.e.tile_end * kTileTokens, c.e.L);
      const int ntok = min(kTileTokens, t_end - tile * kTileTokens);
      if (my_page * p.P >= ntok) return -1;
      int page = p.block_table[(int64_t)c.e.req * p.max_pages_per_req + tile * pages_per_tile + my_page];
      if (page < 0 || page >= p.num_pages) {
        page = 0;  // keep the copy in bounds; the request is flagged and its rows are voided
        atomicOr(p.dev_status, SPX_DEV_BAD_PAGE);
        p.req_bad[c.e.req] = 1;
      }
      return page;
    };
    GCursor la;
    la.idx = item_index(0);
    if (la.idx >= 0) la.e = entry_of(la.idx);
    open(la, 0);
    int page_la = load_page(la);
    uint32_t tc_ = 0;
    bool ok = true;
    // bytes of one Q box pair: G * max_q_len packed rows of D columns (rows past the tensor read as zero)
    const uint32_t q_bytes = (uint32_t)(p.G * p.q_box_rows) * D * 2;
    while (la.valid && ok && !bars->abort) {
      const GCursor cur = la;
      const int page = page_la;
      advance(la);
      page_la = load_page(la);
      const int g = cur.e.g;
      if (cur.tile0 == cur.e.tile_begin) {
        // a new work entry: its packed query rows go into the Q buffer of its parity, as soon as the
        // last score MMA of the entry that used the buffer before has read it.  The copy is issued
        // ahead of the entry's first K tile, so it has the tiles still in the ring to arrive.
        const uint32_t qc = (uint32_t)cur.it;
        const uint32_t qb = Cfg::kQBufs == 2 ? (qc & 1) : 0;
        const uint32_t uses = Cfg::kQBufs == 2 ? (qc >> 1) : qc;   // earlier uses of this buffer
        if (uses >= 1) {
          ok = warp_wait(&bars->q_empty[qb], (uses - 1) & 1, 2);
          if (!ok) break;
        }
        if (lane == 0) {
          mbar_expect_tx(&bars->q_full[qb], q_bytes);
#pragma unroll
          for (int h = 0; h < Cfg::kHalves; ++h)
            tma_load_3d(smem_u32(sQ + qb * Cfg::kQBytes + h * Cfg::kQHalfBytes), &qmap, &bars->q_full[qb], h * 64, g * p.G, cur.e.q0);
        }
      }
      const int t_end = min(cur.e.tile_end * kTileTokens, cur.e.L);
      for (int ti = 0; ti < tiles_per_group && cur.tile0 + ti < cur.e.tile_end; ++ti, ++tc_) {
        const int tile = cur.tile0 + ti;
        const int slot = tc_ % Cfg::kStages;
        const uint32_t ph = (tc_ / Cfg::kStages) & 1;
        const int ntok = min(kTileTokens, t_end - tile * kTileTokens);
        const int npages = (ntok + p.P - 1) >> p.log2P;
        const uint32_t bytes = (uint32_t)npages * p.P * D * 2;
        const bool mine = (my_tile == ti) && page >= 0;
        ok = warp_wait(&bars->k_empty[slot], ph ^ 1, 0);
        if (!ok) break;
        if (lane == 0) mbar_expect_tx(&bars->k_full[slot], bytes);
        if (mine) {
#pragma unroll
          for (int h = 0; h < Cfg::kHalves; ++h)
            tma_load_4d(smem_u32(sK + slot * Cfg::kTileBytes + h * Cfg::kHalfBytes + my_page * p.P * 128), &kmap,
                        &bars->k_full[slot], h * 64, p.head_inner ? g : 0, p.head_inner ? 0 : g, page);
        }
        ok = warp_wait(&bars->v_empty[slot], ph ^ 1, 1);
        if (!ok) break;
        if (lane == 0) mbar_expect_tx(&bars->v_full[slot], bytes);
        if (mine) {
#pragma unroll
          for (int h = 0; h < Cfg::kHalves; ++h)
            tma_load_4d(smem_u32(sV + slot * Cfg::kTileBytes + h * Cfg::kHalfBytes + my_page * p.P * 128), &vmap,
                        &bars->v_full[slot], h * 64, p.head_inner ? g : 0, p.head_inner ? 0 : g, page);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t kIdescQK = idesc_ws(MROWS, kTileTokens, false);
      constexpr uint32_t kIdescPV = idesc_ws(MROWS, D, true);
      // Two cursors over the CTA's flat tile sequence: the score MMA runs one tile ahead of the
      // value MMA, across work-item boundaries too.
      struct Cursor { int it, n_tiles, n_tiles_next, i; uint32_t qc, t; bool valid; };
      auto tiles_of = [&](int it) -> int {
        const int idx = item_index(it);
        if (idx < 0) return 0;
        const WorkEntry *we = p.work + idx;
        return we->tile_end - we->tile_begin;
      };
      // the tile count of the following item is loaded when an item opens, long before it is needed
      auto open_item = [&](Cursor &c) {
        c.valid = item_index(c.it) >= 0;
        c.i = 0;
        c.n_tiles_next = tiles_of(c.it + 1);
      };
      auto advance = [&](Cursor &c) {
        ++c.t;
        if (++c.i >= c.n_tiles) { ++c.it; ++c.qc; c.n_tiles = c.n_tiles_next; open_item(c); }
      };
      Cursor qk{0, 0, 0, 0, 0, 0, false}, pv{0, 0, 0, 0, 0, 0, false};
      qk.n_tiles = pv.n_tiles = tiles_of(0);
      open_item(qk);
      open_item(pv);
      bool ok = true;
      auto issue_qk = [&]() -> bool {
        const uint32_t t = qk.t, qb = Cfg::kQBufs == 2 ? (qk.qc & 1) : 0;
        if (qk.i == 0 && !lane_wait(&bars->q_full[qb], (Cfg::kQBufs == 2 ? (qk.qc >> 1) : qk.qc) & 1, 3)) return false;
        const int slot = t % Cfg::kStages;
        if (!lane_wait(&bars->k_full[slot], (t / Cfg::kStages) & 1, 0)) return false;
        fence_after();
        const uint32_t qa = smem_u32(sQ + qb * Cfg::kQBytes), ka = smem_u32(sK + slot * Cfg::kTileBytes);
        const uint32_t ts = tmem + ((t & 1) ? Cfg::kColS1 : Cfg::kColS0);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t qoff = (k / 4) * Cfg::kQHalfBytes + (k % 4) * 32;
          const uint32_t koff = (k / 4) * Cfg::kHalfBytes + (k % 4) * 32;
          mma_ws_ss(ts, smem_desc(qa + qoff, 16, 1024), smem_desc(ka + koff, 16, 1024), kIdescQK, k > 0);
        }
        mma_commit(&bars->s_full[t & 1]);
        mma_commit(&bars->k_empty[slot]);
        if (qk.i + 1 >= qk.n_tiles) mma_commit(&bars->q_empty[qb]);  // last score MMA of the item
        advance(qk);
        return true;
      };
      if (qk.valid) ok = issue_qk();
      while (ok && pv.valid && !bars->abort) {
        if (qk.valid) ok = issue_qk();
        if (!ok) break;
        const uint32_t t = pv.t;
        ok = lane_wait(&bars->p_full[t & 1], (t >> 1) & 1, 1);
        // the O buffer of this item's parity was last used two items ago
        if (ok && pv.i == 0 && pv.qc >= 2) ok = lane_wait(&bars->o_free2[pv.qc & 1], ((pv.qc >> 1) - 1) & 1, 3);
        const int slot = t % Cfg::kStages;
        if (ok) ok = lane_wait(&bars->v_full[slot], (t / Cfg::kStages) & 1, 2);
        if (!ok) break;
        fence_after();
        const uint32_t va = smem_u32(sV + slot * Cfg::kTileBytes);
        const uint32_t pa = smem_u32(sP);
#pragma unroll
        for (int k = 0; k < kTileTokens / 16; ++k)
          mma_ws_ss(tmem + Cfg::kColO + (pv.qc & 1) * Cfg::kColBlock, smem_desc(pa + (k / 4) * Cfg::kPHalfBytes + (k % 4) * 32, 16, 1024),
                    smem_desc(va + k * 2 * 1024, Cfg::kHalfBytes, 1024), kIdescPV, (pv.i > 0) || (k > 0));
        mma_commit(&bars->v_empty[slot]);
        mma_commit(&bars->pv_done[t & 1]);
        advance(pv);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax / epilogue
    const int quad = warp & 3;
    // the accumulator layouts of the M = 32 / M = 64 weight-stationary MMAs: quadrant -> (row group,
    // token block); the same split applies to the columns of O
    const int rgrp = kSplit == 4 ? 0 : (quad & 1);
    const int tblk = kSplit == 4 ? quad : (quad >> 1);
    const int row = rgrp * 32 + lane;                       // packed query row
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const int sm_tid = tid - 64;
    __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(p.out);
    constexpr int CB = Cfg::kColBlock;

    uint32_t tc_ = 0, qc = 0, ec = 0;
    bool ok = true;
    // bounded barrier among the four softmax warps (a named barrier could not time out)
    auto softmax_sync = [&]() -> bool {
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->e_bar);
      const bool r = warp_wait(&bars->e_bar, ec & 1, 2);
      ++ec;
      return r;
    };
    // Row sums of the four quadrants are merged through sL (written at the end of the item's last
    // tile, visible after the next bounded barrier); each thread then finishes its D/4 columns.
    struct Pending { bool valid; ItemInfo I; float m_ref; uint32_t last_tc, qc; } pend;
    pend.valid = false;
    auto run_epilogue = [&]() -> bool {
      const long long pe0 = kProfile ? clock64() : 0;
      const ItemInfo &J = pend.I;
      const float *sl = sL + (pend.qc & 1) * 128;
      float l_row = 0.f;
#pragma unroll
      for (int tb = 0; tb < kSplit; ++tb) l_row += sl[tb * MROWS + row];
      if (!warp_wait(&bars->pv_done[pend.last_tc & 1], (pend.last_tc >> 1) & 1, 1)) return false;
      fence_after();
      uint32_t o[CB];
      tmem_ld<CB>(tmem + Cfg::kColO + (pend.qc & 1) * CB + lane_addr, o);
      wait_ld();
      // O has been read: the item after next may overwrite this buffer
      fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->o_free2[pend.qc & 1]);
      const int j = row / p.G, hg = row % p.G;
      if (row < J.R) {
        if (J.part_slot < 0) {
          const float inv = 1.f / l_row;
          __nv_bfloat16 *dst = out + ((int64_t)(J.q0 + j) * p.Hq + J.g * p.G + hg) * D + tblk * CB;
#pragma unroll
          for (int v = 0; v < CB / 8; ++v) {
            uint4 u;
            u.x = pack_bf16(__uint_as_float(o[8 * v + 0]) * inv, __uint_as_float(o[8 * v + 1]) * inv);
            u.y = pack_bf16(__uint_as_float(o[8 * v + 2]) * inv, __uint_as_float(o[8 * v + 3]) * inv);
            u.z = pack_bf16(__uint_as_float(o[8 * v + 4]) * inv, __uint_as_float(o[8 * v + 5]) * inv);
            u.w = pack_bf16(__uint_as_float(o[8 * v + 6]) * inv, __uint_as_float(o[8 * v + 7]) * inv);
            *reinterpret_cast<uint4 *>(dst + v * 8) = u;
          }
          if (tblk == 0 && p.lse) p.lse[(int64_t)(J.q0 + j) * p.Hq + J.g * p.G + hg] = (pend.m_ref + log2f(l_row)) * kLn2;
        } else {
          const int64_t slot = (int64_t)J.part_slot * p.rows_cap + row;
          float *dst = p.part_o + slot * D + tblk * CB;
#pragma unroll
          for (int v = 0; v < CB / 4; ++v)
            *reinterpret_cast<uint4 *>(dst + v * 4) = make_uint4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
          if (tblk == 0) p.part_ml[slot] = make_float2(pend.m_ref, l_row);
        }
      }
      pend.valid = false;
      if (kProfile) prof_acc[3] += clock64() - pe0;
      return true;
    };
    ItemInfo I, Inext;
    int idx = item_index(0);
    if (idx >= 0) I = make_item(entry_of(idx), idx);
    for (int it = 0; idx >= 0 && ok; ++it, ++qc) {
      if (bars->abort) break;
      // the next item's work entry is requested now and unpacked at the end of this item (the query
      // rows themselves are fetched by the producer warp)
      const int idx_next = item_index(it + 1);
      WorkEntry e_next;
      if (idx_next >= 0) e_next = entry_of(idx_next);
      const bool valid_row = row < I.R;
      float m_ref = -INFINITY, l_sum = 0.f;     // m_ref is the same in all four quadrants of a row
      const int limit = I.L - I.m + row / p.G;  // last visible token of this row
      for (int tile = I.tile_begin; tile < I.tile_end && ok; ++tile, ++tc_) {
        const uint32_t b = tc_ & 1;
        const uint32_t ts = tmem + (b ? Cfg::kColS1 : Cfg::kColS0) + lane_addr;
        const int t0 = tile * kTileTokens + tblk * TPT;  // first token of this thread's block
        const bool mask_tile = tile * kTileTokens + kTileTokens - 1 > I.L - I.m;
        ok = warp_wait(&bars->s_full[b], (tc_ >> 1) & 1, 0);
        if (!ok) break;
        fence_after();
        uint32_t r[TPT];
        tmem_ld<TPT>(ts, r);
        wait_ld();
        float mx = -INFINITY;
        if (mask_tile) {
#pragma unroll
          for (int i = 0; i < TPT; ++i) {
            r[i] = (t0 + i <= limit) ? r[i] : 0xff800000u;  // -inf
            mx = fmaxf(mx, __uint_as_float(r[i]));
          }
        } else {
#pragma unroll
          for (int i = 0; i < TPT; ++i) mx = fmaxf(mx, __uint_as_float(r[i]));
        }
        // agree on the row maximum of the whole tile
        sMx[(b * kSplit + tblk) * MROWS + row] = mx * p.scale_log2;
        ok = softmax_sync();
        if (!ok) break;
        float mrow = -INFINITY;
#pragma unroll
        for (int tb = 0; tb < kSplit; ++tb) mrow = fmaxf(mrow, sMx[(b * kSplit + tb) * MROWS + row]);
        // lazy rescale: the reference moves only when the maximum grows by more than 2^8; a row
        // that has seen no visible token yet adopts the tile maximum for free (its O is zero)
        float alpha = 1.f;
        bool need_scale = false;
        if (valid_row) {
          if (m_ref == -INFINITY) {
            m_ref = mrow;
          } else if (mrow > m_ref + kRescaleThreshold) {
            alpha = fast_exp2(m_ref - mrow);
            m_ref = mrow;
            l_sum *= alpha;
            need_scale = true;
          }
        }
        if (__any_sync(0xffffffffu, need_scale)) {
          // this quadrant's block of O columns holds earlier tiles: wait for the last PV, scale
          ok = warp_wait(&bars->pv_done[(tc_ - 1) & 1], ((tc_ - 1) >> 1) & 1, 3);
          if (!ok) break;
          fence_after();
          uint32_t o[CB];
          tmem_ld<CB>(tmem + Cfg::kColO + (qc & 1) * CB + lane_addr, o);
          wait_ld();
#pragma unroll
          for (int i = 0; i < CB; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
          tmem_st<CB>(tmem + Cfg::kColO + (qc & 1) * CB + lane_addr, o);
          wait_st();
        }
        const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
        float sum = 0.f;
        uint32_t pk[TPT / 2];
#pragma unroll
        for (int i = 0; i < TPT / 2; ++i) {
          const float p0 = fast_exp2(fmaf(__uint_as_float(r[2 * i]), p.scale_log2, -m_use));
          const float p1 = fast_exp2(fmaf(__uint_as_float(r[2 * i + 1]), p.scale_log2, -m_use));
          sum += p0 + p1;
          pk[i] = pack_bf16(p0, p1);
        }
        l_sum += sum;
        // the single P tile is free once the previous tile's value MMA has read it
        if (tc_ > 0) {
          ok = warp_wait(&bars->pv_done[(tc_ - 1) & 1], ((tc_ - 1) >> 1) & 1, 3);
          if (!ok) break;
        }
        {
          // P tile in shared memory: K-major, 128-byte swizzle, tokens [64h, 64h+64) in half h
          constexpr int kChunks = TPT / 8;                       // 16-byte chunks this thread writes
          const int tok0 = tblk * TPT;
          unsigned char *pr = sP + (tok0 >> 6) * Cfg::kPHalfBytes + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll
          for (int jj = 0; jj < kChunks; ++jj) {
            const int c = ((tok0 & 63) >> 3) + jj;
            *reinterpret_cast<uint4 *>(pr + ((c ^ (row & 7)) << 4)) = make_uint4(pk[4 * jj], pk[4 * jj + 1], pk[4 * jj + 2], pk[4 * jj + 3]);
          }
        }
        // rows of V past the end of the request must be zero (see attn_tc_kernel)
        const int ntok = min(kTileTokens, I.t_end - tile * kTileTokens);
        if (ntok < kTileTokens) {
          const int slot = tc_ % Cfg::kStages;
          ok = warp_wait(&bars->v_full[slot], (tc_ / Cfg::kStages) & 1, 3);
          if (!ok) break;
          unsigned char *vt = sV + slot * Cfg::kTileBytes;
          const int per_half = (kTileTokens - ntok) * 8;
          for (int i = sm_tid; i < per_half * Cfg::kHalves; i += 128) {
            const int h = i / per_half, rem = i % per_half;
            const int tok = ntok + rem / 8;
            *reinterpret_cast<uint4 *>(vt + (tok >> 3) * 1024 + h * Cfg::kHalfBytes + (tok & 7) * 128 + (rem % 8) * 16) = make_uint4(0, 0, 0, 0);
          }
        }
        fence_async_smem();
        fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->p_full[b]);
        if (pend.valid) ok = run_epilogue();  // previous item (its sL became visible at this tile's barrier)
      }
      if (!ok) break;
      if (idx_next >= 0) Inext = make_item(e_next, idx_next);

      // ---- the item's epilogue is deferred: it runs after the first tile of the next item, when
      // the last PV has long completed, so the softmax never idles at an item boundary
      sL[((qc & 1) * kSplit + tblk) * MROWS + row] = l_sum;
      pend.valid = true; pend.I = I; pend.m_ref = m_ref; pend.last_tc = tc_ - 1; pend.qc = qc;
      idx = idx_next;
      I = Inext;
    }
    if (ok && pend.valid && !bars->abort) {
      ok = softmax_sync();  // make the last item's row sums visible
      if (ok) ok = run_epilogue();
    }
  }
  if (kProfile && p.prof && lane == 0 && (warp == 0 || warp == 1 || warp == 4)) {
    // slots: [0] CTA cycles, then 4 per role (producer: k_empty, v_empty; MMA: k_full, p_full,
    // v_full, other; softmax quadrant 0: s_full, pv_done at item end, merge syncs, whole epilogue)
    long long *dst = p.prof + (long long)blockIdx.x * kProfSlots;
    const int base = warp == 0 ? 1 : (warp == 1 ? 5 : 9);
    for (int i = 0; i < 4; ++i) dst[base + i] = prof_acc[i];
    if (warp == 4) {
      dst[0] = clock64() - prof_t0;
      long long g1;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g1));
      dst[1 + 2] = prof_x[0]; dst[1 + 3] = prof_x[1]; dst[15] = prof_x[2];
      dst[13] = prof_g0;  // kernel entry of this CTA (ns)
      dst[14] = g1;       // end of this CTA's work loop (ns)
    }
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();
  if (bars->abort) {
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
