// LM head on the 5th-generation tensor cores: logits[M, V] = H[M, K] W[V, K]^T in bf16 with fp32
// accumulation, with the sampling half's row statistics produced in the epilogue.
//
// The product is computed transposed, vocabulary along the MMA's M dimension, so that a pair of
// CTAs on two SMs (a cluster of two) can share tcgen05.mma.cta_group::2 instructions of M = 256:
// every output tile is 256 vocabulary rows (128 per CTA, one TMEM lane each) by up to 512 tokens
// (TMEM columns), covered by one or two MMAs of N = NT <= 256 per k-step of 16 that share the A
// operand.  Per k-step of 64 a CTA stages only its own 128 rows of W (16 KB) and its own half of
// the tile's rows of H with ordinary TMA loads: 40 KB for all 384 rows of the Llama-3-8B shape,
// where three single-CTA tiles of M = 128, N = 256 staged 144 KB for the same products, and the
// tensor core reads less shared memory per MMA (the single-CTA form ran at 171 cycles per MMA of
// K = 16 where 128 would be its rate).  What bounds the kernel is how many bytes a CTA can keep in
// flight against the 2 us its loads take under load, so bytes per product are what counts.
//
// Each CTA, warp-specialised (320 threads):
//   warp 0      producer (one lane): the TMA boxes of every k-step into a ring of shared-memory
//               stages.  The loads of both CTAs complete on the LEADER's barrier of the stage
//               (the .cta_group::2 form of the copy lets the barrier live in the peer CTA);
//   warp 1      leader CTA only: MMA issuer (one lane) into the TMEM accumulator (two of them,
//               alternating, when a tile has at most 256 tokens);
//   warps 2-9   epilogue, two warps per TMEM lane quadrant taking alternate chunks of 32 tokens.
//               A warp first reads its chunks out of the accumulator (one vocabulary row per
//               lane), rounds them to bf16 pairs that stay in registers and hands the accumulator
//               back: a tile of more than 256 tokens has no second accumulator, and the next
//               tile's MMAs wait for exactly this.  Then, beside those MMAs, a partial transpose
//               across the warp hands every lane eight consecutive columns of four tokens, which
//               it stores as 16-byte vectors (64 contiguous bytes per token and warp) and
//               reduces - as stored - to (max, sum 2^((x - max) log2 e)); the four quadrants'
//               pairs of a token are merged through shared memory.
// The MMA's completions are committed twice, once to the leader's barrier and once to the peer's
// (a commit takes a shared::cluster address); the epilogue's "accumulator drained" signals of the
// peer are plain remote mbarrier arrivals on the leader's barrier.  No copy and no commit is sent
// to more than one CTA at a time.
// Tiles are numbered vocabulary-major and dealt round-robin to the pairs, so the pairs that need
// the same block of W run side by side and it crosses HBM once; H is small and lives in L2.
//
// Every wait on an mbarrier is bounded: on expiry the CTA raises SPX_DEV_TIMEOUT, its roles leave
// their loops (the peer's waits then run out too), pending copies get time to land, both CTAs meet
// at the cluster barrier - which every thread reaches, whatever happened - and TMEM is released.
#pragma once
#include <cuda.h>

#include "attn_tc.cuh"
#include "common.cuh"

namespace spx {

constexpr int kLmVB = 128;           // vocabulary rows per CTA (TMEM lanes); a pair covers 256
constexpr int kLmStatCols = kLmVB;   // vocabulary columns one statistics pair covers
constexpr int kLmBK = 64;
constexpr int kLmMaxStages = 8;
constexpr int kLmMaxNT = 256;                          // tokens per MMA, at most
constexpr int kLmMaxTileTok = 512;                     // tokens per tile, at most (TMEM columns)
constexpr int kLmABytes = kLmVB * kLmBK * 2;           // 16 KB: this CTA's rows of W
constexpr int kLmEpiWarps = 8;        // two per TMEM lane quadrant, taking alternate chunks of 32 tokens
constexpr int kLmThreads = (2 + kLmEpiWarps) * 32;
constexpr int kLmRedFloats = (kLmMaxTileTok / 32) * 4 * 32;            // [chunk][warp][token], two floats each
constexpr int kLmBarBytes = 512;
constexpr int kLmSmemBytes = 232448;                                   // all of it: the ring takes what the rest leaves
constexpr int kLmRingBytes = kLmSmemBytes - 1024 - 2 * kLmRedFloats * 4 - kLmBarBytes;

struct LmBarriers {
  uint64_t full[kLmMaxStages];    // leader: the stage has landed in both CTAs (TMA bytes of both)
  uint64_t empty[kLmMaxStages];   // the pair MMAs that read the stage are done (committed to both CTAs' barriers)
  uint64_t acc_full[2];           // accumulator complete (committed to both CTAs' barriers)
  uint64_t acc_empty[2];          // leader only: all epilogue warps of the pair have drained the accumulator
  uint64_t e_bar;                 // the epilogue warps of this CTA
  uint32_t tmem_base;
  volatile int32_t abort;
};
static_assert(sizeof(LmBarriers) <= kLmBarBytes, "barrier block");

struct LmParams {
  int32_t M, K, V;
  int32_t tok_tiles, tile_tok;    // token tiles and tokens per tile (n_sub * NT)
  int32_t n_sub, NT;              // MMAs per k-step of 16 and their N (a multiple of 32, at most 256)
  int32_t n_buf;                  // TMEM accumulators in rotation: 2 if tile_tok <= 256, else 1
  int32_t n_stages, stage_bytes;  // the ring
  int32_t v_tiles, k_blocks;      // vocabulary tiles of 256 rows, k-steps of 64
  int32_t stat_tiles;             // ceil(V / kLmStatCols)
  __nv_bfloat16 *logits;
  int64_t row_stride;
  float2 *tile_stats;  // [M][stat_tiles]: (max * log2 e, sum 2^((x - max) log2 e)) of the block's columns; may be NULL
  int32_t *dev_status;
};

__device__ __forceinline__ bool lm_wait(uint64_t *b, uint32_t parity, LmBarriers *bars, int32_t *dev_status) {
  if (tc::mbar_try_wait(b, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (tc::mbar_try_wait(b, parity)) return true;
    if (bars->abort) return false;
    if (clock64() - t0 > kWaitLimitCycles) {  // about a second
      bars->abort = 1;
      atomicOr(dev_status, SPX_DEV_TIMEOUT);
      return false;
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(dst), "l"(map), "r"(tc::smem_u32(bar)), "r"(c0), "r"(c1) : "memory");
}

namespace lm {
// the same copy with its completion counted on a barrier of either CTA of the pair (`bar_cluster`
// is a shared::cluster address, see cluster_addr)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar_cluster, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1) : "memory");
}
// shared::cluster address of a shared-memory object of CTA `rank` of the cluster
__device__ __forceinline__ uint32_t cluster_addr(const void *p, uint32_t rank) {
  uint32_t ra;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(tc::smem_u32(p)), "r"(rank));
  return ra;
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// arrive on the barrier at the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ void remote_arrive(uint64_t *bar, uint32_t rank) {
  asm volatile(
      "{ .reg .b32 ra; mapa.shared::cluster.u32 ra, %0, %1; mbarrier.arrive.release.cluster.shared::cluster.b64 _, [ra]; }"
      ::"r"(tc::smem_u32(bar)), "r"(rank) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mma_pair_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p; }"
               ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// The four MMAs (K = 16 each) of one 64-wide k-step on one accumulator.  The operands' descriptors
// advance by 32 bytes per MMA inside the 128-byte swizzled rows: +2 in the descriptor's address
// field.  One block of straight-line code: the issuing thread runs alone in its warp, every
// instruction it spends between two MMAs is dead time of the tensor pipe once the queue runs dry.
__device__ __forceinline__ void mma_pair_ss_x4(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc_first) {
  asm volatile(
      "{ .reg .pred p, t; .reg .b64 a1, a2, a3, b1, b2, b3;\n\t"
      "setp.ne.b32 p, %4, 0; setp.eq.b32 t, 0, 0;\n\t"
      "add.u64 a1, %1, 2; add.u64 a2, %1, 4; add.u64 a3, %1, 6;\n\t"
      "add.u64 b1, %2, 2; add.u64 b2, %2, 4; add.u64 b3, %2, 6;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], a1, b1, %3, t;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], a2, b2, %3, t;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], a3, b3, %3, t; }"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc_first) : "memory");
}
// arrives on a barrier (shared::cluster address: of this CTA or of its peer) once every pair MMA
// issued so far has completed in both CTAs
__device__ __forceinline__ void mma_pair_commit(uint32_t bar_cluster) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_cluster) : "memory");
}
// instruction descriptor: D fp32, A/B bf16, both K-major, M = 256 over the pair, N = n
__host__ __device__ constexpr uint32_t idesc_pair(uint32_t n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((256u >> 4) << 24);
}
// Partial transpose across the warp of a chunk held as bf16 pairs.  Before, lane l (a row of the
// accumulator) holds u[i] = (columns 2 i, 2 i + 1 of row l); the column's bit 0 sits in the half,
// its bits 1-4 in the register index, the row's bits 0-4 in the lane index.  Three exchanges swap
// the column's bits 0-2 with the row's bits 0-2: halves against lane bit 0 (16 shuffles and byte
// permutes), register bits 0 and 1 against lane bits 1 and 2 (8 shuffles each).  After, lane
// (a, b) = 8 a + b holds u[4 g + i] = (rows 8 a + 2 i, 8 a + 2 i + 1 of column 8 g + b): eight
// consecutive rows of one column per group of four registers.
__device__ __forceinline__ void warp_transpose_pairs(uint32_t (&u)[16], int lane) {
  const bool odd = (lane & 1) != 0;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const uint32_t o = __shfl_xor_sync(0xffffffffu, u[i], 1);
    u[i] = odd ? __byte_perm(o, u[i], 0x7632) : __byte_perm(u[i], o, 0x5410);
  }
#pragma unroll
  for (int o = 1; o <= 2; o <<= 1) {
    const bool upper = (lane & (2 * o)) != 0;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      if ((j & o) == 0) {
        const uint32_t send = upper ? u[j] : u[j + o];
        const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, 2 * o);
        if (upper) u[j] = recv; else u[j + o] = recv;
      }
    }
  }
}
}  // namespace lm

// kCh: chunks of 32 tokens an epilogue warp holds at most (tile_tok <= 64 kCh); the rounded
// accumulator stays in 16 kCh registers per thread while it is stored.
template <int kCh>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kLmThreads, 1)
lm_head_kernel(const __grid_constant__ CUtensorMap hmap, const __grid_constant__ CUtensorMap wmap, LmParams p) {
  using namespace tc;
  extern __shared__ __align__(1024) unsigned char lm_smem[];
  unsigned char *stages = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(lm_smem) + 1023) & ~uintptr_t(1023));
  float2 *s_ms = reinterpret_cast<float2 *>(stages + kLmRingBytes);  // [chunks][4][32] (max * log2 e, sum) per warp
  LmBarriers *bars = reinterpret_cast<LmBarriers *>(s_ms + kLmRedFloats);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = lm::cluster_rank();  // 0: leader (issues the pair MMAs)
  const bool leader = rank == 0;
  const int S = p.n_stages;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kLmMaxStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&bars->acc_full[b], 1); mbar_init(&bars->acc_empty[b], 2 * kLmEpiWarps); }
    mbar_init(&bars->e_bar, kLmEpiWarps);
    bars->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    // the same warp of both CTAs allocates the pair's tensor memory: the same columns in each
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "n"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  lm::cluster_sync_all();  // the peer's barriers exist before anything arrives on them
  fence_after();
  const uint32_t tmem = bars->tmem_base;
  const int n_tiles_total = p.v_tiles * p.tok_tiles;
  const int n_pairs = gridDim.x >> 1, pair = blockIdx.x >> 1;
  const int half_nt = p.NT >> 1;                                  // rows of H per MMA this CTA stages per k-step
  const uint32_t sub_bytes = (uint32_t)half_nt * kLmBK * 2;
  const uint32_t stage_tx = kLmABytes + (uint32_t)p.n_sub * sub_bytes;   // bytes one CTA lands per stage
  const uint32_t nb = (uint32_t)p.n_buf;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer (both CTAs)
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int t = pair; t < n_tiles_total && ok; t += n_pairs) {
        const int vt = t / p.tok_tiles, tt = t % p.tok_tiles;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int s = it % S;
          if (it >= (uint32_t)S) ok = lm_wait(&bars->empty[s], ((it / S) - 1) & 1, bars, p.dev_status);
          if (!ok || bars->abort) { ok = false; break; }
          unsigned char *st = stages + (size_t)s * p.stage_bytes;
          // both CTAs' bytes are counted on the leader's barrier, which the MMA issuer waits on
#ifdef LM_DBG_NOLOAD
          if (it >= (uint32_t)S) { if (leader) mbar_arrive(&bars->full[s]); continue; }
#endif
          if (leader) mbar_expect_tx(&bars->full[s], 2 * stage_tx);
          const uint32_t bar = lm::cluster_addr(&bars->full[s], 0);
          lm::tma_load_2d_pair(smem_u32(st), &wmap, bar, kb * kLmBK, vt * 2 * kLmVB + (int)rank * kLmVB);
          for (int u = 0; u < p.n_sub; ++u)
            lm::tma_load_2d_pair(smem_u32(st + kLmABytes + u * sub_bytes), &hmap, bar, kb * kLmBK,
                                 tt * p.tile_tok + u * p.NT + (int)rank * half_nt);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && leader) {
      // ---------------------------------------------------------------- MMA issuer (leader CTA)
      static_assert(kLmBK == 64, "four MMAs of K = 16 per stage and accumulator");
      const uint32_t kIdesc = lm::idesc_pair((uint32_t)p.NT);
      // descriptors of stage 0; a stage, a sub-tile of H or a k-step only moves the address field
      const uint64_t a_desc0 = smem_desc(smem_u32(stages), 16, 1024);
      const uint64_t w_desc0 = smem_desc(smem_u32(stages) + kLmABytes, 16, 1024);
      const uint64_t stage_step = (uint64_t)(p.stage_bytes >> 4), sub_step = (uint64_t)(sub_bytes >> 4);
      const uint32_t empty_mine = lm::cluster_addr(&bars->empty[0], 0), empty_peer = lm::cluster_addr(&bars->empty[0], 1);
      const uint32_t accf_mine = lm::cluster_addr(&bars->acc_full[0], 0), accf_peer = lm::cluster_addr(&bars->acc_full[0], 1);
      const bool two = p.n_sub == 2;
      uint32_t it = 0, j = 0;
      int s = 0;
      uint32_t ph = 0;  // parity of the ring's current round
      bool ok = true;
      for (int t = pair; t < n_tiles_total && ok; t += n_pairs, ++j) {
        const uint32_t b = j % nb;
        if (j >= nb) ok = lm_wait(&bars->acc_empty[b], ((j / nb) - 1) & 1, bars, p.dev_status);
        if (!ok) break;
        fence_after();
        const uint32_t d0 = tmem + b * kLmMaxNT, d1 = d0 + p.NT;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          ok = lm_wait(&bars->full[s], ph, bars, p.dev_status);
          if (!ok) break;
          fence_after();
          const uint64_t ad = a_desc0 + (uint64_t)s * stage_step, wd = w_desc0 + (uint64_t)s * stage_step;
          lm::mma_pair_ss_x4(d0, ad, wd, kIdesc, kb > 0);
          if (two) lm::mma_pair_ss_x4(d1, ad, wd + sub_step, kIdesc, kb > 0);
          // one arrival per CTA: each producer waits on its own barrier of the stage
          lm::mma_pair_commit(empty_mine + 8 * s);
          lm::mma_pair_commit(empty_peer + 8 * s);
          if (++s == S) { s = 0; ph ^= 1; }
        }
        if (ok) {
          lm::mma_pair_commit(accf_mine + 8 * b);
          lm::mma_pair_commit(accf_peer + 8 * b);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (both CTAs)
    const int q = warp & 3;  // TMEM lane quadrant this warp may read
    const int epi = warp - 2, c_first = epi >> 2;  // the quadrant's two warps take the even and the odd chunks
    const int n_chunks = p.tile_tok >> 5;
    uint32_t j = 0, ec = 0;
    bool ok = true;
    // bounded barrier among the epilogue warps
    auto epi_sync = [&]() -> bool {
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->e_bar);
      const bool r = __all_sync(0xffffffffu, lm_wait(&bars->e_bar, ec & 1, bars, p.dev_status));
      ++ec;
      return r;
    };
    for (int t = pair; t < n_tiles_total && ok; t += n_pairs, ++j) {
      const int vt = t / p.tok_tiles, tt = t % p.tok_tiles;
      const uint32_t b = j % nb;
      ok = __all_sync(0xffffffffu, lm_wait(&bars->acc_full[b], (j / nb) & 1, bars, p.dev_status));
      if (!ok) break;
      fence_after();
      const int tok0 = tt * p.tile_tok;
      const uint32_t taddr = tmem + b * kLmMaxNT + ((uint32_t)(q * 32) << 16);
      const int vrow0 = vt * 2 * kLmVB + (int)rank * kLmVB + q * 32;  // first vocabulary index of this warp
      const int v_left = p.V - vrow0;                                  // valid columns among the warp's 32 (may be <= 0)
      // The accumulator is drained first: per chunk of 32 tokens it comes out one vocabulary row
      // per lane and is rounded to bf16 pairs that stay in registers, so that the MMAs of the next
      // tile start while this one is still being transposed, stored and reduced.
      uint32_t u[kCh][16];
#pragma unroll
      for (int ci = 0; ci < kCh; ++ci) {
        const int c = c_first + ci * (kLmEpiWarps / 4);
        if (c < n_chunks) {
          uint32_t r[32];
          tmem_ld32(taddr + c * 32, r);
          wait_ld();
#pragma unroll
          for (int i = 0; i < 16; ++i) u[ci][i] = pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
        }
      }
      fence_before();
      __syncwarp();
      if (lane == 0) {
        if (leader) mbar_arrive(&bars->acc_empty[b]);
        else lm::remote_arrive(&bars->acc_empty[b], 0);
      }
      // Per chunk: a partial transpose across the warp leaves lane (a, b) with eight consecutive
      // vocabulary columns 8a..8a+7 of the tokens b, 8 + b, 16 + b, 24 + b: 16 bytes of a logits row
      // per token, so that one store instruction writes 64 contiguous bytes of eight rows; the
      // statistics of a token's 32 values are finished by two shuffle steps across its four lanes.
      const int va = lane >> 3, tb = lane & 7;
      const int v_mine = v_left - 8 * va;   // valid columns among this lane's eight (may be <= 0)
#pragma unroll
      for (int ci = 0; ci < kCh; ++ci) {
        const int c = c_first + ci * (kLmEpiWarps / 4);
        if (c >= n_chunks) break;
        lm::warp_transpose_pairs(u[ci], lane);
        uint32_t (&pk)[16] = u[ci];
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          const int tok = tok0 + c * 32 + g * 8 + tb;
          if (tok < p.M && v_mine > 0) {
            __nv_bfloat16 *dst = p.logits + (int64_t)tok * p.row_stride + vrow0 + 8 * va;
            if (v_mine >= 8) {
              *reinterpret_cast<uint4 *>(dst) = make_uint4(pk[g * 4], pk[g * 4 + 1], pk[g * 4 + 2], pk[g * 4 + 3]);
            } else {
#pragma unroll
              for (int i = 0; i < 8; ++i)
                if (i < v_mine) dst[i] = __ushort_as_bfloat16((unsigned short)((i & 1) ? (pk[g * 4 + (i >> 1)] >> 16) : (pk[g * 4 + (i >> 1)] & 0xffffu)));
            }
          }
        }
        if (p.tile_stats) {
          // (max, sum) of the values as stored over the warp's valid columns of each of the four
          // tokens; the four tokens go through every step together so that the shuffles overlap
          float mx[4], sum[4];
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            mx[g] = -INFINITY;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              if (2 * i < v_mine) mx[g] = fmaxf(mx[g], __uint_as_float(pk[g * 4 + i] << 16));
              if (2 * i + 1 < v_mine) mx[g] = fmaxf(mx[g], __uint_as_float(pk[g * 4 + i] & 0xffff0000u));
            }
          }
#pragma unroll
          for (int g = 0; g < 4; ++g) mx[g] = fmaxf(mx[g], __shfl_xor_sync(0xffffffffu, mx[g], 8));
#pragma unroll
          for (int g = 0; g < 4; ++g) mx[g] = fmaxf(mx[g], __shfl_xor_sync(0xffffffffu, mx[g], 16));
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            // a warp whose columns are all past the vocabulary has mx = -inf: the terms are skipped
            const float m2 = mx[g] == -INFINITY ? 0.f : mx[g] * kLog2e;
            sum[g] = 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              if (2 * i < v_mine) sum[g] += fast_exp2(fmaf(__uint_as_float(pk[g * 4 + i] << 16), kLog2e, -m2));
              if (2 * i + 1 < v_mine) sum[g] += fast_exp2(fmaf(__uint_as_float(pk[g * 4 + i] & 0xffff0000u), kLog2e, -m2));
            }
          }
#pragma unroll
          for (int g = 0; g < 4; ++g) sum[g] += __shfl_xor_sync(0xffffffffu, sum[g], 8);
#pragma unroll
          for (int g = 0; g < 4; ++g) sum[g] += __shfl_xor_sync(0xffffffffu, sum[g], 16);
          if (va == 0) {
#pragma unroll
            for (int g = 0; g < 4; ++g) s_ms[(c * 4 + q) * 32 + g * 8 + tb] = make_float2(mx[g] * kLog2e, sum[g]);
          }
        }
      }
      if (p.tile_stats) {
        ok = epi_sync();
        if (!ok) break;
        // merge the four warps' pairs of a token: pairs of (max, sum) combine exactly
        const int st_idx = vt * 2 + (int)rank;
        for (int c = epi; c < n_chunks; c += kLmEpiWarps) {
          const float2 *mc = s_ms + c * 128 + lane;
          const float2 a0 = mc[0], a1 = mc[32], a2 = mc[64], a3 = mc[96];
          const float M2 = fmaxf(fmaxf(a0.x, a1.x), fmaxf(a2.x, a3.x));
          float sum = 0.f;
          if (M2 > -INFINITY)
            sum = (a0.y * fast_exp2(a0.x - M2) + a1.y * fast_exp2(a1.x - M2)) + (a2.y * fast_exp2(a2.x - M2) + a3.y * fast_exp2(a3.x - M2));
          const int tok = tok0 + c * 32 + lane;
          if (tok < p.M && st_idx < p.stat_tiles) p.tile_stats[(int64_t)tok * p.stat_tiles + st_idx] = make_float2(M2, sum);
        }
        ok = epi_sync();  // the scratch is rewritten by the next tile
        if (!ok) break;
      }
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
  lm::cluster_sync_all();  // neither CTA leaves while the other may still signal it or the pair MMA may still run
  if (warp == 1) {
    fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(512) : "memory");
  }
}

// tile_stats [rows][n_tiles] -> the sampling half's sub-segment statistics [rows][nsub]
// (tiles_per_sub blocks of kLmStatCols columns per sub-segment).
__global__ void lm_stats_merge_kernel(const float2 *tile_stats, int rows, int n_tiles, int nsub, int tiles_per_sub, float2 *seg_stats) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= rows * nsub) return;
  const int row = i / nsub, sub = i % nsub;
  const float2 *t = tile_stats + (int64_t)row * n_tiles;
  float M = -INFINITY;
  for (int j = sub * tiles_per_sub; j < min((sub + 1) * tiles_per_sub, n_tiles); ++j) M = fmaxf(M, t[j].x);
  float S = 0.f;
  if (M > -INFINITY)
    for (int j = sub * tiles_per_sub; j < min((sub + 1) * tiles_per_sub, n_tiles); ++j) S += t[j].y * fast_exp2(t[j].x - M);
  seg_stats[i] = make_float2(M, S);
}

}  // namespace spx
