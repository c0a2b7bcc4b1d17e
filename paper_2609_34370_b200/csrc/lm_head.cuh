// LM head on the 5th-generation tensor cores: logits[M, V] = H[M, K] W[V, K]^T in bf16 with fp32
// accumulation, with the sampling half's row statistics produced in the epilogue.
//
// One persistent CTA per SM, warp-specialised:
//   warp 0      producer: one TMA box of H (128 rows x 64 k) and one of W (256 rows x 64 k) per
//               k-step into a ring of shared-memory stages (128-byte swizzle, K-major);
//   warp 1      MMA issuer (one lane): four tcgen05.mma (M 128, N 256, K 16) per k-step into one of
//               two 256-column TMEM accumulators;
//   warps 2-5   epilogue: thread = output row (TMEM lane).  Reads the finished accumulator while the
//               next tile's products run into the other one, rounds to bf16, stores the logits and
//               reduces the row's 256 values - as stored - to (max, sum 2^((x - max) log2 e)).
// Tiles are numbered n-major (tile = n_tile * m_tiles + m_tile) and dealt round-robin, so the CTAs
// that share a block of W run side by side and it crosses HBM once; H is small and lives in L2.
//
// Every wait is bounded: on expiry the CTA raises SPX_DEV_TIMEOUT, all roles leave their loops,
// pending copies get time to land and TMEM is released.
#pragma once
#include <cuda.h>

#include "attn_tc.cuh"
#include "common.cuh"

namespace spx {

constexpr int kLmBM = 128, kLmBN = 256, kLmBK = 64;
constexpr int kLmStages = 4;
constexpr int kLmABytes = kLmBM * kLmBK * 2;
constexpr int kLmBBytes = kLmBN * kLmBK * 2;
constexpr int kLmStageBytes = kLmABytes + kLmBBytes;
constexpr int kLmThreads = 192;
constexpr int kLmSmemBytes = 1024 + kLmStages * kLmStageBytes + 256;

struct LmBarriers {
  uint64_t full[kLmStages], empty[kLmStages], acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  volatile int32_t abort;
};

struct LmParams {
  int32_t M, K, V, m_tiles, n_tiles, k_blocks;
  __nv_bfloat16 *logits;
  int64_t row_stride;
  float2 *tile_stats;  // [M][n_tiles]: (max * log2 e, sum 2^((x - max) log2 e)) of the tile's columns; may be NULL
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

__global__ void __launch_bounds__(kLmThreads, 1)
lm_head_kernel(const __grid_constant__ CUtensorMap hmap, const __grid_constant__ CUtensorMap wmap, LmParams p) {
  using namespace tc;
  extern __shared__ __align__(1024) unsigned char lm_smem[];
  unsigned char *stages = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(lm_smem) + 1023) & ~uintptr_t(1023));
  LmBarriers *bars = reinterpret_cast<LmBarriers *>(stages + kLmStages * kLmStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kLmStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&bars->acc_full[b], 1); mbar_init(&bars->acc_empty[b], 4); }
    bars->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "n"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem = bars->tmem_base;
  const int n_tiles_total = p.m_tiles * p.n_tiles;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < n_tiles_total && ok; t += gridDim.x) {
        const int mt = t % p.m_tiles, nt = t / p.m_tiles;
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int s = it % kLmStages;
          if (it >= kLmStages) ok = lm_wait(&bars->empty[s], ((it / kLmStages) - 1) & 1, bars, p.dev_status);
          if (!ok || bars->abort) { ok = false; break; }
          unsigned char *st = stages + s * kLmStageBytes;
          mbar_expect_tx(&bars->full[s], kLmStageBytes);
          tma_load_2d(smem_u32(st), &hmap, &bars->full[s], kb * kLmBK, mt * kLmBM);
          tma_load_2d(smem_u32(st + kLmABytes), &wmap, &bars->full[s], kb * kLmBK, nt * kLmBN);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t kIdesc = idesc(kLmBN, false);
      uint32_t it = 0, j = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < n_tiles_total && ok; t += gridDim.x, ++j) {
        const uint32_t b = j & 1;
        if (j >= 2) ok = lm_wait(&bars->acc_empty[b], ((j >> 1) - 1) & 1, bars, p.dev_status);
        if (!ok) break;
        fence_after();
        for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
          const int s = it % kLmStages;
          ok = lm_wait(&bars->full[s], (it / kLmStages) & 1, bars, p.dev_status);
          if (!ok) break;
          fence_after();
          const uint32_t a = smem_u32(stages + s * kLmStageBytes), w = a + kLmABytes;
#pragma unroll
          for (int k4 = 0; k4 < kLmBK / 16; ++k4)
            mma_ss(tmem + b * kLmBN, smem_desc(a + k4 * 32, 16, 1024), smem_desc(w + k4 * 32, 16, 1024), kIdesc, (kb > 0) || (k4 > 0));
          mma_commit(&bars->empty[s]);
        }
        if (ok) mma_commit(&bars->acc_full[b]);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int q = warp & 3;  // TMEM lane quadrant this warp may read
    uint32_t j = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < n_tiles_total && ok; t += gridDim.x, ++j) {
      const int mt = t % p.m_tiles, nt = t / p.m_tiles;
      const uint32_t b = j & 1;
      ok = lm_wait(&bars->acc_full[b], (j >> 1) & 1, bars, p.dev_status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      fence_after();
      const int row = mt * kLmBM + q * 32 + lane;
      const bool row_ok = row < p.M;
      const uint32_t taddr = tmem + b * kLmBN + ((uint32_t)(q * 32) << 16);
      __nv_bfloat16 *dst = p.logits + (int64_t)row * p.row_stride + (int64_t)nt * kLmBN;
      const int cols_left = p.V - nt * kLmBN;  // > 0
      float mx = -INFINITY;
      // pass 1: round, store, row maximum of the stored values
#pragma unroll 1
      for (int c = 0; c < kLmBN / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(taddr + c * 32, r);
        wait_ld();
        uint32_t packed[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) packed[i] = pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
        const int c0 = c * 32;
        if (row_ok) {
          if (c0 + 32 <= cols_left) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
              *reinterpret_cast<uint4 *>(dst + c0 + 8 * i) = make_uint4(packed[4 * i], packed[4 * i + 1], packed[4 * i + 2], packed[4 * i + 3]);
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (c0 + i < cols_left)
                dst[c0 + i] = __ushort_as_bfloat16((unsigned short)((i & 1) ? (packed[i >> 1] >> 16) : (packed[i >> 1] & 0xffffu)));
          }
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          if (c0 + 2 * i < cols_left) mx = fmaxf(mx, __uint_as_float(packed[i] << 16));
          if (c0 + 2 * i + 1 < cols_left) mx = fmaxf(mx, __uint_as_float(packed[i] & 0xffff0000u));
        }
      }
      if (p.tile_stats) {
        // pass 2: sum of 2^((x - max) log2 e) over the stored values
        const float m2 = mx * kLog2e;
        float sum = 0.f;
#pragma unroll 1
        for (int c = 0; c < kLmBN / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(taddr + c * 32, r);
          wait_ld();
          const int c0 = c * 32;
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const uint32_t pk = pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
            if (c0 + 2 * i < cols_left) sum += fast_exp2(fmaf(__uint_as_float(pk << 16), kLog2e, -m2));
            if (c0 + 2 * i + 1 < cols_left) sum += fast_exp2(fmaf(__uint_as_float(pk & 0xffff0000u), kLog2e, -m2));
          }
        }
        if (row_ok) p.tile_stats[(int64_t)row * p.n_tiles + nt] = make_float2(m2, sum);
      }
      fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->acc_empty[b]);
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
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(512) : "memory");
  }
}

// tile_stats [rows][n_tiles] -> the sampling half's sub-segment statistics [rows][nsub]
// (kSubTiles tiles of 256 columns per 2048-token sub-segment).
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
