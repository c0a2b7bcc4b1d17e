// libspx: C ABI, argument validation, workspace layout and kernel launches.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <type_traits>

#include "attn_simt.cuh"
#include "attn_tc.cuh"
#include "attn_tc4.cuh"
#include "common.cuh"
#include "kv_cache.cuh"
#include "select.cuh"
#include "lookahead.cuh"
#include "lm_head.cuh"
#include "plan.cuh"
#include "sampler.cuh"
#include "spx.h"
#if SPX_WAIT_TEST
#include "wait_test.cuh"
#endif

namespace spx {

static thread_local int32_t t_launches = 0;
static thread_local cudaEvent_t t_ev_start = nullptr, t_ev_stop = nullptr;
static thread_local long long *t_prof = nullptr;  // profiling builds only

// spx_verify_step runs its two halves concurrently: the sampling half on an internal stream that
// is forked from and joined back into the caller's stream.  One stream and two events per (host
// thread, device), created on first use.  They are kept for the life of the process: a thread may
// exit after the CUDA runtime has begun to shut down, when destroying a stream is no longer safe,
// so the few handles of an exited thread are deliberately left to the driver's process teardown.
struct SideStream {
  int device = -1;
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr, mid = nullptr;
};
static thread_local SideStream t_side[16];

static SideStream *get_side_stream(int device) {
  if (device < 0 || device >= 16) return nullptr;
  SideStream &s = t_side[device];
  if (s.device != device) {
    // a priority of its own: the sampling kernels are short and latency-bound, and a stream of
    // another priority does not share a hardware queue with the caller's stream.  Built in locals
    // and committed only when all four handles exist, so a failure half way leaks nothing.
    int prio_lo = 0, prio_hi = 0;
    cudaStream_t stream = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr, mid = nullptr;
    bool ok = cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi) == cudaSuccess;
    ok = ok && cudaStreamCreateWithPriority(&stream, cudaStreamNonBlocking, prio_hi) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&fork, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&join, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&mid, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      if (mid) cudaEventDestroy(mid);
      if (join) cudaEventDestroy(join);
      if (fork) cudaEventDestroy(fork);
      if (stream) cudaStreamDestroy(stream);
      return nullptr;
    }
    s.stream = stream; s.fork = fork; s.join = join; s.mid = mid;
    s.device = device;
  }
  return &s;
}

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct DeviceInfo {
  int device = -1;
  int num_sms = 0;
  int cc_major = 0;
  int max_smem_optin = 0;
};

// Properties of the current device (queried per call: cheap attribute reads, no global state).
static bool get_device_info(DeviceInfo *info) {
  if (cudaGetDevice(&info->device) != cudaSuccess) return false;
  if (cudaDeviceGetAttribute(&info->num_sms, cudaDevAttrMultiProcessorCount, info->device) != cudaSuccess) return false;
  if (cudaDeviceGetAttribute(&info->cc_major, cudaDevAttrComputeCapabilityMajor, info->device) != cudaSuccess) return false;
  if (cudaDeviceGetAttribute(&info->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, info->device) != cudaSuccess) return false;
  return true;
}

constexpr int kPlanSmCount = 148;  // workspace sizing must not depend on a device query

// ---------------------------------------------------------------------------------------------
// workspace layout
// ---------------------------------------------------------------------------------------------
struct AttnWs {
  size_t hdr, nchunks, part_base, combine_list, tile_prefix, valid_prefix, cost_prefix, cta_off, req_bad, work, part_ml, part_o, total;
  int32_t max_work, max_part_slots, rows_cap;
};

static spx_status_t check_attn(const spx_attn_args_t *a, bool need_ptrs) {
  if (!a) return SPX_ERR_INVALID_ARG;
  if (a->batch < 0 || a->total_q < a->batch || a->num_q_heads <= 0 || a->num_kv_heads <= 0 || a->head_dim <= 0 ||
      a->page_size <= 0 || a->num_pages < 0 || a->max_pages_per_req < 0 || a->max_q_len < 0)
    return SPX_ERR_INVALID_ARG;
  if (a->kv_dtype != SPX_BF16 && a->kv_dtype != SPX_F32) return SPX_ERR_INVALID_ARG;
  if (!(a->sm_scale >= 0.f) || std::isinf(a->sm_scale)) return SPX_ERR_INVALID_ARG;
  if (a->head_dim != 64 && a->head_dim != 128) return SPX_ERR_UNSUPPORTED;
  if (a->num_q_heads % a->num_kv_heads != 0) return SPX_ERR_UNSUPPORTED;
  if (a->page_size > 128 || (a->page_size & (a->page_size - 1)) != 0) return SPX_ERR_UNSUPPORTED;
  const int max_q = a->max_q_len == 0 ? SPX_MAX_K + 1 : a->max_q_len;
  if (max_q > SPX_MAX_K + 1) return SPX_ERR_UNSUPPORTED;
  if ((a->num_q_heads / a->num_kv_heads) * max_q > SPX_MAX_PACKED_ROWS) return SPX_ERR_UNSUPPORTED;
  if (a->kv_stride_page < 0 || a->kv_stride_head < 0 || a->kv_stride_token < a->head_dim) return SPX_ERR_INVALID_ARG;
  if (need_ptrs && a->batch > 0) {
    if (!a->q || !a->k_cache || !a->v_cache || !a->block_table || !a->seq_lens || !a->q_indptr || !a->out)
      return SPX_ERR_INVALID_ARG;
    const int es = a->kv_dtype == SPX_BF16 ? 2 : 4;
    if (((uintptr_t)a->q | (uintptr_t)a->k_cache | (uintptr_t)a->v_cache | (uintptr_t)a->out) & 15) return SPX_ERR_INVALID_ARG;
    if (((a->kv_stride_page * es) | (a->kv_stride_head * es) | (a->kv_stride_token * es)) & 15) return SPX_ERR_INVALID_ARG;
  }
  return SPX_OK;
}

static AttnWs attn_ws_layout(const spx_attn_args_t *a) {
  AttnWs w{};
  const int max_q = a->max_q_len == 0 ? SPX_MAX_K + 1 : a->max_q_len;
  const int G = a->num_q_heads / a->num_kv_heads;
  w.rows_cap = G * max_q;
  // one entry per (request, kv head) pair plus one per cut of the tile axis; a cut adds at most
  // one chunk to a pair, so the split pairs have at most two chunks per cut between them
  const size_t pairs = (size_t)a->batch * a->num_kv_heads;
  w.max_work = (int)(pairs + kPlanSmCount + 1);
  w.max_part_slots = 2 * kPlanSmCount;
  size_t off = 0;
  w.hdr = off; off = align_up(off + sizeof(PlanHeader), 256);
  w.nchunks = off; off = align_up(off + sizeof(int32_t) * pairs, 256);
  w.part_base = off; off = align_up(off + sizeof(int32_t) * pairs, 256);
  w.combine_list = off; off = align_up(off + sizeof(CombineEntry) * (pairs > (size_t)kCombineListPad ? pairs : (size_t)kCombineListPad), 256);
  w.tile_prefix = off; off = align_up(off + sizeof(int32_t) * ((size_t)a->batch + 1), 256);
  w.valid_prefix = off; off = align_up(off + sizeof(int32_t) * ((size_t)a->batch + 1), 256);
  w.cost_prefix = off; off = align_up(off + sizeof(int32_t) * ((size_t)a->batch + 1), 256);
  w.cta_off = off; off = align_up(off + sizeof(int32_t) * (kPlanSmCount + 1), 256);
  w.req_bad = off; off = align_up(off + sizeof(int32_t) * (size_t)a->batch, 256);
  w.work = off; off = align_up(off + sizeof(WorkEntry) * (size_t)w.max_work, 256);
  const size_t slots = (size_t)w.max_part_slots;
  w.part_ml = off; off = align_up(off + sizeof(float2) * slots * w.rows_cap, 256);
  w.part_o = off; off = align_up(off + sizeof(float) * slots * w.rows_cap * a->head_dim, 256);
  w.total = off;
  return w;
}

struct SampleWs {
  size_t seg_stats, seg_resid, req_norm, row_scale, row_req, row_thresh, row_z, req_thresh, seg_pmass, total;
  int32_t nseg, nsub;
};

static spx_status_t check_sample(const spx_sample_args_t *s, bool need_ptrs) {
  if (!s) return SPX_ERR_INVALID_ARG;
  if (s->batch < 0 || s->total_q < s->batch || s->vocab <= 0 || s->logits_row_stride < s->vocab) return SPX_ERR_INVALID_ARG;
  if (s->logits_dtype != SPX_BF16 && s->logits_dtype != SPX_F32) return SPX_ERR_INVALID_ARG;
  const int vec = s->logits_dtype == SPX_BF16 ? 8 : 4;
  if (s->logits_row_stride % vec != 0) return SPX_ERR_INVALID_ARG;
  if ((int64_t)s->total_q - s->batch > (int64_t)s->batch * SPX_MAX_K) return SPX_ERR_INVALID_ARG;
  if (need_ptrs && s->batch > 0) {
    const int td = s->total_q - s->batch;
    if (!s->target_logits || !s->q_indptr || !s->u_sample || !s->accepted_len || !s->out_tokens) return SPX_ERR_INVALID_ARG;
    if (td > 0 && (!s->draft_logits || !s->draft_token_ids || !s->u_accept)) return SPX_ERR_INVALID_ARG;
    if (((uintptr_t)s->target_logits | (uintptr_t)s->draft_logits) & 15) return SPX_ERR_INVALID_ARG;
  }
  return SPX_OK;
}

static SampleWs sample_ws_layout(const spx_sample_args_t *s) {
  SampleWs w{};
  w.nseg = (s->vocab + kSegElems - 1) / kSegElems;
  w.nsub = (s->vocab + kSubElems - 1) / kSubElems;
  const size_t rows = (size_t)s->total_q + (size_t)(s->total_q - s->batch);
  size_t off = 0;
  w.seg_stats = off; off = align_up(off + sizeof(float2) * rows * w.nsub, 256);
  w.seg_resid = off; off = align_up(off + sizeof(float) * (size_t)s->batch * w.nseg, 256);
  w.req_norm = off; off = align_up(off + sizeof(float4) * (size_t)s->batch, 256);
  w.row_scale = off;
  const bool filtered = s->top_k || s->top_p;
  if (s->temperature || filtered) off = align_up(off + sizeof(float) * rows, 256);
  if (filtered) {
    w.row_req = off; off = align_up(off + sizeof(int32_t) * rows, 256);
    w.row_thresh = off; off = align_up(off + sizeof(uint32_t) * rows, 256);
    w.row_z = off; off = align_up(off + sizeof(double) * rows, 256);
    w.req_thresh = off; off = align_up(off + sizeof(uint2) * (size_t)s->batch, 256);
    w.seg_pmass = off; off = align_up(off + sizeof(float) * (size_t)s->batch * w.nseg, 256);
  }
  w.total = off;
  return w;
}


// ---------------------------------------------------------------------------------------------
// TMA tensor maps over the KV pools
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = [] {
    void *ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess) ptr = nullptr;
    return reinterpret_cast<EncodeTiledFn>(ptr);
  }();
  return fn;
}

// 4-D bf16 view of a pool: dims ordered by increasing stride, (d, head, token, page) when heads are
// the inner dimension and (d, token, head, page) otherwise; one box = one page x one kv-head x 64
// columns, 128-byte swizzle.  (A 5-D view that fetches both 64-column halves of a page with one
// box was measured slower: 5.3 TB/s against 6.1 TB/s on the selective-mix workload.)
static bool make_pool_map(CUtensorMap *map, const void *pool, const spx_attn_args_t *a, bool head_inner) {
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return false;
  const cuuint64_t D = a->head_dim, P = a->page_size, H = a->num_kv_heads, N = a->num_pages > 0 ? a->num_pages : 1;
  const cuuint64_t st = (cuuint64_t)a->kv_stride_token * 2, sh = (cuuint64_t)a->kv_stride_head * 2,
                   sp = (cuuint64_t)a->kv_stride_page * 2;
  cuuint64_t dims[4], strides[3];
  cuuint32_t box[4], estr[4] = {1, 1, 1, 1};
  if (head_inner) {
    dims[0] = D; dims[1] = H; dims[2] = P; dims[3] = N;
    strides[0] = sh; strides[1] = st; strides[2] = sp;
    box[0] = 64; box[1] = 1; box[2] = (cuuint32_t)P; box[3] = 1;
  } else {
    dims[0] = D; dims[1] = P; dims[2] = H; dims[3] = N;
    strides[0] = st; strides[1] = sh; strides[2] = sp;
    box[0] = 64; box[1] = (cuuint32_t)P; box[2] = 1; box[3] = 1;
  }
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(pool), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 3-D bf16 view of the query rows [TQ, Hq, D]: one box = 64 columns x the G heads of one kv-head x
// `rows` consecutive query positions, which lands in shared memory as the packed rows j*G + h of a
// work entry, 128 bytes each, 128-byte swizzle: the K-major A operand of the score MMA.
static bool make_q_map(CUtensorMap *map, const spx_attn_args_t *a, int rows) {
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return false;
  const cuuint64_t D = a->head_dim, H = a->num_q_heads, G = a->num_q_heads / a->num_kv_heads;
  cuuint64_t dims[3] = {D, H, (cuuint64_t)a->total_q};
  cuuint64_t strides[2] = {D * 2, H * D * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)G, (cuuint32_t)rows}, estr[3] = {1, 1, 1};
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(a->q), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The tensor-core kernel handles bf16 pools whose pages hold at least one 8-row swizzle atom.
static bool use_tensor_core_path(const spx_attn_args_t *a) {
  return a->kv_dtype == SPX_BF16 && a->page_size >= 8 && a->num_pages > 0 && a->kv_stride_page > 0 &&
         a->kv_stride_head > 0;
}

// Launch with programmatic stream serialization: the grid may be scheduled while the previous
// kernel of the stream drains; the kernel waits (griddepcontrol.wait) before it touches anything
// the previous kernel wrote.
template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <int D, int MROWS>
static cudaError_t launch_tc4(const CUtensorMap &kmap, const CUtensorMap &vmap, const CUtensorMap &qmap, const AttnParams &p,
                              int num_sms, cudaStream_t stream) {
  using Cfg = Tc4Cfg<D, MROWS>;
  auto kernel = attn_tc4_kernel<D, MROWS>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes);
  if (e != cudaSuccess) return e;
  // (A programmatic dependent launch behind the planner was measured: no gain, the early-resident
  // CTAs only take registers away from the sampling kernels that run beside them.)
  if (t_ev_start) cudaEventRecord(t_ev_start, stream);
  kernel<<<num_sms, kTcThreads, Cfg::kSmemBytes, stream>>>(kmap, vmap, qmap, p);
  if (t_ev_stop) cudaEventRecord(t_ev_stop, stream);
  ++t_launches;
  return cudaGetLastError();
}

template <int D, int QROWS>
static cudaError_t launch_tc(const CUtensorMap &kmap, const CUtensorMap &vmap, const AttnParams &p, int num_sms,
                             cudaStream_t stream) {
  using Cfg = TcCfg<D, QROWS>;
  auto kernel = attn_tc_kernel<D, QROWS>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes);
  if (e != cudaSuccess) return e;
  // (A programmatic dependent launch behind the planner was measured: no gain, the early-resident
  // CTAs only take registers away from the sampling kernels that run beside them.)
  if (t_ev_start) cudaEventRecord(t_ev_start, stream);
  kernel<<<num_sms, kTcThreads, Cfg::kSmemBytes, stream>>>(kmap, vmap, p);
  if (t_ev_stop) cudaEventRecord(t_ev_stop, stream);
  ++t_launches;
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// launches
// ---------------------------------------------------------------------------------------------
enum { kPhasePlan = 1, kPhaseMain = 2, kPhaseAll = 3 };                        // attention: planner, kernels behind it
enum { kPhaseStats = 1, kPhaseTail = 2, kPhaseFilter = 4, kPhaseSampAll = 7 };  // sampling: statistics, top-k / top-p thresholds, the rest

static spx_status_t launch_attention(const spx_attn_args_t *a, unsigned char *ws, int32_t *dev_status,
                                     cudaStream_t stream, const DeviceInfo &dev, int phases = kPhaseAll) {
  if (a->batch == 0) return SPX_OK;
  const AttnWs w = attn_ws_layout(a);
  AttnParams p{};
  p.batch = a->batch; p.total_q = a->total_q;
  p.max_q_len = a->max_q_len == 0 ? SPX_MAX_K + 1 : a->max_q_len;
  p.Hq = a->num_q_heads; p.Hkv = a->num_kv_heads; p.G = p.Hq / p.Hkv; p.D = a->head_dim; p.P = a->page_size;
  p.log2P = 0;
  while ((1 << p.log2P) < p.P) ++p.log2P;
  p.num_pages = a->num_pages; p.max_pages_per_req = a->max_pages_per_req;
  const float scale = a->sm_scale == 0.f ? 1.f / sqrtf((float)a->head_dim) : a->sm_scale;
  p.scale_log2 = scale * kLog2e;
  p.q = a->q; p.k_cache = a->k_cache; p.v_cache = a->v_cache;
  p.stride_page = a->kv_stride_page; p.stride_head = a->kv_stride_head; p.stride_token = a->kv_stride_token;
  p.block_table = a->block_table; p.seq_lens = a->seq_lens; p.q_indptr = a->q_indptr;
  p.out = a->out; p.lse = a->lse;
  p.hdr = reinterpret_cast<PlanHeader *>(ws + w.hdr);
  p.pair_nchunks = reinterpret_cast<int32_t *>(ws + w.nchunks);
  p.pair_part_base = reinterpret_cast<int32_t *>(ws + w.part_base);
  p.combine_list = reinterpret_cast<CombineEntry *>(ws + w.combine_list);
  p.tile_prefix = reinterpret_cast<int32_t *>(ws + w.tile_prefix);
  p.valid_prefix = reinterpret_cast<int32_t *>(ws + w.valid_prefix);
  p.cost_prefix = reinterpret_cast<int32_t *>(ws + w.cost_prefix);
  p.cta_off = reinterpret_cast<int32_t *>(ws + w.cta_off);
  p.req_bad = reinterpret_cast<int32_t *>(ws + w.req_bad);
  p.work = reinterpret_cast<WorkEntry *>(ws + w.work);
  p.max_work = w.max_work;
  p.max_part_slots = w.max_part_slots;
  p.part_ml = reinterpret_cast<float2 *>(ws + w.part_ml);
  p.part_o = reinterpret_cast<float *>(ws + w.part_o);
  p.rows_cap = w.rows_cap;
  p.dev_status = dev_status;
  p.prof = t_prof;

  // one range of the plan per CTA of the persistent kernels, never more than the workspace was sized for
  const int sms = dev.num_sms < kPlanSmCount ? dev.num_sms : kPlanSmCount;
  if (phases & kPhasePlan) {
    plan_kernel<<<1, 1024, 0, stream>>>(p, sms);
    ++t_launches;
    if (cudaGetLastError() != cudaSuccess) return SPX_ERR_CUDA;
  }
  if (!(phases & kPhaseMain)) return SPX_OK;

  cudaError_t e;
  if (use_tensor_core_path(a)) {
    p.head_inner = a->kv_stride_head < a->kv_stride_token ? 1 : 0;
    CUtensorMap kmap, vmap;
    if (!make_pool_map(&kmap, a->k_cache, a, p.head_inner) || !make_pool_map(&vmap, a->v_cache, a, p.head_inner))
      return SPX_ERR_CUDA;
    if (p.rows_cap <= 64) {
      // the packed query rows of a work entry arrive by one box pair of a 3-D map over Q
      CUtensorMap qmap;
      p.q_box_rows = p.max_q_len < p.total_q ? p.max_q_len : p.total_q;
      if (!make_q_map(&qmap, a, p.q_box_rows)) return SPX_ERR_CUDA;
      if (p.rows_cap <= 32)
        e = p.D == 128 ? launch_tc4<128, 32>(kmap, vmap, qmap, p, sms, stream) : launch_tc4<64, 32>(kmap, vmap, qmap, p, sms, stream);
      else
        e = p.D == 128 ? launch_tc4<128, 64>(kmap, vmap, qmap, p, sms, stream) : launch_tc4<64, 64>(kmap, vmap, qmap, p, sms, stream);
    } else
      e = p.D == 128 ? launch_tc<128, 128>(kmap, vmap, p, sms, stream) : launch_tc<64, 128>(kmap, vmap, p, sms, stream);
  } else {
    const SimtSmem lay(p.rows_cap, p.D);
    if (lay.total > dev.max_smem_optin) return SPX_ERR_UNSUPPORTED;
    auto launch_simt = [&](auto kernel) -> cudaError_t {
      cudaError_t er = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, lay.total);
      if (er != cudaSuccess) return er;
      int per_sm = 0;
      er = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kSimtThreads, lay.total);
      if (er != cudaSuccess) return er;
      if (per_sm < 1) per_sm = 1;
      if (t_ev_start) cudaEventRecord(t_ev_start, stream);
      kernel<<<dev.num_sms * per_sm, kSimtThreads, lay.total, stream>>>(p);
      if (t_ev_stop) cudaEventRecord(t_ev_stop, stream);
      ++t_launches;
      return cudaGetLastError();
    };
    if (a->kv_dtype == SPX_F32)
      e = p.D == 64 ? launch_simt(attn_simt_kernel<float, 64>) : launch_simt(attn_simt_kernel<float, 128>);
    else
      e = p.D == 64 ? launch_simt(attn_simt_kernel<__nv_bfloat16, 64>) : launch_simt(attn_simt_kernel<__nv_bfloat16, 128>);
  }
  if (e != cudaSuccess) return SPX_ERR_CUDA;
  // one row of blocks per listed pair on the named workloads (a cut of the tile axis lists at most one
  // pair); longer lists - many invalid requests - are walked
  const int pairs_all = p.batch * p.Hkv;
  const dim3 cgrid(pairs_all < kPlanSmCount ? pairs_all : kPlanSmCount, (p.rows_cap * (p.D / 4) + kCombineThreads - 1) / kCombineThreads);
  e = a->kv_dtype == SPX_F32 ? launch_pdl(combine_kernel<float>, cgrid, dim3(kCombineThreads), 0, stream, p)
                             : launch_pdl(combine_kernel<__nv_bfloat16>, cgrid, dim3(kCombineThreads), 0, stream, p);
  ++t_launches;
  return e == cudaSuccess ? SPX_OK : SPX_ERR_CUDA;
}

template <typename T, bool kScaled, bool kFiltered = false>
static spx_status_t launch_sampler_t(const SampleParams &p, cudaStream_t stream, int num_sms, int phases,
                                     const float2 *tile_stats = nullptr, int spare_sms = 0) {
  // SMs the bulk-copy statistics kernel leaves alone (its CTAs fill an SM's registers and shared
  // memory: nothing else starts on an SM it occupies)
  const int ring_sms = num_sms - spare_sms > 0 ? num_sms - spare_sms : num_sms;
  const int rows = p.total_q + p.total_d;
  const int n_units = rows * p.nsub;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, row_stats_kernel<T, kScaled>, kSampThreads, 0) != cudaSuccess)
    return SPX_ERR_CUDA;
  if (per_sm < 1) per_sm = 1;
  int grid = num_sms * per_sm;
  const int max_grid = (n_units + kSampThreads / 32 - 1) / (kSampThreads / 32);
  if (grid > max_grid) grid = max_grid;
  if (phases & kPhaseStats) {
    if constexpr (kScaled) {
      row_scale_kernel<<<(p.batch + 127) / 128, 128, 0, stream>>>(p);
      ++t_launches;
    }
    if constexpr (std::is_same<T, __nv_bfloat16>::value) {
      // bf16 logits: the bulk-copy ring kernel, one CTA per SM
      static_assert(kSubElems == 2048, "the ring kernel reduces 2048-token sub-segments");
      if (cudaFuncSetAttribute(row_stats_ring_kernel<kScaled>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingSmemBytes) !=
          cudaSuccess)
        return SPX_ERR_CUDA;
      const int chunks_per_row = (p.vocab + kRingStageElems - 1) / kRingStageElems;
      const int n_chunks = (rows - p.first_row) * chunks_per_row;
      if (p.first_row > 0) {
        // the target rows' statistics came out of the LM-head epilogue, per 256-column tile: fold them
        // into sub-segments; only the draft rows are read here
        const int n = p.first_row * p.nsub;
        lm_stats_merge_kernel<<<(n + 255) / 256, 256, 0, stream>>>(tile_stats, p.first_row, (p.vocab + kLmStatCols - 1) / kLmStatCols, p.nsub,
                                                                  kSubElems / kLmStatCols, p.seg_stats);
        ++t_launches;
      }
      if (n_chunks > 0)
        row_stats_ring_kernel<kScaled><<<ring_sms < n_chunks ? ring_sms : n_chunks, kRingThreads, kRingSmemBytes, stream>>>(
            p, chunks_per_row, n_chunks);
    } else {
      row_stats_kernel<T, kScaled><<<grid, kSampThreads, 0, stream>>>(p, n_units);
    }
    ++t_launches;
  }
  if constexpr (kFiltered) {
    if (phases & kPhaseFilter) {
      if (cudaFuncSetAttribute(filter_rows_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFilterSmemBytes) != cudaSuccess)
        return SPX_ERR_CUDA;
      if (p.top_k) {   // the short way for small K; without a top-k array every row is the general kernel's
        topk_list_kernel<T><<<rows, kTopkThreads, 0, stream>>>(p);
        ++t_launches;
      }
      filter_rows_kernel<T><<<rows, kFilterThreads, kFilterSmemBytes, stream>>>(p);
      ++t_launches;
    }
  }
  if (phases & kPhaseTail) {
    const int accept_blocks = (p.batch * 32 + 127) / 128;
    accept_kernel<T, kScaled, kFiltered><<<accept_blocks + (kScaled ? p.batch : 0), 128, 0, stream>>>(p, accept_blocks);
    resid_mass_kernel<T, kScaled, kFiltered><<<dim3(p.nseg, p.batch), kResidThreads, sizeof(T) == 2 ? kResidStageBytes : 0, stream>>>(p);
    if (launch_pdl(resid_pick_kernel<T, kScaled, kFiltered>, dim3(p.batch), dim3(kResidThreads), 0, stream, p) != cudaSuccess)
      return SPX_ERR_CUDA;
    t_launches += 3;
  }
  return cudaGetLastError() == cudaSuccess ? SPX_OK : SPX_ERR_CUDA;
}

static spx_status_t launch_sampler(const spx_sample_args_t *s, unsigned char *ws, int32_t *dev_status,
                                   cudaStream_t stream, int num_sms, int phases = kPhaseSampAll, int spare_sms = 0) {
  if (s->batch == 0) return SPX_OK;
  if (s->batch > 65535) return SPX_ERR_UNSUPPORTED;  // grid.y limit of the residual pass
  const SampleWs w = sample_ws_layout(s);
  SampleParams p{};
  p.batch = s->batch; p.total_q = s->total_q; p.total_d = s->total_q - s->batch; p.vocab = s->vocab; p.nseg = w.nseg; p.nsub = w.nsub;
  if ((int64_t)(p.total_q + p.total_d) * p.nsub > 0x7fffffff) return SPX_ERR_UNSUPPORTED;
  p.row_stride = s->logits_row_stride;
  p.target = s->target_logits; p.draft = s->draft_logits; p.draft_ids = s->draft_token_ids;
  p.q_indptr = s->q_indptr; p.u_accept = s->u_accept; p.u_sample = s->u_sample;
  p.accepted_len = s->accepted_len; p.out_tokens = s->out_tokens; p.diag_ratio = s->diag_ratio;
  p.seg_stats = reinterpret_cast<float2 *>(ws + w.seg_stats);
  p.seg_resid = reinterpret_cast<float *>(ws + w.seg_resid);
  p.req_norm = reinterpret_cast<float4 *>(ws + w.req_norm);
  p.dev_status = dev_status;
  if (s->top_k || s->top_p) {
    p.temperature = s->temperature; p.top_k = s->top_k; p.top_p = s->top_p;
    p.row_scale = reinterpret_cast<float *>(ws + w.row_scale);
    p.row_req = reinterpret_cast<int32_t *>(ws + w.row_req);
    p.row_thresh = reinterpret_cast<uint32_t *>(ws + w.row_thresh);
    p.row_z = reinterpret_cast<double *>(ws + w.row_z);
    p.req_thresh = reinterpret_cast<uint2 *>(ws + w.req_thresh);
    p.seg_pmass = reinterpret_cast<float *>(ws + w.seg_pmass);
    return s->logits_dtype == SPX_BF16 ? launch_sampler_t<__nv_bfloat16, true, true>(p, stream, num_sms, phases, nullptr, spare_sms)
                                       : launch_sampler_t<float, true, true>(p, stream, num_sms, phases, nullptr, spare_sms);
  }
  if (s->temperature) {
    p.temperature = s->temperature;
    p.row_scale = reinterpret_cast<float *>(ws + w.row_scale);
    return s->logits_dtype == SPX_BF16 ? launch_sampler_t<__nv_bfloat16, true>(p, stream, num_sms, phases, nullptr, spare_sms)
                                       : launch_sampler_t<float, true>(p, stream, num_sms, phases, nullptr, spare_sms);
  }
  if (s->logits_dtype == SPX_BF16 && s->target_tile_stats) {
    p.first_row = p.total_q;   // base rule on bf16 logits: the LM head's statistics stand in for the target rows
    return launch_sampler_t<__nv_bfloat16, false>(p, stream, num_sms, phases, reinterpret_cast<const float2 *>(s->target_tile_stats), spare_sms);
  }
  return s->logits_dtype == SPX_BF16 ? launch_sampler_t<__nv_bfloat16, false>(p, stream, num_sms, phases, nullptr, spare_sms)
                                     : launch_sampler_t<float, false>(p, stream, num_sms, phases, nullptr, spare_sms);
}

static spx_status_t check_ws(const void *ws, size_t ws_bytes, size_t need, const int32_t *dev_status) {
  if (!dev_status) return SPX_ERR_INVALID_ARG;
  if (need == 0) return SPX_OK;
  if (!ws || ((uintptr_t)ws & 255) || ws_bytes < need) return SPX_ERR_WORKSPACE;
  return SPX_OK;
}

}  // namespace spx

using namespace spx;

extern "C" {

size_t spx_workspace_size(const spx_attn_args_t *attn, const spx_sample_args_t *sample) {
  size_t total = 0;
  if (attn) {
    if (check_attn(attn, false) != SPX_OK) return 0;
    total += attn_ws_layout(attn).total;
  }
  if (sample) {
    if (check_sample(sample, false) != SPX_OK) return 0;
    total += sample_ws_layout(sample).total;
  }
  return total ? total : 256;
}

spx_status_t spx_verify_attention(const spx_attn_args_t *args, void *ws, size_t ws_bytes, int32_t *dev_status,
                                  void *cuda_stream) {
  t_launches = 0;
  spx_status_t st = check_attn(args, true);
  if (st != SPX_OK) return st;
  st = check_ws(ws, ws_bytes, attn_ws_layout(args).total, dev_status);
  if (st != SPX_OK) return st;
  DeviceInfo dev;
  if (!get_device_info(&dev) || dev.cc_major < 10) return SPX_ERR_CUDA;
  return launch_attention(args, static_cast<unsigned char *>(ws), dev_status, static_cast<cudaStream_t>(cuda_stream), dev);
}

spx_status_t spx_rejection_sample(const spx_sample_args_t *args, void *ws, size_t ws_bytes, int32_t *dev_status,
                                  void *cuda_stream) {
  t_launches = 0;
  spx_status_t st = check_sample(args, true);
  if (st != SPX_OK) return st;
  st = check_ws(ws, ws_bytes, sample_ws_layout(args).total, dev_status);
  if (st != SPX_OK) return st;
  DeviceInfo dev;
  if (!get_device_info(&dev) || dev.cc_major < 10) return SPX_ERR_CUDA;
  return launch_sampler(args, static_cast<unsigned char *>(ws), dev_status, static_cast<cudaStream_t>(cuda_stream), dev.num_sms);
}

spx_status_t spx_verify_step(const spx_attn_args_t *attn, const spx_sample_args_t *sample, void *ws, size_t ws_bytes,
                             int32_t *dev_status, void *cuda_stream) {
  t_launches = 0;
  spx_status_t st = check_attn(attn, true);
  if (st != SPX_OK) return st;
  st = check_sample(sample, true);
  if (st != SPX_OK) return st;
  if (attn->batch != sample->batch || attn->total_q != sample->total_q) return SPX_ERR_INVALID_ARG;
  const size_t attn_bytes = attn_ws_layout(attn).total;
  st = check_ws(ws, ws_bytes, attn_bytes + sample_ws_layout(sample).total, dev_status);
  if (st != SPX_OK) return st;
  DeviceInfo dev;
  if (!get_device_info(&dev) || dev.cc_major < 10) return SPX_ERR_CUDA;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  unsigned char *base = static_cast<unsigned char *>(ws);
  // The halves are independent given their inputs: the sampling half is forked onto the internal
  // stream and joined back before the call hands the caller's stream back.  On the Llama-3-8B
  // shape the step then runs as: logits statistics (about 31 us, every SM but one), attention
  // (about 111 us; its CTAs take the SMs as the statistics CTAs leave them, with the accept
  // kernel's few warps beside them), and a tail of about 17 us in which the residual kernel and
  // the combine kernel share the SMs the attention CTAs free.  The residual kernel cannot run beside
  // the attention CTAs: their six warps leave about 3000 registers free on two of an SM's four
  // sub-partitions, less than two of its warps need; a four-warp variant that did fit slowed the
  // attention kernel by 27 us a step.
  SideStream *side = get_side_stream(dev.device);
  if (!side) return SPX_ERR_CUDA;
  bool ok = cudaEventRecord(side->fork, stream) == cudaSuccess;
  ok = ok && cudaStreamWaitEvent(side->stream, side->fork, 0) == cudaSuccess;
  if (!ok) return SPX_ERR_CUDA;
  // The logits pass is on the step's critical path (the attention CTAs need its SMs), so it is
  // launched first.  It keeps one SM clear: a CTA of it fills an SM, and on a full GPU the
  // one-block planner, which the attention kernel waits for, ran only when the first logits CTA
  // had left (8 us per step on the Llama-3-8B shape).
  // From here on the internal stream is forked: whatever fails below, it is joined back into the
  // caller's stream before the call returns (an unjoined fork would invalidate a stream capture
  // and, outside one, leave the caller's stream unordered against sampling kernels already queued).
  // With top-k / top-p the threshold kernels sweep the logits once more, with blocks that do not fit
  // beside the attention CTAs: left to themselves the two halves take the SMs from each other and the
  // step is longer than their sum.  The attention kernel is therefore held back until the thresholds
  // are known; accept, residual and draw then run beside and behind it as in the base rule.
  const bool filtered = sample->top_k || sample->top_p;
  spx_status_t s1 = launch_sampler(sample, base + attn_bytes, dev_status, side->stream, dev.num_sms,
                                   filtered ? (kPhaseStats | kPhaseFilter) : kPhaseSampAll, 1);
  const spx_status_t s0 = launch_attention(attn, base, dev_status, stream, dev, kPhasePlan);
  bool held = true;
  if (filtered) {
    held = cudaEventRecord(side->mid, side->stream) == cudaSuccess && cudaStreamWaitEvent(stream, side->mid, 0) == cudaSuccess;
    const spx_status_t s1b = launch_sampler(sample, base + attn_bytes, dev_status, side->stream, dev.num_sms, kPhaseTail, 1);
    if (s1 == SPX_OK) s1 = s1b;
  }
  const bool rec = cudaEventRecord(side->join, side->stream) == cudaSuccess;
  const spx_status_t s2 = s0 == SPX_OK && held ? launch_attention(attn, base, dev_status, stream, dev, kPhaseMain) : s0;
  const bool joined = rec && cudaStreamWaitEvent(stream, side->join, 0) == cudaSuccess;
  if (!joined || !held) return SPX_ERR_CUDA;
  return s0 != SPX_OK ? s0 : s1 != SPX_OK ? s1 : s2;
}

// ---- host-buffer convenience ---------------------------------------------------------------
namespace {
struct HostStepLayout {
  size_t q, k, v, bt, sl, qi, out, lse, tl, dl, ids, ua, us, tau, topk, topp, acc, tok, status, ws, total;
  size_t q_bytes, kv_bytes, bt_bytes, out_bytes, lse_bytes, tl_bytes, dl_bytes, ws_bytes;
};
HostStepLayout host_layout(const spx_attn_args_t *a, const spx_sample_args_t *s, int64_t kv_pool_elems) {
  HostStepLayout L{};
  const size_t es = a->kv_dtype == SPX_BF16 ? 2 : 4, ls = s->logits_dtype == SPX_BF16 ? 2 : 4;
  const size_t B = a->batch, TQ = a->total_q, TD = TQ - B;
  L.q_bytes = TQ * a->num_q_heads * a->head_dim * es;
  L.kv_bytes = (size_t)kv_pool_elems * es;
  L.bt_bytes = B * (size_t)a->max_pages_per_req * 4;
  L.out_bytes = L.q_bytes;
  L.lse_bytes = TQ * a->num_q_heads * 4;
  L.tl_bytes = TQ ? ((TQ - 1) * (size_t)s->logits_row_stride + s->vocab) * ls : 0;
  L.dl_bytes = TD ? ((TD - 1) * (size_t)s->logits_row_stride + s->vocab) * ls : 0;
  L.ws_bytes = spx_workspace_size(a, s);
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t o = off; off = align_up(off + bytes, 256); return o; };
  L.q = take(L.q_bytes); L.k = take(L.kv_bytes); L.v = take(L.kv_bytes); L.bt = take(L.bt_bytes);
  L.sl = take(B * 4); L.qi = take((B + 1) * 4); L.out = take(L.out_bytes); L.lse = take(L.lse_bytes);
  L.tl = take(L.tl_bytes); L.dl = take(L.dl_bytes); L.ids = take(TD * 4); L.ua = take(TD * 4); L.us = take(B * 4);
  L.tau = take(s->temperature ? B * 4 : 0); L.topk = take(s->top_k ? B * 4 : 0); L.topp = take(s->top_p ? B * 4 : 0);
  L.acc = take(B * 4); L.tok = take(TQ * 4); L.status = take(4); L.ws = take(L.ws_bytes);
  L.total = off;
  return L;
}
}  // namespace

size_t spx_host_step_arena_size(const spx_attn_args_t *attn, const spx_sample_args_t *sample, int64_t kv_pool_elems) {
  if (check_attn(attn, false) != SPX_OK || check_sample(sample, false) != SPX_OK || kv_pool_elems < 0) return 0;
  if (attn->batch != sample->batch || attn->total_q != sample->total_q) return 0;
  return host_layout(attn, sample, kv_pool_elems).total;
}

spx_status_t spx_verify_step_host(const spx_attn_args_t *attn, const spx_sample_args_t *sample, int64_t kv_pool_elems,
                                  void *dev_arena, size_t arena_bytes, int32_t *dev_status_host, void *cuda_stream) {
  t_launches = 0;
  if (check_attn(attn, false) != SPX_OK || check_sample(sample, false) != SPX_OK || kv_pool_elems < 0 || !dev_status_host)
    return SPX_ERR_INVALID_ARG;
  if (attn->batch != sample->batch || attn->total_q != sample->total_q) return SPX_ERR_INVALID_ARG;
  const HostStepLayout L = host_layout(attn, sample, kv_pool_elems);
  if (!dev_arena || ((uintptr_t)dev_arena & 255) || arena_bytes < L.total) return SPX_ERR_WORKSPACE;
  unsigned char *d = static_cast<unsigned char *>(dev_arena);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const size_t B = attn->batch, TQ = attn->total_q, TD = TQ - B;
  bool ok = true;
  auto h2d = [&](size_t off, const void *src, size_t bytes) {
    if (bytes && src) ok = ok && cudaMemcpyAsync(d + off, src, bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  };
  auto d2h = [&](void *dst, size_t off, size_t bytes) {
    if (bytes && dst) ok = ok && cudaMemcpyAsync(dst, d + off, bytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
  };
  h2d(L.q, attn->q, L.q_bytes); h2d(L.k, attn->k_cache, L.kv_bytes); h2d(L.v, attn->v_cache, L.kv_bytes);
  h2d(L.bt, attn->block_table, L.bt_bytes); h2d(L.sl, attn->seq_lens, B * 4); h2d(L.qi, attn->q_indptr, (B + 1) * 4);
  h2d(L.tl, sample->target_logits, L.tl_bytes); h2d(L.dl, sample->draft_logits, L.dl_bytes);
  h2d(L.ids, sample->draft_token_ids, TD * 4); h2d(L.ua, sample->u_accept, TD * 4); h2d(L.us, sample->u_sample, B * 4);
  h2d(L.tau, sample->temperature, B * 4); h2d(L.topk, sample->top_k, B * 4); h2d(L.topp, sample->top_p, B * 4);
  ok = ok && cudaMemsetAsync(d + L.status, 0, 4, stream) == cudaSuccess;
  if (!ok) return SPX_ERR_CUDA;
  spx_attn_args_t a = *attn;
  spx_sample_args_t s = *sample;
  a.q = d + L.q; a.k_cache = d + L.k; a.v_cache = d + L.v;
  a.block_table = reinterpret_cast<int32_t *>(d + L.bt); a.seq_lens = reinterpret_cast<int32_t *>(d + L.sl);
  a.q_indptr = reinterpret_cast<int32_t *>(d + L.qi); a.out = d + L.out;
  a.lse = attn->lse ? reinterpret_cast<float *>(d + L.lse) : nullptr;
  s.target_logits = d + L.tl; s.draft_logits = d + L.dl; s.draft_token_ids = reinterpret_cast<int32_t *>(d + L.ids);
  s.q_indptr = a.q_indptr; s.u_accept = reinterpret_cast<float *>(d + L.ua); s.u_sample = reinterpret_cast<float *>(d + L.us);
  s.accepted_len = reinterpret_cast<int32_t *>(d + L.acc); s.out_tokens = reinterpret_cast<int32_t *>(d + L.tok);
  s.diag_ratio = nullptr;
  s.target_tile_stats = nullptr;  // a host pointer here: the statistics pass reads the target rows itself
  s.temperature = sample->temperature ? reinterpret_cast<float *>(d + L.tau) : nullptr;
  s.top_k = sample->top_k ? reinterpret_cast<int32_t *>(d + L.topk) : nullptr;
  s.top_p = sample->top_p ? reinterpret_cast<float *>(d + L.topp) : nullptr;
  const spx_status_t st = spx_verify_step(&a, &s, d + L.ws, L.ws_bytes, reinterpret_cast<int32_t *>(d + L.status), cuda_stream);
  if (st != SPX_OK) return st;
  d2h(attn->out, L.out, L.out_bytes); d2h(attn->lse, L.lse, L.lse_bytes);
  d2h(sample->accepted_len, L.acc, B * 4); d2h(sample->out_tokens, L.tok, TQ * 4); d2h(dev_status_host, L.status, 4);
  return ok ? SPX_OK : SPX_ERR_CUDA;
}

// ---- cache maintenance ------------------------------------------------------------------------
spx_status_t spx_kv_append(const spx_kv_append_args_t *a, int32_t *dev_status, void *cuda_stream) {
  t_launches = 0;
  if (!a || !dev_status) return SPX_ERR_INVALID_ARG;
  if (a->batch < 0 || a->total_q < a->batch || a->num_kv_heads <= 0 || a->head_dim <= 0 || a->page_size <= 0 ||
      a->num_pages < 0 || a->max_pages_per_req < 0)
    return SPX_ERR_INVALID_ARG;
  if (a->kv_dtype != SPX_BF16 && a->kv_dtype != SPX_F32) return SPX_ERR_INVALID_ARG;
  if ((a->page_size & (a->page_size - 1)) != 0) return SPX_ERR_UNSUPPORTED;
  const int es = a->kv_dtype == SPX_BF16 ? 2 : 4;
  if ((a->head_dim * es) % 16 != 0) return SPX_ERR_UNSUPPORTED;
  if (a->kv_stride_page < 0 || a->kv_stride_head < 0 || a->kv_stride_token < a->head_dim) return SPX_ERR_INVALID_ARG;
  if (!(a->rope_base >= 0.f) || std::isinf(a->rope_base)) return SPX_ERR_INVALID_ARG;
  const bool rope = a->rope_base > 0.f;
  if (rope && ((a->head_dim & 1) || ((a->head_dim / 2) * es) % 16 != 0 || a->head_dim > kRopeMaxHeadDim)) return SPX_ERR_UNSUPPORTED;
  if (rope && a->q_rows && a->num_q_heads <= 0) return SPX_ERR_INVALID_ARG;
  if (a->batch == 0) return SPX_OK;
  if (!a->new_k || !a->new_v || !a->k_cache || !a->v_cache || !a->block_table || !a->seq_lens || !a->q_indptr)
    return SPX_ERR_INVALID_ARG;
  if (((uintptr_t)a->new_k | (uintptr_t)a->new_v | (uintptr_t)a->k_cache | (uintptr_t)a->v_cache) & 15) return SPX_ERR_INVALID_ARG;
  if (rope && ((uintptr_t)a->q_rows & 15)) return SPX_ERR_INVALID_ARG;
  if (((a->kv_stride_page * es) | (a->kv_stride_head * es) | (a->kv_stride_token * es)) & 15) return SPX_ERR_INVALID_ARG;
  KvAppendParams p{};
  p.batch = a->batch; p.total_q = a->total_q; p.Hkv = a->num_kv_heads; p.D = a->head_dim; p.P = a->page_size;
  while ((1 << p.log2P) < p.P) ++p.log2P;
  p.num_pages = a->num_pages; p.max_pages_per_req = a->max_pages_per_req; p.elem_size = es;
  p.new_k = static_cast<const unsigned char *>(a->new_k); p.new_v = static_cast<const unsigned char *>(a->new_v);
  p.k_cache = static_cast<unsigned char *>(a->k_cache); p.v_cache = static_cast<unsigned char *>(a->v_cache);
  p.stride_page = a->kv_stride_page; p.stride_head = a->kv_stride_head; p.stride_token = a->kv_stride_token;
  p.block_table = a->block_table; p.seq_lens = a->seq_lens; p.q_indptr = a->q_indptr; p.dev_status = dev_status;
  p.rope_base = rope ? (double)a->rope_base : 0.0;
  p.q_rows = rope ? static_cast<unsigned char *>(a->q_rows) : nullptr;
  p.Hq = a->num_q_heads;
  kv_append_kernel<<<a->batch, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(p);
  ++t_launches;
  return cudaGetLastError() == cudaSuccess ? SPX_OK : SPX_ERR_CUDA;
}

spx_status_t spx_kv_rollback(int32_t batch, const int32_t *seq_lens, const int32_t *q_indptr, const int32_t *accepted_len,
                             int32_t *new_seq_lens, int32_t *dev_status, void *cuda_stream) {
  t_launches = 0;
  if (batch < 0 || !dev_status) return SPX_ERR_INVALID_ARG;
  if (batch == 0) return SPX_OK;
  if (!seq_lens || !q_indptr || !accepted_len || !new_seq_lens) return SPX_ERR_INVALID_ARG;
  kv_rollback_kernel<<<(batch + 127) / 128, 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(batch, seq_lens, q_indptr,
                                                                                               accepted_len, new_seq_lens, dev_status);
  ++t_launches;
  return cudaGetLastError() == cudaSuccess ? SPX_OK : SPX_ERR_CUDA;
}

// ---- selective speculation support ------------------------------------------------------------
static spx_status_t check_conf(const spx_conf_args_t *c, bool need_ptrs) {
  if (!c) return SPX_ERR_INVALID_ARG;
  if (c->batch < 0 || c->total_q < c->batch || c->vocab <= 0 || c->logits_row_stride < c->vocab) return SPX_ERR_INVALID_ARG;
  if (c->logits_dtype != SPX_BF16 && c->logits_dtype != SPX_F32) return SPX_ERR_INVALID_ARG;
  if (c->logits_row_stride % (c->logits_dtype == SPX_BF16 ? 8 : 4) != 0) return SPX_ERR_INVALID_ARG;
  if ((int64_t)c->total_q - c->batch > (int64_t)c->batch * SPX_MAX_K) return SPX_ERR_INVALID_ARG;
  if (need_ptrs && c->batch > 0) {
    if (!c->q_indptr || !c->req_conf) return SPX_ERR_INVALID_ARG;
    if (c->total_q > c->batch && (!c->draft_logits || !c->conf_max || ((uintptr_t)c->draft_logits & 15))) return SPX_ERR_INVALID_ARG;
    if (c->conf_tok && c->total_q > c->batch && !c->draft_token_ids) return SPX_ERR_INVALID_ARG;
  }
  return SPX_OK;
}

size_t spx_draft_confidence_workspace(const spx_conf_args_t *c) {
  if (check_conf(c, false) != SPX_OK) return 0;
  const size_t nsub = (c->vocab + kSubElems - 1) / kSubElems;
  return align_up(sizeof(float2) * (size_t)(c->total_q - c->batch) * nsub + 256, 256);
}

spx_status_t spx_draft_confidence(const spx_conf_args_t *c, void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                  void *cuda_stream) {
  t_launches = 0;
  const spx_status_t st = check_conf(c, true);
  if (st != SPX_OK) return st;
  if (!dev_status) return SPX_ERR_INVALID_ARG;
  if (c->batch == 0) return SPX_OK;
  const size_t need = spx_draft_confidence_workspace(c);
  if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return SPX_ERR_WORKSPACE;
  DeviceInfo info;
  if (!get_device_info(&info)) return SPX_ERR_CUDA;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const int td = c->total_q - c->batch;
  const int nsub = (c->vocab + kSubElems - 1) / kSubElems;
  if ((int64_t)td * nsub > 0x7fffffff) return SPX_ERR_UNSUPPORTED;
  if (td > 0) {
    // the statistics pass of the sampling half, over the draft rows only
    SampleParams p{};
    p.batch = c->batch; p.total_q = td; p.total_d = 0; p.vocab = c->vocab; p.nsub = nsub;
    p.nseg = (c->vocab + kSegElems - 1) / kSegElems;
    p.row_stride = c->logits_row_stride;
    p.target = c->draft_logits; p.draft = c->draft_logits;
    p.seg_stats = static_cast<float2 *>(workspace);
    p.dev_status = dev_status;
    const spx_status_t ls = c->logits_dtype == SPX_BF16 ? launch_sampler_t<__nv_bfloat16, false>(p, stream, info.num_sms, kPhaseStats)
                                                        : launch_sampler_t<float, false>(p, stream, info.num_sms, kPhaseStats);
    if (ls != SPX_OK) return ls;
  }
  ConfParams q{};
  q.batch = c->batch; q.total_d = td; q.vocab = c->vocab; q.nsub = nsub; q.row_stride = c->logits_row_stride;
  q.draft = c->draft_logits; q.draft_ids = c->draft_token_ids; q.q_indptr = c->q_indptr;
  q.seg_stats = static_cast<const float2 *>(workspace);
  q.conf_max = c->conf_max; q.conf_tok = c->conf_tok; q.req_conf = c->req_conf; q.dev_status = dev_status;
  const int blocks = (c->batch * 32 + 127) / 128;
  if (c->logits_dtype == SPX_BF16) confidence_kernel<__nv_bfloat16><<<blocks, 128, 0, stream>>>(q);
  else confidence_kernel<float><<<blocks, 128, 0, stream>>>(q);
  ++t_launches;
  return cudaGetLastError() == cudaSuccess ? SPX_OK : SPX_ERR_CUDA;
}

spx_status_t spx_select_speculation(int32_t batch, const float *confidence, const int32_t *k_in, double alpha, int32_t *k_out,
                                    int32_t *n_drop, int32_t *dev_status, void *cuda_stream) {
  t_launches = 0;
  if (batch < 0 || !dev_status || !(alpha >= 0.0 && alpha <= 1.0)) return SPX_ERR_INVALID_ARG;
  if (batch == 0) return SPX_OK;
  if (!confidence || !k_in || !k_out) return SPX_ERR_INVALID_ARG;
  select_kernel<<<1, kSelThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(batch, confidence, k_in, alpha, k_out, n_drop,
                                                                               dev_status);
  ++t_launches;
  return cudaGetLastError() == cudaSuccess ? SPX_OK : SPX_ERR_CUDA;
}

// ---- the paper's scheduler numerics -----------------------------------------------------------
spx_status_t spx_lookahead_memory(int32_t nreq, const int32_t *ell, const int32_t *tau, const double *prec, int32_t pp,
                                  double theta, int32_t horizon, double *mem_estimate, void *cuda_stream) {
  t_launches = 0;
  if (nreq < 0 || pp < 1 || horizon < 1 || horizon > kLookMaxHorizon || !(theta >= 0.0 && theta <= 1.0) || !mem_estimate)
    return SPX_ERR_INVALID_ARG;
  if (nreq > 0 && (!ell || !tau || !prec)) return SPX_ERR_INVALID_ARG;
  lookahead_kernel<<<horizon, kLookThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(nreq, ell, tau, prec, pp, theta,
                                                                                         mem_estimate);
  ++t_launches;
  return cudaGetLastError() == cudaSuccess ? SPX_OK : SPX_ERR_CUDA;
}

double spx_sp_effective_batch(double batch, int32_t stages, double theta) {
  return batch / ((double)stages - theta * (double)(stages - 1));
}
double spx_selective_batch(double batch, int32_t stages, double alpha) { return batch / (1.0 + alpha * (double)(stages - 1)); }
double spx_selective_effective_batch(double batch, int32_t stages, double alpha, double theta_alpha) {
  const double ba = spx_selective_batch(batch, stages, alpha);
  return alpha * ba + (1.0 - alpha) * spx_sp_effective_batch(ba, stages, theta_alpha);
}
double spx_delay_gain(double iterations, int32_t n_evictions, double pdr, double running, double i_delay, const double *i_wait) {
  double waited = 0.0;
  for (int k = 0; k < n_evictions; ++k) waited += i_wait[k];
  const double recompute = (iterations + (double)(n_evictions + 1) * (pdr - 1.0)) / (iterations + pdr - 1.0);
  const double idle = (running + 1.0 - i_delay / iterations) / (running + 1.0 - waited / iterations);
  return recompute * idle;
}

// ---- LM head ------------------------------------------------------------------------------------
static bool make_matrix_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) return false;
  cuuint64_t dims[2] = {cols, rows}, strides[1] = {cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)kLmBK, box_rows}, estr[2] = {1, 1};
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

spx_status_t spx_lm_head(const spx_lm_head_args_t *a, int32_t *dev_status, void *cuda_stream) {
  t_launches = 0;
  if (!a || !dev_status) return SPX_ERR_INVALID_ARG;
  if (a->rows < 0 || a->hidden_dim <= 0 || a->vocab <= 0 || a->logits_row_stride < a->vocab) return SPX_ERR_INVALID_ARG;
  if (a->hidden_dim % 8 != 0 || a->logits_row_stride % 8 != 0) return SPX_ERR_UNSUPPORTED;
  if (a->rows == 0) return SPX_OK;
  if (!a->hidden || !a->weight || !a->logits) return SPX_ERR_INVALID_ARG;
  if (((uintptr_t)a->hidden | (uintptr_t)a->weight | (uintptr_t)a->logits) & 15) return SPX_ERR_INVALID_ARG;
  DeviceInfo info;
  if (!get_device_info(&info)) return SPX_ERR_CUDA;
  LmParams p{};
  p.M = a->rows; p.K = a->hidden_dim; p.V = a->vocab;
  // the rows are cut into equal token tiles of at most 512 (the TMEM columns); a tile of more than
  // 256 tokens is covered by two MMAs per k-step and has one accumulator instead of two in rotation
  p.tok_tiles = (a->rows + kLmMaxTileTok - 1) / kLmMaxTileTok;
  const int per_tile = (a->rows + p.tok_tiles - 1) / p.tok_tiles;
  p.n_sub = per_tile > kLmMaxNT ? 2 : 1;
  p.NT = ((per_tile + p.n_sub - 1) / p.n_sub + 31) / 32 * 32;
  p.tile_tok = p.n_sub * p.NT;
  p.n_buf = p.tile_tok <= kLmMaxNT ? 2 : 1;
  p.stage_bytes = (kLmABytes + p.n_sub * (p.NT / 2) * kLmBK * 2 + 1023) / 1024 * 1024;
  p.n_stages = kLmRingBytes / p.stage_bytes < kLmMaxStages ? kLmRingBytes / p.stage_bytes : kLmMaxStages;
  p.v_tiles = (a->vocab + 2 * kLmVB - 1) / (2 * kLmVB);
  p.k_blocks = (a->hidden_dim + kLmBK - 1) / kLmBK;
  p.stat_tiles = (a->vocab + kLmStatCols - 1) / kLmStatCols;
  p.logits = static_cast<__nv_bfloat16 *>(a->logits);
  p.row_stride = a->logits_row_stride;
  p.tile_stats = reinterpret_cast<float2 *>(a->tile_stats);
  p.dev_status = dev_status;
  CUtensorMap hmap, wmap;
  if (!make_matrix_map(&hmap, a->hidden, a->rows, a->hidden_dim, p.NT / 2) ||
      !make_matrix_map(&wmap, a->weight, a->vocab, a->hidden_dim, kLmVB))
    return SPX_ERR_CUDA;
  // the epilogue keeps a tile's rounded accumulator in registers: 6 chunks of 32 tokens per warp for
  // tiles of at most 384 tokens, 8 beyond
  auto kernel = p.tile_tok <= 384 ? lm_head_kernel<6> : lm_head_kernel<8>;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kLmSmemBytes) != cudaSuccess) return SPX_ERR_CUDA;
  // one resident CTA pair per two SMs of a GPC (a GPC with an odd SM count leaves one SM out)
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(info.num_sms / 2 * 2); cfg.blockDim = dim3(kLmThreads); cfg.dynamicSmemBytes = kLmSmemBytes;
  cfg.stream = static_cast<cudaStream_t>(cuda_stream);
  int max_pairs = 0;
  if (cudaOccupancyMaxActiveClusters(&max_pairs, kernel, &cfg) != cudaSuccess || max_pairs < 1) return SPX_ERR_CUDA;
  const long long tiles = (long long)p.v_tiles * p.tok_tiles;
  const int pairs = tiles < max_pairs ? (int)tiles : max_pairs;
  kernel<<<2 * pairs, kLmThreads, kLmSmemBytes, static_cast<cudaStream_t>(cuda_stream)>>>(hmap, wmap, p);
  ++t_launches;
  return cudaGetLastError() == cudaSuccess ? SPX_OK : SPX_ERR_CUDA;
}

// ---- sampling without caller-provided scratch ------------------------------------------------
// The scratch of the sampling kernels in a fixed device array that is part of the library image.
// In host code `g_static_scratch` is only a handle for the symbol, never an address a kernel could
// use: the device address is looked up once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[SPX_STATIC_SCRATCH_BYTES];

namespace {
std::mutex g_static_scratch_mutex;
void *g_static_scratch_addr[64] = {};  // device address of g_static_scratch, per device ordinal
}  // namespace

spx_status_t spx_rejection_sample_static(const spx_sample_args_t *args, int32_t *dev_status, void *cuda_stream) {
  t_launches = 0;
  spx_status_t st = check_sample(args, true);
  if (st != SPX_OK) return st;
  if (!dev_status) return SPX_ERR_INVALID_ARG;
  if (sample_ws_layout(args).total > SPX_STATIC_SCRATCH_BYTES) return SPX_ERR_WORKSPACE;  // beyond the fixed array
  DeviceInfo dev;
  if (!get_device_info(&dev) || dev.cc_major < 10) return SPX_ERR_CUDA;
  if (dev.device < 0 || dev.device >= 64) return SPX_ERR_UNSUPPORTED;
  void *scratch = nullptr;
  {
    // set-up, once per device, with that device current (it is: dev.device is the current device)
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (!g_static_scratch_addr[dev.device]) {
      void *addr = nullptr;
      if (cudaGetSymbolAddress(&addr, g_static_scratch) != cudaSuccess || !addr) return SPX_ERR_CUDA;
      g_static_scratch_addr[dev.device] = addr;
    }
    scratch = g_static_scratch_addr[dev.device];
  }
  return launch_sampler(args, static_cast<unsigned char *>(scratch), dev_status, static_cast<cudaStream_t>(cuda_stream),
                        dev.num_sms);
}

const char *spx_status_string(spx_status_t status) {
  switch (status) {
    case SPX_OK: return "ok";
    case SPX_ERR_INVALID_ARG: return "invalid argument";
    case SPX_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case SPX_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case SPX_ERR_CUDA: return "CUDA error (or no sm_100 device)";
  }
  return "unknown status";
}

void spx_set_timing_events(void *start_event, void *stop_event) {
  t_ev_start = static_cast<cudaEvent_t>(start_event);
  t_ev_stop = static_cast<cudaEvent_t>(stop_event);
}

int32_t spx_last_launch_count(void) { return t_launches; }

spx_status_t spx_debug_timeline(uint64_t *host_out, int64_t capacity, int32_t *kernels, int32_t *ctas_per_kernel) {
  if (kernels) *kernels = kTlKernels;
  if (ctas_per_kernel) *ctas_per_kernel = kTlCtas;
#if SPX_TIMELINE
  const int64_t need = (int64_t)kTlKernels * kTlCtas * 4;
  if (!host_out || capacity < need) return SPX_ERR_INVALID_ARG;
  return cudaMemcpyFromSymbol(host_out, g_timeline, (size_t)need * sizeof(uint64_t)) == cudaSuccess ? SPX_OK : SPX_ERR_CUDA;
#else
  (void)host_out; (void)capacity;
  return SPX_ERR_UNSUPPORTED;
#endif
}

spx_status_t spx_debug_wait_expiry(int32_t *report, int32_t *dev_status, void *cuda_stream) {
#if SPX_WAIT_TEST
  if (!report || !dev_status) return SPX_ERR_INVALID_ARG;
  wait_expiry_kernel<<<1, 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(report, dev_status);
  return cudaGetLastError() == cudaSuccess ? SPX_OK : SPX_ERR_CUDA;
#else
  (void)report; (void)dev_status; (void)cuda_stream;
  return SPX_ERR_UNSUPPORTED;
#endif
}

spx_status_t spx_plan_layout(const spx_attn_args_t *attn, int64_t *out) {
  if (!out) return SPX_ERR_INVALID_ARG;
  const spx_status_t st = check_attn(attn, false);
  if (st != SPX_OK) return st;
  const AttnWs w = attn_ws_layout(attn);
  out[0] = (int64_t)w.hdr; out[1] = (int64_t)w.cta_off; out[2] = (int64_t)w.work; out[3] = w.max_work;
  out[4] = (int64_t)w.nchunks; out[5] = (int64_t)w.part_base; out[6] = w.max_part_slots; out[7] = (int64_t)w.total;
  return SPX_OK;
}

#if SPX_PROFILE
// Profiling builds only (not declared in spx.h): per-CTA cycle counters of the attention kernel.
void spx_debug_set_profile_buffer(long long *device_buffer) { t_prof = device_buffer; }
#endif

}  // extern "C"
