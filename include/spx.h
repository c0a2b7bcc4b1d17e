/*
 * spx.h - C ABI of libspx: the speculative-decoding verify step on one NVIDIA B200 (sm_100a).
 *
 * The verify step is the per-iteration GPU work underneath speculative(-parallel) scheduling:
 * a batch of requests each carries k_r >= 0 draft tokens (k_r = 0 where selective speculation,
 * Section 5.1 of the paper, switched speculation off for that request); the target model's
 * k_r+1 new positions attend jointly over the request's paged, shared KV cache (Section 2
 * "Speculative decoding", Section 4 "Self-speculation and parallel scheduling": all drafts of a
 * request are checked in one pass, and speculative and normal execution use one cache), and the
 * drafts are then accepted or rejected by speculative sampling (the rule of the
 * speculative-decoding work cited in Section 2).
 *
 * Conventions for every entry point
 *   - Pointers inside the argument structs are DEVICE pointers unless the field name ends in
 *     _host.  The structs themselves, `ws_bytes` and all scalars live on the host.
 *   - The caller owns every buffer and the CUDA stream (`cuda_stream` is a cudaStream_t passed
 *     as void*; NULL = the legacy default stream).  The library allocates no device memory
 *     (spx_verify_step keeps one internal stream and three events per host thread and device).
 *   - Calls only enqueue work on the stream and return; nothing synchronises the device.
 *   - Host-visible argument errors return a non-zero spx_status_t and launch nothing.
 *   - Errors in device-resident data (a page id out of range, a draft token id >= vocab, a
 *     context shorter than its query count) cannot be seen by the host without a sync: they OR
 *     a SPX_DEV_* bit into *dev_status (a caller-owned int32 on the device, which the caller
 *     zeroes and reads back when it wants), the affected request gets sentinel outputs
 *     (attention rows zero, lse NaN; accepted_len 0 and out_tokens -1) and the other requests
 *     are unaffected.  No kernel traps, asserts or waits without bound.
 *   - `ws` is scratch of at least spx_workspace_size(...) bytes, 256-byte aligned.  Its
 *     contents are meaningless between calls.  Two calls may overlap on the device only if
 *     they use different workspaces.
 *   - bf16 means the upper half of an IEEE binary32 (round-to-nearest-even on output).
 */
#ifndef SPX_H_
#define SPX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPX_MAX_K 15            /* at most 15 draft tokens (16 query positions) per request   */
#define SPX_MAX_PACKED_ROWS 128 /* (num_q_heads / num_kv_heads) * (k+1) must not exceed this  */

typedef enum {
  SPX_OK = 0,
  SPX_ERR_INVALID_ARG = 1, /* NULL where a pointer is required, negative size, misalignment  */
  SPX_ERR_UNSUPPORTED = 2, /* shape outside what the kernels implement (see each call)        */
  SPX_ERR_WORKSPACE = 3,   /* ws is NULL, misaligned or smaller than spx_workspace_size       */
  SPX_ERR_CUDA = 4         /* a CUDA runtime/driver call failed (launch error, no sm_100 GPU) */
} spx_status_t;

/* Bits OR-ed into *dev_status by the kernels. */
enum {
  SPX_DEV_BAD_PAGE = 1,   /* a needed block-table entry was outside [0, num_pages)            */
  SPX_DEV_BAD_TOKEN = 2,  /* a draft token id was outside [0, vocab)                          */
  SPX_DEV_BAD_LEN = 4,    /* seq_len < k+1, k+1 outside [1, max_q_len], or too many pages     */
  SPX_DEV_TIMEOUT = 8,    /* a bounded wait inside a kernel gave up                           */
  SPX_DEV_DEGENERATE = 16,/* residual mass was zero; the target row was sampled instead       */
  SPX_DEV_BAD_PARAM = 32  /* a per-request temperature was negative, NaN or infinite          */
};

typedef enum { SPX_BF16 = 0, SPX_F32 = 1 } spx_dtype_t;

/*
 * Attention half.  For request r with m_r = q_indptr[r+1]-q_indptr[r] = k_r+1 query rows and
 * L_r = seq_lens[r] cached tokens (the m_r new positions INCLUDED, their K/V already written),
 * query j (0 <= j < m_r), q-head h, kv-head g = h / (num_q_heads/num_kv_heads):
 *     visible tokens t = 0 .. L_r - m_r + j            (causal among the new positions)
 *     s_t = sm_scale * <Q[q_indptr[r]+j, h, :], K[r, t, g, :]>
 *     out[q_indptr[r]+j, h, :] = sum_t softmax_t(s)_t * V[r, t, g, :]
 *     lse[q_indptr[r]+j, h]    = log sum_t exp(s_t)       (natural log)
 * Token t of request r lives in page block_table[r*max_pages_per_req + t/page_size], slot
 * t % page_size; element (page, g, slot, d) of a pool is at
 *     page*kv_stride_page + g*kv_stride_head + slot*kv_stride_token + d        (elements).
 * Slots past L_r and block-table entries past ceil(L_r/page_size) are never read.
 *
 * Supported: head_dim 64 or 128; num_q_heads a multiple of num_kv_heads with
 * (num_q_heads/num_kv_heads)*max_q_len <= SPX_MAX_PACKED_ROWS; page_size a power of two in
 * 1..128; kv_dtype BF16 (tensor-core path; pools and strides 16-byte aligned) or F32 (true fp32
 * arithmetic).  Accumulation is fp32 in both.
 */
typedef struct {
  int32_t batch;             /* B >= 0                                                        */
  int32_t total_q;           /* TQ = q_indptr[B] = rows of q/out (host copy of that number)   */
  int32_t max_q_len;         /* upper bound on k_r+1 over the batch, 1..SPX_MAX_K+1; 0 = 16   */
  int32_t num_q_heads, num_kv_heads, head_dim, page_size;
  int32_t num_pages;         /* pages in each pool                                            */
  int32_t max_pages_per_req; /* row length of block_table                                     */
  spx_dtype_t kv_dtype;      /* dtype of q, k_cache, v_cache and out                          */
  float sm_scale;            /* 0 => 1/sqrt(head_dim)                                         */
  const void *q;             /* [TQ, num_q_heads, head_dim] contiguous                        */
  const void *k_cache;       /* K pool                                                        */
  const void *v_cache;       /* V pool (same strides)                                         */
  int64_t kv_stride_page, kv_stride_head, kv_stride_token; /* elements; head_dim contiguous   */
  const int32_t *block_table; /* [B, max_pages_per_req]                                       */
  const int32_t *seq_lens;    /* [B]                                                          */
  const int32_t *q_indptr;    /* [B+1], q_indptr[0] = 0, non-decreasing                       */
  void *out;                  /* [TQ, num_q_heads, head_dim], written                         */
  float *lse;                 /* [TQ, num_q_heads], written; may be NULL                      */
} spx_attn_args_t;

/*
 * Sampling half.  Request r has target rows T_0..T_k (rows q_indptr[r] .. q_indptr[r]+k of
 * target_logits), draft rows D_0..D_{k-1} (rows q_indptr[r]-r .. of draft_logits), draft ids
 * x_i and uniforms a_i at the same indices as the draft rows, and one uniform s = u_sample[r].
 * With p_i = softmax(T_i), q_i = softmax(D_i) over the whole vocabulary at temperature 1:
 *   for i = 0..k-1 in order: accept x_i iff a_i < p_i(x_i)/q_i(x_i); stop at the first failure, n = i;
 *   if n < k : y = invCDF over r(v) = max(0, p_n(v) - q_n(v)), i.e. the first v (ascending id)
 *              whose inclusive cumulative sum exceeds s * sum_v r(v);
 *   if n = k : y = the same inverse CDF over p_k (the bonus token);
 *   accepted_len[r] = n; out_tokens[q_indptr[r] ..] = x_0..x_{n-1}, y, then -1 up to k+1 slots.
 * Logits rows after n are never needed.  Arithmetic: fp32 exponentials and in-segment sums,
 * float64 across segments and for the accept ratio.
 *
 * Verification variants (the paper fixes no sampling parameters; temperature == NULL is the
 * rule above).  temperature[r] = tau > 0: p_i = softmax(T_i / tau), q_i = softmax(D_i / tau) (the
 * draft was sampled at the request's temperature), everything else unchanged.  temperature[r] = 0:
 * greedy verification - x_i is accepted iff it is the lowest token id attaining the maximum of
 * T_i; y is that id for row n; no uniforms are read and diag_ratio stays NaN.  Any other value
 * sets SPX_DEV_BAD_PARAM and the request emits n = 0 and -1 tokens.  Requests of one batch may mix
 * all three.
 *
 * top_k / top_p (each NULL = off, else [B]) filter the target AND the draft rows of a request
 * before the rule is applied (the draft was sampled under the request's parameters):
 *   top_k[r] = K with 1 <= K < vocab: keep every token whose logit is >= the K-th largest logit of
 *     the row (tokens tying that value are all kept); other values switch it off;
 *   top_p[r] = P < 1, applied to the survivors' distribution softmax(x / tau): going down the
 *     distinct logit values, the first value at which the running mass reaches P is the last one
 *     kept; P = 1 switches it off; P outside (0, 1] sets SPX_DEV_BAD_PARAM like a bad temperature;
 *   p and q are softmax(x / tau) renormalised over the kept tokens and 0 elsewhere.  A drafted
 *   token with p(x) = 0 is rejected; one with q(x) = 0 < p(x) is accepted.
 * The top-p comparison is made on sums of fp32 exponentials (2^-44 fixed point, order
 * independent); it can differ from an exact evaluation when the running mass comes within about
 * 1e-6 of P.  Greedy requests ignore both filters.  The workspace is larger when temperature,
 * top_k or top_p is given: size it with the same pointers set.
 *
 * Supported: vocab >= 1; logits_row_stride >= vocab and a multiple of 8 (BF16) or 4 (F32)
 * elements; both logits pointers 16-byte aligned.
 */
typedef struct {
  int32_t batch;               /* B >= 0                                                      */
  int32_t total_q;             /* TQ = q_indptr[B]; draft rows TD = TQ - B                    */
  int32_t vocab;
  int64_t logits_row_stride;   /* elements, same for target and draft                         */
  spx_dtype_t logits_dtype;
  const void *target_logits;   /* [TQ, vocab]                                                 */
  const void *draft_logits;    /* [TD, vocab]; may be NULL when TD = 0                        */
  const int32_t *draft_token_ids; /* [TD]                                                     */
  const int32_t *q_indptr;     /* [B+1]                                                       */
  const float *u_accept;       /* [TD], each in [0,1)                                         */
  const float *u_sample;       /* [B], each in [0,1)                                          */
  int32_t *accepted_len;       /* [B], written                                                */
  int32_t *out_tokens;         /* [TQ], written                                               */
  float *diag_ratio;           /* optional [TD]: p/q of each consulted draft (NaN otherwise)  */
  const float *temperature;    /* optional [B]: see "Verification variants"; NULL = all 1     */
  const int32_t *top_k;        /* optional [B]                                                */
  const float *top_p;          /* optional [B]                                                */
  const float *target_tile_stats; /* optional: spx_lm_head's tile_stats of the target rows    */
} spx_sample_args_t;

/*
 * Bytes of scratch the calls below need for these arguments (host integers only are read;
 * either pointer may be NULL to size one half alone).  Returns 0 on invalid arguments.
 */
size_t spx_workspace_size(const spx_attn_args_t *attn, const spx_sample_args_t *sample);

/* The attention half alone (see spx_attn_args_t). */
spx_status_t spx_verify_attention(const spx_attn_args_t *args, void *ws, size_t ws_bytes,
                                  int32_t *dev_status, void *cuda_stream);

/* The sampling half alone (see spx_sample_args_t). */
spx_status_t spx_rejection_sample(const spx_sample_args_t *args, void *ws, size_t ws_bytes,
                                  int32_t *dev_status, void *cuda_stream);

/*
 * The whole verify step.  The halves are independent given their inputs (logits are inputs
 * here), so the sampling half is forked onto a library-internal stream and joined back into
 * `cuda_stream` before the call returns: work enqueued on `cuda_stream` afterwards sees both
 * halves' outputs.  With top_k / top_p the attention kernel additionally waits (one event) for
 * the thresholds, whose kernels do not share an SM with it.  The internal stream and its three
 * events are created on the first call of a host thread on a device and are kept until the
 * process ends.  If a launch fails after the
 * fork, the internal stream is still joined back before the error is returned.  `ws` must hold
 * spx_workspace_size(attn, sample) bytes.
 */
spx_status_t spx_verify_step(const spx_attn_args_t *attn, const spx_sample_args_t *sample, void *ws,
                             size_t ws_bytes, int32_t *dev_status, void *cuda_stream);

/*
 * Cache maintenance around the step (the paper's Section 4: speculative execution shares the
 * paged cache with normal execution; its Figure 3: accepted speculation continues, rejected
 * speculation is re-executed).
 *
 * spx_kv_append writes the K/V of every request's k_r+1 new positions into their pages BEFORE
 * attention: row q_indptr[r]+j of new_k/new_v ([TQ, num_kv_heads, head_dim], contiguous, same
 * dtype as the pools) goes to logical token L_r-(k_r+1)+j of request r, i.e. page
 * block_table[r][t/page_size], slot t%page_size (seq_lens already counts the new positions).
 * Values are copied bit for bit; no other slot is touched.  Requests with an invalid length or
 * page id set SPX_DEV_BAD_LEN / SPX_DEV_BAD_PAGE and are skipped.  Pools and strides as in
 * spx_attn_args_t; head_dim * element size must be a multiple of 16 bytes.
 *
 * Optional rotary embedding on the way (the paper does not discuss positional encoding; this is
 * the rotation of the Llama and Qwen families it evaluates): with rope_base > 0 every new K row is
 * rotated to its absolute position t before it is stored - for each head vector x and i < D/2,
 * with a = t * rope_base^(-2i/D):  y[i] = x[i] cos a - x[i+D/2] sin a,  y[i+D/2] = x[i+D/2] cos a +
 * x[i] sin a, computed in float64 and rounded float64 -> binary32 -> kv_dtype (nearest-even each).
 * V is copied as it is.  If q_rows is given ([TQ, num_q_heads, head_dim], kv_dtype, 16-byte
 * aligned), row q_indptr[r]+j is rotated IN PLACE to the same position, so that the attention that
 * follows sees rotated Q and K.  rope_base = 0: no rotation, q_rows ignored.  Needs head_dim/2 *
 * element size to be a multiple of 16 bytes and head_dim <= 512 (SPX_ERR_UNSUPPORTED otherwise); a negative, NaN or
 * infinite rope_base is SPX_ERR_INVALID_ARG.
 *
 * spx_kv_rollback computes, AFTER sampling, the lengths that drop the rejected drafts:
 * new_seq_lens[r] = seq_lens[r] - (k_r - accepted_len[r]) (position 0 and the accepted drafts
 * stay; the emitted token is the next step's position 0 and is not cached yet).  An accepted
 * length outside [0, k_r] sets SPX_DEV_BAD_LEN and writes -1.  new_seq_lens may alias seq_lens.
 */
typedef struct {
  int32_t batch, total_q;
  int32_t num_kv_heads, head_dim, page_size, num_pages, max_pages_per_req;
  spx_dtype_t kv_dtype;
  const void *new_k, *new_v;          /* [TQ, num_kv_heads, head_dim]                         */
  void *k_cache, *v_cache;            /* pools, written                                       */
  int64_t kv_stride_page, kv_stride_head, kv_stride_token;
  const int32_t *block_table;         /* [B, max_pages_per_req]                               */
  const int32_t *seq_lens;            /* [B], counts the new positions                        */
  const int32_t *q_indptr;            /* [B+1]                                                */
  float rope_base;                    /* 0: plain copy; > 0: rotary base (e.g. 10000, 500000) */
  int32_t num_q_heads;                /* heads of q_rows (ignored when q_rows is NULL)        */
  void *q_rows;                       /* optional, rotated in place; NULL: none               */
} spx_kv_append_args_t;

spx_status_t spx_kv_append(const spx_kv_append_args_t *args, int32_t *dev_status, void *cuda_stream);
spx_status_t spx_kv_rollback(int32_t batch, const int32_t *seq_lens, const int32_t *q_indptr,
                             const int32_t *accepted_len, int32_t *new_seq_lens, int32_t *dev_status,
                             void *cuda_stream);

/*
 * Selective speculation support (the paper's Section 5.1: drafted tokens are ranked by the
 * draft's confidence and a fixed fraction alpha of the lowest-ranked is not speculated on;
 * Section 7.4 applies it per sequence).  The paper does not define the confidence further; this
 * library takes the draft's top-1 probability.
 *
 * spx_draft_confidence: for every draft row d (indexed as in the sampling half: request r owns
 * rows q_indptr[r]-r .. +k_r-1 of draft_logits) at temperature 1
 *   conf_max[d] = max_v softmax(D_d)(v);  conf_tok[d] = softmax(D_d)(x_d)  (optional, needs ids);
 *   req_conf[r] = product of conf_max over the request's drafts (1 when k_r = 0).
 * fp32 results of float64 merges of fp32 partial sums (relative error of order 1e-6).  Workspace
 * from spx_draft_confidence_workspace (0 = invalid arguments), 256-byte aligned, caller-owned.
 * An id outside [0, vocab) sets SPX_DEV_BAD_TOKEN and conf_tok = NaN for that draft.
 *
 * spx_select_speculation: among the requests with k_in[r] > 0 (N of them) the
 * floor(alpha * N) with the lowest confidence get k_out[r] = 0, the others k_out[r] = k_in[r].
 * Order: the IEEE total order on the stored fp32 confidences (bit patterns; -0 < +0, NaNs at the
 * ends by sign); among equal confidences the higher index is dropped first.  Integer-exact.
 * alpha outside [0, 1] is SPX_ERR_INVALID_ARG; a negative k_in sets SPX_DEV_BAD_LEN and counts as
 * 0.  n_drop (device, optional) receives floor(alpha * N).  k_out may alias k_in.  One thread
 * block: meant for batches up to a few 10^4 requests.
 */
typedef struct {
  int32_t batch, total_q;            /* total_q = q_indptr[B]; draft rows TD = total_q - B      */
  int32_t vocab;
  int64_t logits_row_stride;         /* elements                                                */
  spx_dtype_t logits_dtype;
  const void *draft_logits;          /* [TD, vocab], 16-byte aligned                            */
  const int32_t *draft_token_ids;    /* [TD]; may be NULL when conf_tok is NULL                 */
  const int32_t *q_indptr;           /* [B+1]                                                   */
  float *conf_max;                   /* [TD], written                                           */
  float *conf_tok;                   /* [TD], written; optional                                 */
  float *req_conf;                   /* [B], written                                            */
} spx_conf_args_t;

size_t spx_draft_confidence_workspace(const spx_conf_args_t *args);
spx_status_t spx_draft_confidence(const spx_conf_args_t *args, void *workspace, size_t workspace_bytes,
                                  int32_t *dev_status, void *cuda_stream);
spx_status_t spx_select_speculation(int32_t batch, const float *confidence, const int32_t *k_in, double alpha,
                                    int32_t *k_out, int32_t *n_drop, int32_t *dev_status, void *cuda_stream);

/*
 * The paper's scheduler numerics.
 *
 * spx_lookahead_memory is its Algorithm 1, the estimate of the batch's cache occupancy over the
 * coming iterations: for i = 1..horizon (the paper uses 64), with pipeline depth pp and speculation
 * accuracy theta, w counting a request's rejected speculations,
 *   t = i - pp w,  k = t + w,  p = C(k, t) theta^t (1 - theta)^w,  w = 0..floor(i / pp),
 *   E[L_gen] = sum_w k p,   P_fin(r) = prec[r] * sum_w [k >= tau[r]] p,
 *   M[i-1] = sum_r ell[r] + (nreq - sum_r P_fin(r)) E[L_gen] - sum_r ell[r] P_fin(r),
 * where ell[r] is the request's current length, tau[r] its predicted remaining length and
 * prec[r] the precision of that prediction (the caller evaluates the predictor's precision
 * table).  All device pointers; float64 arithmetic; 0^0 = 1.  Supported: 1 <= horizon <= 256,
 * pp >= 1, theta in [0, 1]; otherwise SPX_ERR_INVALID_ARG.
 *
 * The closed forms run on the host (they are scalar): Eq. 2 (steady-state effective batch of
 * speculative-parallel execution, B / (N - theta (N - 1))), Eq. 3's limit (steady-state batch
 * under drop ratio alpha, B / (1 + alpha (N - 1))), Eq. 4 (effective batch under selective
 * speculation), and the gain G of delayed over aggressive admission (Section 5.2).
 */
spx_status_t spx_lookahead_memory(int32_t nreq, const int32_t *ell, const int32_t *tau, const double *prec, int32_t pp,
                                  double theta, int32_t horizon, double *mem_estimate, void *cuda_stream);
double spx_sp_effective_batch(double batch, int32_t stages, double theta);
double spx_selective_batch(double batch, int32_t stages, double alpha);
double spx_selective_effective_batch(double batch, int32_t stages, double alpha, double theta_alpha);
double spx_delay_gain(double iterations, int32_t n_evictions, double pdr, double running, double i_delay,
                      const double *i_wait /* host, [n_evictions] */);

/*
 * LM head with the sampling half's statistics fused into its epilogue (the paper's Section 6
 * keeps an LM head on the stage that verifies; the step's target logits are its output):
 *   logits[m][v] = sum_k hidden[m][k] * weight[v][k],  m < rows, v < vocab,
 * bf16 operands, fp32 accumulation on the tensor cores, result rounded to bf16 (nearest even) and
 * stored at logits[m * logits_row_stride + v].  hidden is [rows, hidden_dim] and weight is
 * [vocab, hidden_dim], both row-major and dense; all device pointers, 16-byte aligned;
 * hidden_dim and logits_row_stride multiples of 8.  tile_stats (optional) receives, for every row
 * and every block of 128 vocabulary columns, (max * log2 e, sum_v 2^((x_v - max) log2 e)) of the
 * values AS STORED: [rows][ceil(vocab / 128)] pairs of floats.  Passed as
 * spx_sample_args_t.target_tile_stats they replace the sampling half's own read of the target
 * logits for its statistics (temperature 1, no filters; ignored otherwise).
 * Errors: SPX_ERR_INVALID_ARG / SPX_ERR_UNSUPPORTED for bad shapes or alignment; a bounded wait
 * that expires inside the kernel sets SPX_DEV_TIMEOUT.
 */
typedef struct {
  int32_t rows, hidden_dim, vocab;
  const void *hidden;          /* [rows, hidden_dim] bf16                                      */
  const void *weight;          /* [vocab, hidden_dim] bf16                                     */
  void *logits;                /* [rows, logits_row_stride] bf16, written                      */
  int64_t logits_row_stride;   /* elements                                                     */
  float *tile_stats;           /* optional [rows][ceil(vocab/128)][2], written                 */
} spx_lm_head_args_t;

spx_status_t spx_lm_head(const spx_lm_head_args_t *args, int32_t *dev_status, void *cuda_stream);

/*
 * Convenience for callers whose data lives on the HOST: every pointer in the two structs is a
 * host pointer (pinned memory recommended); device staging buffers, the workspace and the
 * status word are carved from `dev_arena` (device memory, `arena_bytes` >=
 * spx_host_step_arena_size).  Copies inputs host->device, runs spx_verify_step, copies
 * out/lse/accepted_len/out_tokens and the status word back, all on `cuda_stream`, and returns
 * after enqueueing; *dev_status_host is valid after the stream is synchronised.  `kv_pool_elems`
 * is the number of elements of each KV pool to copy.
 */
size_t spx_host_step_arena_size(const spx_attn_args_t *attn, const spx_sample_args_t *sample,
                                int64_t kv_pool_elems);
spx_status_t spx_verify_step_host(const spx_attn_args_t *attn, const spx_sample_args_t *sample,
                                  int64_t kv_pool_elems, void *dev_arena, size_t arena_bytes,
                                  int32_t *dev_status_host, void *cuda_stream);

/*
 * spx_rejection_sample for callers that cannot provide scratch memory.  (The paper has no
 * counterpart: this entry point exists for integration reasons only.)
 *
 * Some callers can neither call cudaMalloc nor hand the library a workspace: code running inside a
 * CUDA-graph capture or a stream-ordered region where an allocation would synchronise or be
 * refused, runtimes whose allocator owns all device memory and offers no hook, and plugins that
 * receive only their input and output tensors.  For them the sampling half is offered with its
 * scratch in a fixed array that is part of the library image: SPX_STATIC_SCRATCH_BYTES of device
 * memory, held by every GPU that loads the library until the process exits.
 *
 * Same arguments, outputs and arithmetic as spx_rejection_sample (bit-identical results); the
 * caller still passes every input and output buffer and the status word.  Differences:
 *   - If spx_workspace_size(NULL, args) exceeds SPX_STATIC_SCRATCH_BYTES the call returns
 *     SPX_ERR_WORKSPACE and launches nothing (e.g. 704 logits rows of 128256 tokens need 0.4 MB;
 *     the limit is reached near 8000 such rows).
 *   - The first call on each device looks up the array's device address (no allocation).  Make
 *     that first call outside any stream capture.
 *   - Every call on a device shares the one array, which keeps the previous call's contents.
 *     Nothing in it has to start at zero from the caller's point of view: the only counters are
 *     cleared by the call itself before they are read.  Two calls that overlap on the same device
 *     (different streams, or different host threads) race on it: serialise them.
 *   - It calls no cudaMalloc, cudaFree or any other allocating routine.
 */
#define SPX_STATIC_SCRATCH_BYTES (4u << 20)
spx_status_t spx_rejection_sample_static(const spx_sample_args_t *args, int32_t *dev_status, void *cuda_stream);

const char *spx_status_string(spx_status_t status);

/*
 * Measurement aid.  While a pair of cudaEvent_t (created by the caller with timing enabled) is
 * set on the calling thread, every spx_verify_attention / spx_verify_step call from that thread
 * records `start` immediately before and `stop` immediately after its verify-attention kernel
 * (the kernel that streams the KV cache) on the call's stream.  Pass NULL, NULL to clear.
 */
void spx_set_timing_events(void *start_event, void *stop_event);

/* Number of kernels the last call on this thread enqueued (for launch accounting). */
int32_t spx_last_launch_count(void);

/*
 * Inspection aid: where, inside the workspace of spx_verify_attention / spx_verify_step, the
 * attention work plan lies after a call with these arguments (the attention part comes first in
 * the workspace of spx_verify_step).  The plan cuts the 128-token tiles of all (request, kv head)
 * pairs, in (request, head) order, into one contiguous range per CTA of the persistent attention
 * kernel.  Writes byte offsets and sizes into out[0..7] (host memory):
 *   out[0] header: int32 n_work, n_cta, n_part_slots, total_tiles, (cursor), overflow, n_combine
 *   out[1] cta_off: int32[n_cta + 1], entries of the work list that belong to the CTAs before c
 *   out[2] work list: 32-byte entries of int32 {req, tile_begin, tile_end, part_slot (-1: the pair
 *          is not split), q0, m, L, kv_head}
 *   out[3] capacity of the work list (entries)
 *   out[4] pair_nchunks: int32[batch * num_kv_heads], chunks of each pair (0: invalid request)
 *   out[5] pair_part_base: int32[batch * num_kv_heads], first partial slot of a split pair, else -1
 *   out[6] capacity in partial slots
 *   out[7] bytes of the attention part of the workspace
 * Returns SPX_ERR_INVALID_ARG / SPX_ERR_UNSUPPORTED as spx_workspace_size would refuse the
 * arguments.  Used by the tests to check the plan's invariants; nothing else depends on it.
 */
spx_status_t spx_plan_layout(const spx_attn_args_t *attn, int64_t *out);

/*
 * Measurement aid of timeline builds of the library (compiled with -DSPX_TIMELINE=1; the regular
 * build returns SPX_ERR_UNSUPPORTED): every kernel of the step stamps the GPU's global
 * nanosecond timer per CTA at entry and exit.  Copies the stamps of the most recent launches to
 * host_out (host memory, uint64 [kernels][ctas_per_kernel][4] = {start ns, end ns, SM id, 0};
 * kernel index: 0 plan, 1 attention, 2 combine, 3 logits statistics, 4 accept, 5 residual masses,
 * 6 residual draw).  capacity is in uint64 elements; the two dimensions are always written to
 * *kernels / *ctas_per_kernel (either may be NULL).  Synchronises the device.
 */
spx_status_t spx_debug_timeline(uint64_t *host_out, int64_t capacity, int32_t *kernels, int32_t *ctas_per_kernel);

/*
 * Test aid of wait-test builds of the library (compiled with -DSPX_WAIT_TEST=1 and a small
 * -DSPX_WAIT_LIMIT_CYCLES; the regular build returns SPX_ERR_UNSUPPORTED).  Every spin on a
 * barrier in the library's kernels has a cycle limit, after which the waiting role raises
 * SPX_DEV_TIMEOUT in *dev_status, sets its CTA's abort flag and returns, so that a lost signal ends
 * in an error status and not in a hung device.  This call launches one block of four warps in
 * which the three wait helpers (attention, logits ring, LM head) each wait on a barrier nothing
 * arrives at.  report (device, int32 [11]): [0..3] 2 = the role's wait gave up (1 would mean it
 * was satisfied); [4..7] cycles each role waited; [8..10] the three abort flags afterwards.
 * Role 1 shares its abort flag with role 0 and leaves through it or through its own limit.
 * Enqueues only; nothing faults, the context stays usable.
 */
spx_status_t spx_debug_wait_expiry(int32_t *report, int32_t *dev_status, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SPX_H_ */
