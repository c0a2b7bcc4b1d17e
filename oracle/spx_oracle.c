/*
 * CPU oracle for the speculative-decoding verify step.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is a plain, slow, float64 restatement of what the verify step computes.  It is
 * used by the tests, by the smoke check and by the benchmark's CPU-baseline leg, and by
 * nothing else: the CUDA library never links, loads or calls it, and it shares no code,
 * header, table or helper with the CUDA path.
 *
 * What it follows.  The paper (Section 2, "Speculative decoding"; Section 4,
 * "Self-speculation and parallel scheduling") states only that a draft proposes several
 * tokens and the base model verifies them jointly against one shared, paged KV cache; it
 * prints no formula for either half.  The two halves are therefore written out from their
 * standard definitions:
 *
 *   (A) attention  - textbook scaled-dot-product attention with a causal mask among the
 *       k+1 new positions, keys and values addressed through a block table (paged cache);
 *   (B) speculative sampling - the rule of the speculative-decoding work the paper cites in
 *       Section 2: accept draft x_i with probability min(1, p_i(x_i)/q_i(x_i)); at the
 *       first rejection draw from the normalised residual max(0, p - q); if every draft is
 *       accepted draw one bonus token from the target distribution.
 *
 * Every input value (bf16 or fp32) is widened exactly to double; all arithmetic is double.
 * There is no tiling, no online softmax, no fusion: two plain passes per softmax and a
 * sequential cumulative sum for the inverse CDF, so that each loop can be checked against
 * the definition by eye.  OpenMP is used only across independent (request, position, head)
 * or row items; it never changes the order of any floating-point sum.
 *
 * Pins (tests/test_oracle_*.py): brute-force numpy float64 attention on tiny inputs,
 * weights-sum-to-one, causal and page-placement invariance, closed forms (K = 0 gives the
 * mean of V and LSE = log n; one token gives V[0]), a needle key, GQA head duplication; for
 * sampling a chi-square test of the output law against the target distribution on a
 * 16-token vocabulary, the identity min(p,q) + (1-beta) r/R = p, closed-form acceptance
 * rates, special cases, and interval-arithmetic brute force on tiny vocabularies; for the
 * cache maintenance (tests/test_oracle_kv.py) torch's indexed scatter on the un-paged view,
 * bit-identity of every untouched slot, append-then-attend against attending a cache that was
 * filled directly, and the closed form of the rolled-back lengths; for the verification
 * variants (tests/test_oracle_variants.py; the paper fixes no sampling parameters, so these are
 * this build's reading: the same temperature divides target and draft logits, temperature 0
 * verifies greedily) the output law against softmax(target / tau), the closed form
 * tau*ln(w) -> w / sum w, exact invariance under doubling logits and temperature together,
 * numpy's argmax on rows with ties, and the tau -> 0 limit meeting the greedy branch; for top-k /
 * top-p filtering (tests/test_oracle_filters.py) a numpy restatement by argsort, unique and
 * cumulative sums, hand-worked rows (0.5, 0.3, 0.15, 0.05), the limits that switch a filter off,
 * ties kept together, and the output law of speculative sampling under filtering; for the
 * selective-speculation support (tests/test_oracle_select.py; Section 5.1) scipy's softmax
 * maxima, the closed forms 1/V and w_max / sum w, numpy's lexsort on (confidence, -index),
 * and the invariants of a keep-top-(1-alpha) selection (count, separation, alpha = 0 and 1);
 * for the scheduler numerics (tests/test_oracle_model.py; Eq. 1-4, Section 5.2, Algorithm 1,
 * Appendix A.1-A.3) conservation s^a + s^r + n = B, the recurrences' limits against the closed
 * forms, G against throughput ratios built from the token counts and times of Appendix A.3, and
 * Algorithm 1 against scipy's binomial pmf, its closed forms at pp = 1 and theta = 1, and a
 * Python brute force; for the LM head (tests/test_oracle_lm_head.py) torch's float64 matmul,
 * identity / one-hot weights, linearity, and integer inputs whose products are exact.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_BF16 = 0, ORACLE_F32 = 1 };

enum {
  ORACLE_OK = 0,
  ORACLE_ERR_ARG = 1,      /* bad scalar argument                                   */
  ORACLE_ERR_LEN = 2,      /* some L_r < k_r + 1                                     */
  ORACLE_ERR_PAGE = 3,     /* a needed block-table entry is outside [0, num_pages)   */
  ORACLE_ERR_TOKEN = 4,    /* a draft token id is outside [0, V)                     */
  ORACLE_ERR_ALLOC = 5,
  ORACLE_ERR_PARAM = 6     /* a per-request sampling parameter is not a temperature  */
};

/* Bit flags written per request by the sampler. */
enum { ORACLE_FLAG_DEGENERATE = 1 /* residual mass R == 0, target row used instead */ };

static inline double widen(const void *base, int dtype, int64_t idx) {
  if (dtype == ORACLE_F32) return (double)((const float *)base)[idx];
  /* bf16 is the upper 16 bits of an IEEE binary32 */
  uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
  float f;
  memcpy(&f, &bits, sizeof f);
  return (double)f;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------------------------ */
/* (A) attention                                                                         */
/* ------------------------------------------------------------------------------------ */

/*
 * For request r with k_r = q_indptr[r+1]-q_indptr[r]-1 drafts and L_r = seq_lens[r] cached
 * tokens (the k_r+1 new positions included), query j in [0,k_r], q-head h, kv-head
 * g = h / (Hq/Hkv), pos = L_r-(k_r+1)+j:
 *
 *   s_t   = scale * sum_d Q[qi,h,d] K[t,g,d]         t = 0..pos
 *   w_t   = exp(s_t - max_t s_t) / sum_t exp(s_t - max)
 *   O     = sum_t w_t V[t,g,:]
 *   LSE   = max + log sum_t exp(s_t - max)
 *
 * Token t of request r lives in page block_table[r][t / P], slot t % P; element
 * (page, g, slot, d) of a pool is at page*stride_page + g*stride_head + slot*stride_token + d.
 *
 * req_list (may be NULL) restricts the computation to the listed requests; rows of other
 * requests in out/lse are left untouched.  out is [TQ,Hq,D] double, lse [TQ,Hq] double
 * (lse may be NULL).
 */
int oracle_verify_attention(int32_t batch, int32_t Hq, int32_t Hkv, int32_t D, int32_t P,
                            int64_t num_pages, int32_t max_pages_per_req, int32_t dtype,
                            double sm_scale, const void *q, const void *k_cache,
                            const void *v_cache, int64_t stride_page, int64_t stride_head,
                            int64_t stride_token, const int32_t *block_table,
                            const int32_t *seq_lens, const int32_t *q_indptr,
                            const int32_t *req_list, int32_t n_req_list, double *out,
                            double *lse) {
  if (batch < 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || D <= 0 || P <= 0) return ORACLE_ERR_ARG;
  if (dtype != ORACLE_BF16 && dtype != ORACLE_F32) return ORACLE_ERR_ARG;
  const int G = Hq / Hkv;
  const double scale = (sm_scale == 0.0) ? 1.0 / sqrt((double)D) : sm_scale;
  const int n_req = req_list ? n_req_list : batch;

  /* validate first, so that the parallel part below has no early exits */
  for (int ri = 0; ri < n_req; ++ri) {
    const int r = req_list ? req_list[ri] : ri;
    if (r < 0 || r >= batch) return ORACLE_ERR_ARG;
    const int m = q_indptr[r + 1] - q_indptr[r];
    const int L = seq_lens[r];
    if (m < 1 || L < m) return ORACLE_ERR_LEN;
    const int n_pages = (L + P - 1) / P;
    if (n_pages > max_pages_per_req) return ORACLE_ERR_PAGE;
    for (int pg = 0; pg < n_pages; ++pg) {
      const int32_t phys = block_table[(int64_t)r * max_pages_per_req + pg];
      if (phys < 0 || phys >= num_pages) return ORACLE_ERR_PAGE;
    }
  }

  /* flatten (request, position, head) so that OpenMP can balance ragged lengths */
  int64_t n_items = 0;
  for (int ri = 0; ri < n_req; ++ri) {
    const int r = req_list ? req_list[ri] : ri;
    n_items += (int64_t)(q_indptr[r + 1] - q_indptr[r]) * Hq;
  }
  int32_t *item_r = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_items > 0 ? n_items : 1));
  int32_t *item_j = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_items > 0 ? n_items : 1));
  int32_t *item_h = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_items > 0 ? n_items : 1));
  if (!item_r || !item_j || !item_h) { free(item_r); free(item_j); free(item_h); return ORACLE_ERR_ALLOC; }
  {
    int64_t it = 0;
    for (int ri = 0; ri < n_req; ++ri) {
      const int r = req_list ? req_list[ri] : ri;
      const int m = q_indptr[r + 1] - q_indptr[r];
      for (int j = 0; j < m; ++j)
        for (int h = 0; h < Hq; ++h) { item_r[it] = r; item_j[it] = j; item_h[it] = h; ++it; }
    }
  }

  int alloc_failed = 0;
#pragma omp parallel
  {
    double *s = NULL;
    int64_t s_cap = 0;
    double *qrow = (double *)malloc(sizeof(double) * (size_t)D);
    double *acc = (double *)malloc(sizeof(double) * (size_t)D);
    if (!qrow || !acc) {
#pragma omp atomic write
      alloc_failed = 1;
    }
#pragma omp for schedule(dynamic, 1)
    for (int64_t it = 0; it < n_items; ++it) {
      if (alloc_failed) continue;
      const int r = item_r[it], j = item_j[it], h = item_h[it];
      const int g = h / G;
      const int m = q_indptr[r + 1] - q_indptr[r];
      const int L = seq_lens[r];
      const int pos = L - m + j;               /* last visible token index */
      const int64_t qi = (int64_t)q_indptr[r] + j;
      const int32_t *bt = block_table + (int64_t)r * max_pages_per_req;
      if (pos + 1 > s_cap) {
        free(s);
        s_cap = pos + 1;
        s = (double *)malloc(sizeof(double) * (size_t)s_cap);
        if (!s) {
#pragma omp atomic write
          alloc_failed = 1;
          s_cap = 0;
          continue;
        }
      }
      for (int d = 0; d < D; ++d) qrow[d] = widen(q, dtype, (qi * Hq + h) * D + d);

      /* pass 1: scores and their maximum */
      double mx = -INFINITY;
      for (int t = 0; t <= pos; ++t) {
        const int64_t base = (int64_t)bt[t / P] * stride_page + (int64_t)g * stride_head +
                             (int64_t)(t % P) * stride_token;
        double dot = 0.0;
        for (int d = 0; d < D; ++d) dot += qrow[d] * widen(k_cache, dtype, base + d);
        s[t] = scale * dot;
        if (s[t] > mx) mx = s[t];
      }
      /* pass 2: normaliser */
      double denom = 0.0;
      for (int t = 0; t <= pos; ++t) denom += exp(s[t] - mx);
      /* weighted sum of values */
      for (int d = 0; d < D; ++d) acc[d] = 0.0;
      for (int t = 0; t <= pos; ++t) {
        const double w = exp(s[t] - mx) / denom;
        const int64_t base = (int64_t)bt[t / P] * stride_page + (int64_t)g * stride_head +
                             (int64_t)(t % P) * stride_token;
        for (int d = 0; d < D; ++d) acc[d] += w * widen(v_cache, dtype, base + d);
      }
      for (int d = 0; d < D; ++d) out[(qi * Hq + h) * D + d] = acc[d];
      if (lse) lse[qi * Hq + h] = mx + log(denom);
    }
    free(s); free(qrow); free(acc);
  }
  free(item_r); free(item_j); free(item_h);
  return alloc_failed ? ORACLE_ERR_ALLOC : ORACLE_OK;
}

/* ------------------------------------------------------------------------------------ */
/* (B) speculative rejection sampling                                                    */
/* ------------------------------------------------------------------------------------ */

/*
 * Step 1: p = softmax(row / tau) over the full vocabulary, max subtracted:
 * p(v) = exp((x_v - max) / tau) / sum_w exp((x_w - max) / tau), tau > 0.  The paper does not fix
 * the sampling temperature; tau = 1 is the base case (the division is then exact).
 */
void oracle_softmax_row_tau(const void *logits, int32_t dtype, int64_t row_offset, int64_t V,
                            double tau, double *p) {
  double mx = -INFINITY;
  for (int64_t v = 0; v < V; ++v) {
    const double x = widen(logits, dtype, row_offset + v);
    if (x > mx) mx = x;
  }
  double denom = 0.0;
  for (int64_t v = 0; v < V; ++v) {
    p[v] = exp((widen(logits, dtype, row_offset + v) - mx) / tau);
    denom += p[v];
  }
  for (int64_t v = 0; v < V; ++v) p[v] /= denom;
}

void oracle_softmax_row(const void *logits, int32_t dtype, int64_t row_offset, int64_t V,
                        double *p) {
  oracle_softmax_row_tau(logits, dtype, row_offset, V, 1.0, p);
}

/* Greedy choice of a row: the lowest token id that attains the row maximum. */
int64_t oracle_argmax_row(const void *logits, int32_t dtype, int64_t row_offset, int64_t V) {
  int64_t best = 0;
  double mx = widen(logits, dtype, row_offset);
  for (int64_t v = 1; v < V; ++v) {
    const double x = widen(logits, dtype, row_offset + v);
    if (x > mx) { mx = x; best = v; }
  }
  return best;
}

static int cmp_desc(const void *a, const void *b) {
  const double x = *(const double *)a, y = *(const double *)b;
  return (x < y) - (x > y);
}

/*
 * Step 1 with top-k / top-p filtering (the paper fixes no sampling parameters; this is the usual
 * serving rule, stated on values so that it does not depend on how ties are ordered):
 *   top-k (1 <= top_k < V): keep every token whose logit is >= the top_k-th largest logit of the
 *     row (tokens tying that value are all kept);
 *   top-p (top_p < 1), applied to the survivors' distribution pi = softmax(x / tau) restricted to
 *     them: walk the distinct logit values downwards, adding the mass of each value's group; the
 *     first value at which the running mass reaches top_p is the last one kept;
 *   p = softmax(x / tau) renormalised over the kept tokens, 0 elsewhere.
 * sorted is scratch for V doubles.  *margin (may be NULL) receives how far, in units of the
 * survivors' mass, the top-p crossing was from tipping to a neighbouring value (+inf when top-p is
 * off): the decision is a floating-point comparison and an fp32 evaluation may legitimately differ
 * when this is tiny.  Returns the number of kept tokens.
 */
int64_t oracle_filtered_row(const void *logits, int32_t dtype, int64_t row_offset, int64_t V,
                            double tau, int32_t top_k, double top_p, double *p, double *sorted,
                            double *margin) {
  for (int64_t v = 0; v < V; ++v) sorted[v] = widen(logits, dtype, row_offset + v);
  qsort(sorted, (size_t)V, sizeof(double), cmp_desc);
  const double mx = sorted[0];
  double thr = -INFINITY;
  if (top_k >= 1 && (int64_t)top_k < V) thr = sorted[top_k - 1];
  if (margin) *margin = INFINITY;
  if (top_p < 1.0) {
    /* survivors' mass, group by group in descending order (the same order as the walk below) */
    double Zk = 0.0;
    for (int64_t j = 0; j < V && sorted[j] >= thr;) {
      int64_t g = j;
      double gm = 0.0;
      while (g < V && sorted[g] == sorted[j]) { gm += exp((sorted[g] - mx) / tau); ++g; }
      Zk += gm;
      j = g;
    }
    double cum = 0.0;
    for (int64_t j = 0; j < V && sorted[j] >= thr;) {
      int64_t g = j;
      double gm = 0.0;
      while (g < V && sorted[g] == sorted[j]) { gm += exp((sorted[g] - mx) / tau); ++g; }
      const double before = cum;
      cum += gm;
      if (cum >= top_p * Zk) {
        thr = sorted[j];
        if (margin) {
          const double over = (cum - top_p * Zk) / Zk, under = (top_p * Zk - before) / Zk;
          *margin = over < under ? over : under;
        }
        break;
      }
      j = g;
    }
  }
  double Z = 0.0;
  int64_t kept = 0;
  for (int64_t v = 0; v < V; ++v) {
    const double x = widen(logits, dtype, row_offset + v);
    if (x >= thr) { p[v] = exp((x - mx) / tau); Z += p[v]; ++kept; }
    else p[v] = 0.0;
  }
  for (int64_t v = 0; v < V; ++v) p[v] /= Z;
  return kept;
}

/* The distribution of one row under a request's sampling parameters. */
typedef struct { double tau; int32_t top_k; double top_p; double *sorted; double margin; } row_params_t;

static void row_dist(const void *logits, int32_t dtype, int64_t row_offset, int64_t V,
                     row_params_t *rp, double *p) {
  const int filtered = (rp->top_k >= 1 && (int64_t)rp->top_k < V) || rp->top_p < 1.0;
  if (!filtered) { oracle_softmax_row_tau(logits, dtype, row_offset, V, rp->tau, p); return; }
  double m;
  oracle_filtered_row(logits, dtype, row_offset, V, rp->tau, rp->top_k, rp->top_p, p, rp->sorted, &m);
  if (m < rp->margin) rp->margin = m;
}

/* Step 3 (first half): r(v) = max(0, p(v) - q(v)); returns R = sum_v r(v), ascending v. */
double oracle_residual(const double *p, const double *q, int64_t V, double *r) {
  double R = 0.0;
  for (int64_t v = 0; v < V; ++v) {
    const double d = p[v] - q[v];
    r[v] = d > 0.0 ? d : 0.0;
    R += r[v];
  }
  return R;
}

/*
 * Steps 3/4 (second half): y = min{ v : sum_{w<=v} r(w) > s*R }.  If rounding leaves no such
 * v, y is the largest v with r(v) > 0.  Bins of zero width are never selected because the
 * inequality is strict and the cumulative sum does not move across them.  cdf_lo/cdf_hi (may
 * be NULL) receive the exclusive/inclusive cumulative sums at y.  Returns -1 only if every
 * r(v) is zero.
 */
int64_t oracle_inverse_cdf(const double *r, int64_t V, double R, double s, double *cdf_lo,
                           double *cdf_hi) {
  const double target = s * R;
  double cum = 0.0;
  int64_t last_pos = -1;
  double last_lo = 0.0, last_hi = 0.0;
  for (int64_t v = 0; v < V; ++v) {
    const double before = cum;
    cum += r[v];
    if (r[v] > 0.0) { last_pos = v; last_lo = before; last_hi = cum; }
    if (cum > target) {
      if (cdf_lo) *cdf_lo = before;
      if (cdf_hi) *cdf_hi = cum;
      return v;
    }
  }
  if (cdf_lo) *cdf_lo = last_lo;
  if (cdf_hi) *cdf_hi = last_hi;
  return last_pos;
}

/* Inclusive cumulative sum of r, ascending v, written to cdf[0..V).  For near-tie accounting. */
void oracle_cumsum(const double *r, int64_t V, double *cdf) {
  double cum = 0.0;
  for (int64_t v = 0; v < V; ++v) { cum += r[v]; cdf[v] = cum; }
}

/*
 * One request.  T_i = target row q_indptr[r]+i (i = 0..k), D_i = draft row q_indptr[r]-r+i
 * (i = 0..k-1), x_i = draft_ids[q_indptr[r]-r+i], a_i = u_accept[same], s = u_sample[r].
 * Scratch p, q, res each hold V doubles.
 */
static int sample_one(int r, int32_t dtype, int64_t V, int64_t row_stride,
                      const void *target_logits, const void *draft_logits,
                      const int32_t *draft_ids, const int32_t *q_indptr, const float *u_accept,
                      const float *u_sample, int32_t *accepted_len, int32_t *out_tokens,
                      double *rho_out, double *resid_mass, double *cdf_lo, double *cdf_hi,
                      int32_t *flags, double *p, double *q, double *res, row_params_t *rp) {
  const double tau = rp->tau;
  const int filtered = (rp->top_k >= 1 && (int64_t)rp->top_k < V) || rp->top_p < 1.0;
  const int64_t t0 = q_indptr[r];          /* first target row / first output slot */
  const int64_t d0 = (int64_t)q_indptr[r] - r; /* first draft row */
  const int k = q_indptr[r + 1] - q_indptr[r] - 1;
  int n = k;
  int bad_token = 0;
  if (flags) flags[r] = 0;
  for (int i = 0; i < k && !bad_token; ++i)
    if (draft_ids[d0 + i] < 0 || draft_ids[d0 + i] >= V) bad_token = 1;
  if (bad_token) {
    accepted_len[r] = 0;
    for (int i = 0; i <= k; ++i) out_tokens[t0 + i] = -1;
    if (rho_out) for (int i = 0; i < k; ++i) rho_out[d0 + i] = NAN;
    if (resid_mass) resid_mass[r] = NAN;
    if (cdf_lo) cdf_lo[r] = NAN;
    if (cdf_hi) cdf_hi[r] = NAN;
    return ORACLE_ERR_TOKEN;
  }
  if (rho_out) for (int i = 0; i < k; ++i) rho_out[d0 + i] = NAN; /* rows after n: not consulted */

  if (!(tau >= 0.0) || isinf(tau) || !(rp->top_p > 0.0 && rp->top_p <= 1.0)) {
    /* not a temperature, or not a nucleus mass: the request emits nothing */
    accepted_len[r] = 0;
    for (int i = 0; i <= k; ++i) out_tokens[t0 + i] = -1;
    if (resid_mass) resid_mass[r] = NAN;
    if (cdf_lo) cdf_lo[r] = NAN;
    if (cdf_hi) cdf_hi[r] = NAN;
    return ORACLE_ERR_PARAM;
  }
  if (tau == 0.0) {
    /* Greedy verification, the tau -> 0 limit with a greedy draft: draft i is accepted iff it is
     * the target's greedy choice at position i; the first mismatch is replaced by that choice;
     * with no mismatch the bonus token is the greedy choice of row k.  No uniforms are used. */
    for (int i = 0; i < k; ++i)
      if (draft_ids[d0 + i] != oracle_argmax_row(target_logits, dtype, (t0 + i) * row_stride, V)) { n = i; break; }
    accepted_len[r] = n;
    for (int i = 0; i < n; ++i) out_tokens[t0 + i] = draft_ids[d0 + i];
    out_tokens[t0 + n] = (int32_t)oracle_argmax_row(target_logits, dtype, (t0 + n) * row_stride, V);
    for (int i = n + 1; i <= k; ++i) out_tokens[t0 + i] = -1;
    if (resid_mass) resid_mass[r] = NAN;
    if (cdf_lo) cdf_lo[r] = NAN;
    if (cdf_hi) cdf_hi[r] = NAN;
    return ORACLE_OK;
  }

  /* step 2: sequential accept tests */
  for (int i = 0; i < k; ++i) {
    const int64_t x = draft_ids[d0 + i];
    row_dist(target_logits, dtype, (t0 + i) * row_stride, V, rp, p);
    row_dist(draft_logits, dtype, (d0 + i) * row_stride, V, rp, q);
    /* with filtering a draft token can have target probability 0: it is rejected whatever q says */
    const double rho = (filtered && p[x] == 0.0) ? 0.0 : ((q[x] == 0.0) ? INFINITY : p[x] / q[x]);
    if (rho_out) rho_out[d0 + i] = rho;
    if (!((double)u_accept[d0 + i] < rho)) { n = i; break; }
  }

  double R, lo = 0.0, hi = 0.0;
  int64_t y;
  if (n < k) {
    /* step 3: p, q still hold rows n */
    R = oracle_residual(p, q, V, res);
    if (R == 0.0) {
      if (flags) flags[r] |= ORACLE_FLAG_DEGENERATE;
      R = 0.0;
      for (int64_t v = 0; v < V; ++v) { res[v] = p[v]; R += p[v]; }
    }
    y = oracle_inverse_cdf(res, V, R, (double)u_sample[r], &lo, &hi);
  } else {
    /* step 4: bonus token from target row k */
    row_dist(target_logits, dtype, (t0 + k) * row_stride, V, rp, p);
    R = 0.0;
    for (int64_t v = 0; v < V; ++v) R += p[v];
    y = oracle_inverse_cdf(p, V, R, (double)u_sample[r], &lo, &hi);
  }

  /* step 5 */
  accepted_len[r] = n;
  for (int i = 0; i < n; ++i) out_tokens[t0 + i] = draft_ids[d0 + i];
  out_tokens[t0 + n] = (int32_t)y;
  for (int i = n + 1; i <= k; ++i) out_tokens[t0 + i] = -1;
  if (resid_mass) resid_mass[r] = R;
  if (cdf_lo) cdf_lo[r] = lo;
  if (cdf_hi) cdf_hi[r] = hi;
  return ORACLE_OK;
}

/*
 * Whole batch.  Outputs accepted_len [B], out_tokens [TQ]; optional diagnostics: rho [TD]
 * (p/q per consulted draft, NaN for drafts after the first rejection), resid_mass [B] (the R
 * used), cdf_lo/cdf_hi [B] (cumulative sums bracketing the emitted token), flags [B].
 * Returns ORACLE_ERR_TOKEN if some request carried an invalid draft id (that request emits
 * n = 0 and -1 tokens; the others are unaffected).
 *
 * temperature (NULL, or [B]) selects the verification variant per request: tau_r > 0 verifies
 * against softmax(target / tau_r) with the draft distribution softmax(draft / tau_r) (the draft
 * was sampled at the request's temperature); tau_r = 0 is greedy verification; anything else
 * (negative, NaN, infinite) makes that request emit n = 0 and -1 tokens and the call return
 * ORACLE_ERR_PARAM.  NULL means tau = 1 everywhere.
 *
 * top_k (NULL, or [B] int32; values < 1 or >= V switch it off) and top_p (NULL, or [B] float;
 * 1 switches it off, values outside (0, 1] are ORACLE_ERR_PARAM like a bad temperature) filter
 * both the target and the draft rows of the request as oracle_filtered_row states (the draft was
 * sampled under the request's parameters); greedy requests ignore them.  margin_out (NULL, or
 * [B]) receives the smallest top-p decision margin over the rows the request consulted.
 */
int oracle_rejection_sample_filtered(int32_t batch, int64_t V, int64_t row_stride, int32_t dtype,
                                     const void *target_logits, const void *draft_logits,
                                     const int32_t *draft_ids, const int32_t *q_indptr,
                                     const float *u_accept, const float *u_sample,
                                     const float *temperature, const int32_t *top_k,
                                     const float *top_p, int32_t *accepted_len,
                                     int32_t *out_tokens, double *rho_out, double *resid_mass,
                                     double *cdf_lo, double *cdf_hi, int32_t *flags,
                                     double *margin_out) {
  if (batch < 0 || V <= 0 || row_stride < V) return ORACLE_ERR_ARG;
  if (dtype != ORACLE_BF16 && dtype != ORACLE_F32) return ORACLE_ERR_ARG;
  for (int r = 0; r < batch; ++r)
    if (q_indptr[r + 1] - q_indptr[r] < 1) return ORACLE_ERR_ARG;
  int status = ORACLE_OK;
#pragma omp parallel
  {
    double *p = (double *)malloc(sizeof(double) * (size_t)V);
    double *q = (double *)malloc(sizeof(double) * (size_t)V);
    double *res = (double *)malloc(sizeof(double) * (size_t)V);
    double *sorted = (double *)malloc(sizeof(double) * (size_t)V);
    if (!p || !q || !res || !sorted) {
#pragma omp atomic write
      status = ORACLE_ERR_ALLOC;
    }
#pragma omp for schedule(dynamic, 1)
    for (int r = 0; r < batch; ++r) {
      if (!p || !q || !res || !sorted) continue;
      row_params_t rp;
      rp.tau = temperature ? (double)temperature[r] : 1.0;
      rp.top_k = top_k ? top_k[r] : 0;
      rp.top_p = top_p ? (double)top_p[r] : 1.0;
      rp.sorted = sorted;
      rp.margin = INFINITY;
      const int st = sample_one(r, dtype, V, row_stride, target_logits, draft_logits, draft_ids,
                                q_indptr, u_accept, u_sample, accepted_len, out_tokens, rho_out,
                                resid_mass, cdf_lo, cdf_hi, flags, p, q, res, &rp);
      if (margin_out) margin_out[r] = rp.margin;
      if (st != ORACLE_OK) {
#pragma omp atomic write
        status = st;
      }
    }
    free(p); free(q); free(res); free(sorted);
  }
  return status;
}

int oracle_rejection_sample_tau(int32_t batch, int64_t V, int64_t row_stride, int32_t dtype,
                                const void *target_logits, const void *draft_logits,
                                const int32_t *draft_ids, const int32_t *q_indptr,
                                const float *u_accept, const float *u_sample,
                                const float *temperature, int32_t *accepted_len,
                                int32_t *out_tokens, double *rho_out, double *resid_mass,
                                double *cdf_lo, double *cdf_hi, int32_t *flags) {
  return oracle_rejection_sample_filtered(batch, V, row_stride, dtype, target_logits, draft_logits,
                                          draft_ids, q_indptr, u_accept, u_sample, temperature, NULL,
                                          NULL, accepted_len, out_tokens, rho_out, resid_mass, cdf_lo,
                                          cdf_hi, flags, NULL);
}

int oracle_rejection_sample(int32_t batch, int64_t V, int64_t row_stride, int32_t dtype,
                            const void *target_logits, const void *draft_logits,
                            const int32_t *draft_ids, const int32_t *q_indptr,
                            const float *u_accept, const float *u_sample,
                            int32_t *accepted_len, int32_t *out_tokens, double *rho_out,
                            double *resid_mass, double *cdf_lo, double *cdf_hi, int32_t *flags) {
  return oracle_rejection_sample_tau(batch, V, row_stride, dtype, target_logits, draft_logits,
                                     draft_ids, q_indptr, u_accept, u_sample, NULL, accepted_len,
                                     out_tokens, rho_out, resid_mass, cdf_lo, cdf_hi, flags);
}

/*
 * The distribution the emitted token of request r was drawn from, as the oracle computed it:
 * cdf[0..V) = inclusive cumulative sum of the residual at row n (n < k) or of the target
 * row k (n == k).  n is passed in (the oracle's accepted_len[r]).  Returns R.
 */
double oracle_emit_cdf_filtered(int32_t r, int32_t n, int64_t V, int64_t row_stride, int32_t dtype,
                                const void *target_logits, const void *draft_logits,
                                const int32_t *q_indptr, double tau, int32_t top_k, double top_p,
                                double *cdf) {
  const int64_t t0 = q_indptr[r];
  const int64_t d0 = (int64_t)q_indptr[r] - r;
  const int k = q_indptr[r + 1] - q_indptr[r] - 1;
  double *p = (double *)malloc(sizeof(double) * (size_t)V);
  double *q = (double *)malloc(sizeof(double) * (size_t)V);
  double *sorted = (double *)malloc(sizeof(double) * (size_t)V);
  double R = NAN;
  if (p && q && sorted) {
    row_params_t rp = {tau, top_k, top_p, sorted, INFINITY};
    row_dist(target_logits, dtype, (t0 + n) * row_stride, V, &rp, p);
    if (n < k) {
      row_dist(draft_logits, dtype, (d0 + n) * row_stride, V, &rp, q);
      R = oracle_residual(p, q, V, q);
      if (R == 0.0) { R = 0.0; for (int64_t v = 0; v < V; ++v) { q[v] = p[v]; R += p[v]; } }
      oracle_cumsum(q, V, cdf);
    } else {
      R = 0.0;
      for (int64_t v = 0; v < V; ++v) R += p[v];
      oracle_cumsum(p, V, cdf);
    }
  }
  free(p); free(q); free(sorted);
  return R;
}

double oracle_emit_cdf_tau(int32_t r, int32_t n, int64_t V, int64_t row_stride, int32_t dtype,
                           const void *target_logits, const void *draft_logits,
                           const int32_t *q_indptr, double tau, double *cdf) {
  return oracle_emit_cdf_filtered(r, n, V, row_stride, dtype, target_logits, draft_logits, q_indptr,
                                  tau, 0, 1.0, cdf);
}

double oracle_emit_cdf(int32_t r, int32_t n, int64_t V, int64_t row_stride, int32_t dtype,
                       const void *target_logits, const void *draft_logits,
                       const int32_t *q_indptr, double *cdf) {
  return oracle_emit_cdf_tau(r, n, V, row_stride, dtype, target_logits, draft_logits, q_indptr, 1.0, cdf);
}

/* ------------------------------------------------------------------------------------ */
/* (E) selective speculation: draft confidence and the keep-top-(1-alpha) selection       */
/* ------------------------------------------------------------------------------------ */

/*
 * Section 5.1 orders drafted tokens by how confident the draft is in them and stops speculating
 * on a fixed share alpha at the bottom of that order; Section 7.4 applies the same rule to whole
 * sequences of a batch.  The paper does not
 * define the confidence beyond citing the self-speculation works that use the draft's top
 * probability, so this build reads it as:
 *   conf_max[d]  = max_v softmax(D_d)(v)              (the draft's top-1 probability)
 *   conf_tok[d]  = softmax(D_d)(x_d)                  (probability of the drafted token)
 *   req_conf[r]  = prod_i conf_max[d0(r) + i]         (1 for k_r = 0; with one draft per
 *                                                      sequence every reading coincides)
 * Draft rows and ids are indexed as in the sampling half (row q_indptr[r] - r + i).
 * conf_tok may be NULL; an id outside [0, V) gives conf_tok = NaN and ORACLE_ERR_TOKEN.
 */
int oracle_draft_confidence(int32_t batch, int64_t V, int64_t row_stride, int32_t dtype,
                            const void *draft_logits, const int32_t *draft_ids,
                            const int32_t *q_indptr, double *conf_max, double *conf_tok,
                            double *req_conf) {
  if (batch < 0 || V <= 0 || row_stride < V) return ORACLE_ERR_ARG;
  if (dtype != ORACLE_BF16 && dtype != ORACLE_F32) return ORACLE_ERR_ARG;
  int status = ORACLE_OK;
  double *q = (double *)malloc(sizeof(double) * (size_t)V);
  if (!q) return ORACLE_ERR_ALLOC;
  for (int r = 0; r < batch; ++r) {
    const int64_t d0 = (int64_t)q_indptr[r] - r;
    const int k = q_indptr[r + 1] - q_indptr[r] - 1;
    if (k < 0) { free(q); return ORACLE_ERR_ARG; }
    double prod = 1.0;
    for (int i = 0; i < k; ++i) {
      oracle_softmax_row(draft_logits, dtype, (d0 + i) * row_stride, V, q);
      double mx = 0.0;
      for (int64_t v = 0; v < V; ++v) if (q[v] > mx) mx = q[v];
      conf_max[d0 + i] = mx;
      prod *= mx;
      if (conf_tok) {
        const int64_t x = draft_ids[d0 + i];
        if (x < 0 || x >= V) { conf_tok[d0 + i] = NAN; status = ORACLE_ERR_TOKEN; }
        else conf_tok[d0 + i] = q[x];
      }
    }
    req_conf[r] = prod;
  }
  free(q);
  return status;
}

/* Total order on fp32 bit patterns (-NaN < -inf < ... < -0 < +0 < ... < +inf < +NaN). */
static uint32_t f32_order_key(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

/*
 * Selection.  Among the requests that carry drafts (k_in[r] > 0; N of them) drop the
 * n_drop = floor(alpha * N) with the lowest confidence; a dropped request continues without
 * speculation (k_out = 0), the others keep k_out = k_in.  Order: the total order above on the
 * stored fp32 confidences; among equal confidences the higher request index is dropped first.
 * alpha outside [0, 1] (or NaN) is an argument error.  Returns n_drop through *n_drop_out.
 * Written as the definition: repeatedly remove the lowest remaining participant.
 */
int oracle_select_speculation(int32_t batch, const float *confidence, const int32_t *k_in,
                              double alpha, int32_t *k_out, int32_t *n_drop_out) {
  if (batch < 0 || !(alpha >= 0.0 && alpha <= 1.0)) return ORACLE_ERR_ARG;
  int64_t N = 0;
  for (int r = 0; r < batch; ++r) {
    if (k_in[r] < 0) return ORACLE_ERR_ARG;
    k_out[r] = k_in[r];
    if (k_in[r] > 0) ++N;
  }
  const int64_t n_drop = (int64_t)floor(alpha * (double)N);
  for (int64_t d = 0; d < n_drop; ++d) {
    int worst = -1;
    for (int r = 0; r < batch; ++r) {
      if (k_out[r] == 0) continue;   /* not a participant, or dropped already */
      if (worst < 0) { worst = r; continue; }
      /* r > worst here (ascending scan), so an equal confidence moves the choice to the higher index */
      if (f32_order_key(confidence[r]) <= f32_order_key(confidence[worst])) worst = r;
    }
    k_out[worst] = 0;
  }
  if (n_drop_out) *n_drop_out = (int32_t)n_drop;
  return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------ */
/* (F) the paper's scheduler numerics: Eq. 1-4, the gain G, Algorithm 1                   */
/* ------------------------------------------------------------------------------------ */

/*
 * Eq. 1 with the initial conditions of Appendix A.1 (s^a_0 = s^r_0 = 0, n_0 = B, everything 0
 * for t < 0), iterated for t = 0..T.  sa, sr, n each hold T+1 doubles.
 *   s^a_t = (s^a_{t-1} + n_{t-1}) Theta
 *   s^r_t = sum_{i=1}^{N-1} (s^a_{t-i} + n_{t-i}) (1 - Theta)
 *   n_t   = (s^a_{t-N} + n_{t-N}) (1 - Theta)
 */
int oracle_sp_recurrence(double B, int32_t N, double theta, int32_t T, double *sa, double *sr,
                         double *n) {
  if (N < 1 || T < 0 || !(theta >= 0.0 && theta <= 1.0)) return ORACLE_ERR_ARG;
  for (int t = 0; t <= T; ++t) {
    if (t == 0) { sa[0] = 0.0; sr[0] = 0.0; n[0] = B; continue; }
    sa[t] = (sa[t - 1] + n[t - 1]) * theta;
    double rej = 0.0;
    for (int i = 1; i <= N - 1; ++i)
      if (t - i >= 0) rej += (sa[t - i] + n[t - i]) * (1.0 - theta);
    sr[t] = rej;
    n[t] = (t - N >= 0) ? (sa[t - N] + n[t - N]) * (1.0 - theta) : 0.0;
  }
  return ORACLE_OK;
}

/* Eq. 2: steady-state effective batch of speculative-parallel execution. */
double oracle_sp_effective_batch(double B, int32_t N, double theta) {
  return B / ((double)N - theta * (double)(N - 1));
}

/*
 * Eq. 3 with the initial conditions of Appendix A.2 (B_i = B (1-alpha)^i for 0 <= i <= N-1):
 * B_{t+1} = alpha B_{t+1-N} + (1-alpha) B_t, for t+1 = N..T.  Bt holds T+1 doubles.
 */
int oracle_alpha_recurrence(double B, int32_t N, double alpha, int32_t T, double *Bt) {
  if (N < 1 || T < 0 || !(alpha >= 0.0 && alpha < 1.0)) return ORACLE_ERR_ARG;
  for (int t = 0; t <= T; ++t) {
    if (t <= N - 1) Bt[t] = B * pow(1.0 - alpha, (double)t);
    else Bt[t] = alpha * Bt[t - N] + (1.0 - alpha) * Bt[t - 1];
  }
  return ORACLE_OK;
}

/* Eq. 3, limit: steady-state batch under drop ratio alpha. */
double oracle_alpha_batch(double B, int32_t N, double alpha) {
  return B / (1.0 + alpha * (double)(N - 1));
}

/* Eq. 4: expected effective batch under selective speculation. */
double oracle_alpha_effective_batch(double B, int32_t N, double alpha, double theta_alpha) {
  const double Ba = oracle_alpha_batch(B, N, alpha);
  return alpha * Ba + (1.0 - alpha) * Ba / ((double)N - theta_alpha * (double)(N - 1));
}

/*
 * Section 5.2, gain of delayed over aggressive admission:
 * G = (I + (n+1)(pdr-1)) / (I + pdr - 1) * (bs + 1 - i_delay/I) / (bs + 1 - sum_k i_wait^k / I).
 */
double oracle_delay_gain(double I, int32_t n, double pdr, double bs, double i_delay,
                         const double *i_wait) {
  double wait = 0.0;
  for (int k = 0; k < n; ++k) wait += i_wait[k];
  const double left = (I + (double)(n + 1) * (pdr - 1.0)) / (I + pdr - 1.0);
  const double right = (bs + 1.0 - i_delay / I) / (bs + 1.0 - wait / I);
  return left * right;
}

/*
 * Algorithm 1: expected KV-cache occupancy (in tokens) of the running batch after each of the next
 * `horizon` iterations (the paper looks 64 ahead).  Inputs per request r: its present length
 * ell[r], the predicted number of tokens it still has to produce tau[r], and prec[r], how often a
 * prediction of that size is right (the caller looks that up).  pp is the pipeline depth, theta
 * the probability that a speculation is accepted.
 *
 * What the algorithm states, in this file's words.  After `step` iterations a request has had
 * some number `rej` of rejected speculations, each of which cost it pp iterations; the other
 * acc = step - pp*rej iterations each produced an accepted token, and every rejection still
 * produced one (corrected) token, so it has made acc + rej tokens.  The rejections can fall
 * anywhere among those tokens: Pr[rej] = C(acc + rej, rej) theta^acc (1-theta)^rej, for
 * rej = 0 .. floor(step / pp), with 0^0 = 1.  From that law:
 *   grown       = sum_rej made(rej) Pr[rej]                    expected tokens made per request
 *   done(r)     = prec[r] * sum_{rej : made(rej) >= tau[r]} Pr[rej]   probability r has finished
 *   estimate    = sum_r ell[r] + (nreq - sum_r done(r)) * grown - sum_r ell[r] done(r).
 * law_of_rejections() tabulates (made, Pr) once per step; the requests are a separate pass.
 */
static int law_of_rejections(int step, int pp, double theta, int *made, double *pr) {
  const int most = step / pp;
  for (int rej = 0; rej <= most; ++rej) {
    const int acc = step - pp * rej;
    double ways = 1.0;                           /* C(acc + rej, rej) as a running product */
    for (int j = 1; j <= rej; ++j) ways = ways * (double)(acc + j) / (double)j;
    made[rej] = acc + rej;
    pr[rej] = ways * pow(theta, (double)acc) * pow(1.0 - theta, (double)rej);
  }
  return most + 1;
}

int oracle_lookahead_memory(int32_t nreq, const int32_t *ell, const int32_t *tau,
                            const double *prec, int32_t pp, double theta, int32_t horizon,
                            double *M) {
  if (nreq < 0 || pp < 1 || horizon < 0 || !(theta >= 0.0 && theta <= 1.0)) return ORACLE_ERR_ARG;
  int *made = (int *)malloc(sizeof(int) * (size_t)(horizon + 2));
  double *pr = (double *)malloc(sizeof(double) * (size_t)(horizon + 2));
  if (!made || !pr) { free(made); free(pr); return ORACLE_ERR_ARG; }
  double held = 0.0;
  for (int r = 0; r < nreq; ++r) held += (double)ell[r];
  for (int step = 1; step <= horizon; ++step) {
    const int cases = law_of_rejections(step, pp, theta, made, pr);
    double grown = 0.0;
    for (int c = 0; c < cases; ++c) grown += (double)made[c] * pr[c];
    double finished = 0.0, released = 0.0;
    for (int r = 0; r < nreq; ++r) {
      double reached = 0.0;
      for (int c = 0; c < cases; ++c)
        if (made[c] >= tau[r]) reached += pr[c];
      const double done = prec[r] * reached;
      finished += done;
      released += (double)ell[r] * done;
    }
    M[step - 1] = held + ((double)nreq - finished) * grown - released;
  }
  free(made);
  free(pr);
  return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------ */
/* (G) LM head: the logits the sampling half consumes                                    */
/* ------------------------------------------------------------------------------------ */

/*
 * logits[m][v] = sum_k H[m][k] W[v][k] for the M new positions' final hidden states H [M, K] and
 * the vocabulary projection W [V, K], both stored row-major in `dtype`; float64 products and a
 * plain left-to-right sum over k.  (Section 6 places the LM head on the stage that verifies; the
 * paper gives no formula beyond that: this is the definition of a linear layer without bias.)
 * Only the columns [v_begin, v_end) are computed (a full-size check samples column blocks);
 * out is [M][v_end - v_begin] doubles.
 */
int oracle_lm_head(int32_t M, int32_t K, int64_t V, int32_t dtype, const void *H, const void *W,
                   int64_t v_begin, int64_t v_end, double *out) {
  if (M < 0 || K <= 0 || V <= 0 || v_begin < 0 || v_end > V || v_begin > v_end) return ORACLE_ERR_ARG;
  if (dtype != ORACLE_BF16 && dtype != ORACLE_F32) return ORACLE_ERR_ARG;
  const int64_t nv = v_end - v_begin;
#pragma omp parallel for collapse(2) schedule(static)
  for (int m = 0; m < M; ++m)
    for (int64_t v = 0; v < nv; ++v) {
      double acc = 0.0;
      for (int k = 0; k < K; ++k)
        acc += widen(H, dtype, (int64_t)m * K + k) * widen(W, dtype, (v_begin + v) * K + k);
      out[(int64_t)m * nv + v] = acc;
    }
  return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------ */
/* (D) cache maintenance around the step                                                 */
/* ------------------------------------------------------------------------------------ */

/*
 * Append: the K/V of request r's m_r = k_r+1 new positions (rows q_indptr[r].. of new_k/new_v,
 * laid out [TQ, Hkv, D]) are written at logical tokens L_r-m_r .. L_r-1 of the request, i.e.
 * page block_table[r][t/P], slot t%P.  L_r already counts the new positions.  This is the shared
 * cache of Section 4 ("speculative execution ... shares the cache with normal execution"): the
 * drafts' entries go into the same pages as everything else, nothing is duplicated.
 * elem_size is 2 (bf16) or 4 (fp32); the values are copied bit for bit.
 */
int oracle_kv_append(int32_t batch, int32_t Hkv, int32_t D, int32_t P, int64_t num_pages,
                     int32_t max_pages_per_req, int32_t elem_size, const void *new_k,
                     const void *new_v, void *k_cache, void *v_cache, int64_t stride_page,
                     int64_t stride_head, int64_t stride_token, const int32_t *block_table,
                     const int32_t *seq_lens, const int32_t *q_indptr) {
  if (batch < 0 || Hkv <= 0 || D <= 0 || P <= 0 || (elem_size != 2 && elem_size != 4)) return ORACLE_ERR_ARG;
  for (int r = 0; r < batch; ++r) {
    const int m = q_indptr[r + 1] - q_indptr[r];
    const int L = seq_lens[r];
    if (m < 1 || L < m) return ORACLE_ERR_LEN;
    if ((L + P - 1) / P > max_pages_per_req) return ORACLE_ERR_PAGE;
    for (int j = 0; j < m; ++j) {
      const int t = L - m + j;
      const int32_t phys = block_table[(int64_t)r * max_pages_per_req + t / P];
      if (phys < 0 || phys >= num_pages) return ORACLE_ERR_PAGE;
    }
  }
  for (int r = 0; r < batch; ++r) {
    const int m = q_indptr[r + 1] - q_indptr[r];
    const int L = seq_lens[r];
    for (int j = 0; j < m; ++j) {
      const int t = L - m + j;
      const int64_t page = block_table[(int64_t)r * max_pages_per_req + t / P];
      for (int g = 0; g < Hkv; ++g) {
        const int64_t dst = page * stride_page + (int64_t)g * stride_head + (int64_t)(t % P) * stride_token;
        const int64_t src = (((int64_t)q_indptr[r] + j) * Hkv + g) * D;
        memcpy((char *)k_cache + dst * elem_size, (const char *)new_k + src * elem_size, (size_t)D * elem_size);
        memcpy((char *)v_cache + dst * elem_size, (const char *)new_v + src * elem_size, (size_t)D * elem_size);
      }
    }
  }
  return ORACLE_OK;
}

/*
 * Rotary position embedding of rows of heads (the optional fusion of the append: the paper is
 * silent on positional encoding; this is the rotation the Llama / Qwen families it evaluates
 * use).  For a row at absolute position t, every head vector x of even length D is rotated pairwise,
 * pair i = (x[i], x[i + D/2]), i < D/2, by the angle t * base^(-2i/D):
 *   y[i]       = x[i] cos a - x[i + D/2] sin a
 *   y[i + D/2] = x[i + D/2] cos a + x[i] sin a.
 * Inputs widened exactly, everything in double, output double [rows, H, D] (the caller rounds to
 * the cache's type: double -> binary32 -> bf16, each round-to-nearest-even).
 */
int oracle_rope_rows(const void *x, int32_t dtype, int64_t rows, int32_t H, int32_t D, const int32_t *pos,
                     double base, double *out) {
  if (rows < 0 || H <= 0 || D <= 0 || (D & 1) || !(base > 0.0)) return ORACLE_ERR_ARG;
  const int half = D / 2;
  for (int64_t r = 0; r < rows; ++r) {
    if (pos[r] < 0) return ORACLE_ERR_LEN;
    for (int h = 0; h < H; ++h) {
      const int64_t o = (r * H + h) * D;
      for (int i = 0; i < half; ++i) {
        const double a = (double)pos[r] * pow(base, -2.0 * (double)i / (double)D);
        const double c = cos(a), sn = sin(a);
        const double x0 = widen(x, dtype, o + i), x1 = widen(x, dtype, o + i + half);
        out[o + i] = x0 * c - x1 * sn;
        out[o + i + half] = x1 * c + x0 * sn;
      }
    }
  }
  return ORACLE_OK;
}

/*
 * Rollback: of the k_r+1 new positions, position 0 (the last committed token) and the n_r accepted
 * drafts stay in the cache; the k_r - n_r rejected drafts' entries are dropped by shrinking the
 * length (Figure 3 of the paper: accepted speculation continues, rejected speculation is
 * re-executed).  new_seq_lens[r] = L_r - (k_r - n_r).  The emitted token is the next step's
 * position 0 and is not in the cache yet.
 */
int oracle_kv_rollback(int32_t batch, const int32_t *seq_lens, const int32_t *q_indptr,
                       const int32_t *accepted_len, int32_t *new_seq_lens) {
  for (int r = 0; r < batch; ++r) {
    const int k = q_indptr[r + 1] - q_indptr[r] - 1;
    const int n = accepted_len[r];
    if (k < 0 || n < 0 || n > k || seq_lens[r] < k + 1) return ORACLE_ERR_LEN;
    new_seq_lens[r] = seq_lens[r] - (k - n);
  }
  return ORACLE_OK;
}
