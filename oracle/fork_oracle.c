/*
 * fork_oracle — plain, slow, fp64 CPU statement of what the Fork-dLLM sampling step computes.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import, link or call this file;
 * it exists so that the CUDA kernels can be checked against the paper's definitions.  It
 * shares no code, header, table or constant with the CUDA path.
 *
 * What is stated here, and where the paper defines it:
 *   - masked set M_t, candidate x_0^k, confidence c_t^k = q_theta^k(x_0^k | x_t)
 *       (Section 2, "Sampling in masked dLLMs"; Algorithm 2 lines 3-5).  With temperature 0
 *       the candidate is the arg-max of the position's distribution and its confidence is the
 *       largest softmax probability.
 *   - threshold set U_t = {k in M_t : c_t^k > lambda}  (strict; Section 2; Algorithm 2 line 6).
 *   - Fork fallback: if U_t is empty, U_t = {leftmost(M_t)}  (Algorithm 2, the highlighted line).
 *   - commit x_{t-1}^k = x_0^k for k in U_t, unchanged elsewhere  (Section 2; Algorithm 2 last line).
 *   - fallback steps F_i = {t : max_k c <= lambda} and the log-likelihood of the token committed
 *       there, log q_theta^{k_{i,t}}(x_0^{k_{i,t}} | x_t)  (Section 3.2, the ratio under Eq. 2).
 *   - semi-autoregressive blocks of length BL inside the generation window (Section 4.1 Setup).
 *   - token entropy of q_theta^k (Section 3.1 / Figure 2), in nats, of the untempered softmax.
 *
 * Softmax quantities are written out from their definitions with the usual max shift:
 *   m = max_v x_v,  a = min{v : x_v = m},  s = sum_v exp(x_v - m),  t = sum_v (x_v - m) exp(x_v - m)
 *   p_v = exp(x_v - m)/s,  conf = p_a = 1/s,
 *   H = -sum_v p_v ln p_v = ln s - t/s,   log p_tok = x_tok - m - ln s.
 * Terms with x_v = -inf contribute 0 to s and t.  Sums run in index order with Neumaier
 * compensation so the oracle's own rounding error is far below the 1e-9 level.
 *
 * Readings where the paper is silent (listed in the design notes): vocabulary ties go to the
 * lowest index; "leftmost" is taken inside the active block; fallback is decided per sequence;
 * a row holding NaN or +inf, or nothing but -inf, is "bad": status bit 0 is set, its confidence
 * is 0 (never above a threshold), entropy and log-probability are NaN, and its candidate is the
 * lowest index of the maximum over the non-NaN entries (0 if there is none).
 *
 * Parity pins (tests, CPU only): brute force without the max shift on tiny V, the one-peak /
 * k-way-tie closed forms, hand-worked rows and steps, library log-sum-exp/entropy, invariants,
 * AR and whole-block special cases of the loop.
 *
 * Build: gcc -O2 -std=c11 -fPIC -shared -pthread fork_oracle.c -lm
 */
#define _GNU_SOURCE
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <unistd.h>

enum { ORA_BF16 = 0, ORA_F32 = 1 };
enum { ORA_OK = 0, ORA_ERR_ARG = -1, ORA_ERR_MAX_STEPS = -4, ORA_ERR_PROVIDER = -5 };
enum { ORA_ROW_BAD = 1u, ORA_ROW_BAD_TOKEN = 2u };

/* exact widening of one stored logit to double */
static double load_logit(const void* row, int64_t v, int dtype) {
  if (dtype == ORA_BF16) {
    uint32_t bits = ((uint32_t)((const uint16_t*)row)[v]) << 16;
    float f; memcpy(&f, &bits, 4); return (double)f;
  }
  return (double)((const float*)row)[v];
}

typedef struct { double sum, comp; } nsum;           /* Neumaier compensated accumulator */
static void nsum_add(nsum* a, double x) {
  double t = a->sum + x;
  if (fabs(a->sum) >= fabs(x)) a->comp += (a->sum - t) + x; else a->comp += (x - t) + a->sum;
  a->sum = t;
}
static double nsum_get(const nsum* a) { return a->sum + a->comp; }

typedef struct {
  double m, s, t;      /* max, sum exp(x-m), sum (x-m) exp(x-m) */
  int32_t a;           /* lowest arg-max */
  uint32_t status;
} row_red;

/* m, a, s, t of one row, straight from the definitions */
static void reduce_row(const void* row, int32_t V, int dtype, row_red* out) {
  int has_nan = 0, has_pinf = 0, any = 0;
  double m = -INFINITY; int32_t a = -1;
  for (int32_t v = 0; v < V; ++v) {
    double x = load_logit(row, v, dtype);
    if (isnan(x)) { has_nan = 1; continue; }
    if (isinf(x) && x > 0) has_pinf = 1;
    if (!any || x > m) { m = x; a = v; any = 1; }    /* strict > keeps the lowest index on ties */
  }
  out->a = (a < 0) ? 0 : a; out->m = m; out->s = 0.0; out->t = 0.0; out->status = 0;
  if (has_nan || has_pinf || !any || (isinf(m) && m < 0)) { out->status = ORA_ROW_BAD; return; }
  nsum s = {0, 0}, t = {0, 0};
  for (int32_t v = 0; v < V; ++v) {
    double x = load_logit(row, v, dtype);
    if (isinf(x)) continue;                          /* -inf: probability 0, term 0 */
    double d = x - m, e = exp(d);
    nsum_add(&s, e); nsum_add(&t, d * e);
  }
  out->s = nsum_get(&s); out->t = nsum_get(&t);
}

/* Exported: statistics of a single row. Any output pointer may be NULL. */
void fork_oracle_row_stats(const void* row, int32_t V, int32_t dtype,
                           double* conf, int32_t* cand, double* entropy, double* logp_cand,
                           double* m_out, double* s_out, double* t_out, uint32_t* status) {
  row_red r; reduce_row(row, V, dtype, &r);
  int bad = (r.status & ORA_ROW_BAD) != 0;
  if (conf) *conf = bad ? 0.0 : 1.0 / r.s;
  if (cand) *cand = r.a;
  if (entropy) *entropy = bad ? NAN : log(r.s) - r.t / r.s;
  if (logp_cand) *logp_cand = bad ? NAN : -log(r.s);
  if (m_out) *m_out = r.m; if (s_out) *s_out = r.s; if (t_out) *t_out = r.t;
  if (status) *status = r.status;
}

/* Exported: log-probability of token tok in one row: x_tok - m - ln s. */
double fork_oracle_row_logp(const void* row, int32_t V, int32_t dtype, int32_t tok, uint32_t* status) {
  row_red r; reduce_row(row, V, dtype, &r);
  uint32_t st = r.status;
  double lp;
  if (tok < 0 || tok >= V) { st |= ORA_ROW_BAD_TOKEN; lp = 0.0; }
  else if (st & ORA_ROW_BAD) lp = NAN;
  else lp = load_logit(row, tok, dtype) - r.m - log(r.s);
  if (status) *status = st;
  return lp;
}

/* ------------------------------------------------------------------------------------------ */
/* One sampling step (Algorithm 2) over a batch of sequences; all pointers are host memory.    */
typedef struct fork_oracle_step_args {
  const void* logits; int64_t stride_b, stride_l; int32_t pos0;
  int32_t B, Lt, Ll, V, dtype;
  int32_t* tokens; uint8_t* mask; const int32_t* blk_lo; const int32_t* blk_hi;
  float threshold; int32_t step;
  double* conf; int32_t* cand; double* entropy; double* logp;          /* [B,Lt], written on the active set */
  int32_t* commit_step; uint8_t* commit_fallback; double* commit_logp; /* [B,Lt], written on the commit set */
  int32_t* n_unmasked; uint8_t* is_fallback; int32_t* fallback_pos;    /* [B] */
  int32_t* nfe; int32_t* n_fallback;                                   /* [B], accumulated */
  uint32_t* row_status;                                                /* [B,Lt], written on the active set */
  int32_t nthreads;                                                    /* <=0: all host cores */
} fork_oracle_step_args;

typedef struct { int32_t b, k; row_red red; } live_row;

typedef struct {
  const void* logits; int64_t stride_b, stride_l; int32_t pos0; int32_t V, dtype; size_t es;
  live_row* rows; int64_t n; int64_t next; pthread_mutex_t mu;
} reduce_job;

static void* reduce_worker(void* p) {
  reduce_job* J = (reduce_job*)p;
  for (;;) {
    pthread_mutex_lock(&J->mu); int64_t r = J->next++; pthread_mutex_unlock(&J->mu);
    if (r >= J->n) break;
    live_row* lr = &J->rows[r];
    const char* row = (const char*)J->logits +
        ((int64_t)lr->b * J->stride_b + (int64_t)(lr->k - J->pos0) * J->stride_l) * (int64_t)J->es;
    reduce_row(row, J->V, J->dtype, &lr->red);
  }
  return NULL;
}

static int host_threads(int req, int64_t n) {
  int nt = req > 0 ? req : (int)sysconf(_SC_NPROCESSORS_ONLN);
  if (nt < 1) nt = 1; if (nt > 256) nt = 256;
  if ((int64_t)nt > n) nt = (int)(n > 0 ? n : 1);
  return nt;
}

static void reduce_rows_parallel(reduce_job* J, int nthreads) {
  J->next = 0; pthread_mutex_init(&J->mu, NULL);
  int nt = host_threads(nthreads, J->n);
  pthread_t th[256];
  for (int i = 1; i < nt; ++i) pthread_create(&th[i], NULL, reduce_worker, J);
  reduce_worker(J);
  for (int i = 1; i < nt; ++i) pthread_join(th[i], NULL);
  pthread_mutex_destroy(&J->mu);
}

int fork_oracle_threads_used(int32_t nthreads, int64_t n_rows) { return host_threads(nthreads, n_rows); }

int fork_oracle_step(const fork_oracle_step_args* A) {
  if (!A || !A->logits || !A->tokens || !A->mask || !A->blk_lo || !A->blk_hi) return ORA_ERR_ARG;
  if (A->B < 0 || A->Lt <= 0 || A->V <= 0 || A->Ll <= 0) return ORA_ERR_ARG;
  if (A->threshold != A->threshold) return ORA_ERR_ARG;
  const int32_t B = A->B, Lt = A->Lt;
  /* M_t restricted to each sequence's active block (Algorithm 2 line 3; semi-AR blocks) */
  live_row* rows = (live_row*)malloc(sizeof(live_row) * (size_t)((int64_t)B * Lt + 1));
  int64_t* first = (int64_t*)malloc(sizeof(int64_t) * (size_t)(B + 1));
  int64_t n = 0;
  for (int32_t b = 0; b < B; ++b) {
    first[b] = n;
    int32_t lo = A->blk_lo[b], hi = A->blk_hi[b];
    if (lo < 0) lo = 0; if (hi > Lt) hi = Lt;
    if (lo < A->pos0) lo = A->pos0; if (hi > A->pos0 + A->Ll) hi = A->pos0 + A->Ll;
    for (int32_t k = lo; k < hi; ++k)
      if (A->mask[(int64_t)b * Lt + k]) { rows[n].b = b; rows[n].k = k; ++n; }
  }
  first[B] = n;
  /* q_theta^k for every k in the active set: the only O(V) work */
  reduce_job J; J.logits = A->logits; J.stride_b = A->stride_b; J.stride_l = A->stride_l; J.pos0 = A->pos0;
  J.V = A->V; J.dtype = A->dtype; J.es = (A->dtype == ORA_BF16) ? 2 : 4; J.rows = rows; J.n = n;
  reduce_rows_parallel(&J, A->nthreads);

  const double lambda = (double)A->threshold;
  for (int32_t b = 0; b < B; ++b) {
    int64_t r0 = first[b], r1 = first[b + 1];
    if (r0 == r1) {                       /* nothing masked in the block: the step does nothing here */
      if (A->n_unmasked) A->n_unmasked[b] = 0;
      if (A->is_fallback) A->is_fallback[b] = 0;
      if (A->fallback_pos) A->fallback_pos[b] = -1;
      continue;
    }
    int any_above = 0;
    for (int64_t r = r0; r < r1; ++r) {
      const row_red* q = &rows[r].red; int64_t at = (int64_t)b * Lt + rows[r].k;
      int bad = (q->status & ORA_ROW_BAD) != 0;
      double c = bad ? 0.0 : 1.0 / q->s;                         /* c_t^k (Algorithm 2 line 5) */
      if (A->conf) A->conf[at] = c;
      if (A->cand) A->cand[at] = q->a;                           /* x_0^k at temperature 0 */
      if (A->entropy) A->entropy[at] = bad ? NAN : log(q->s) - q->t / q->s;
      if (A->logp) A->logp[at] = bad ? NAN : -log(q->s);
      if (A->row_status) A->row_status[at] = q->status;
      if (c > lambda) any_above = 1;                             /* U_t non-empty (line 6) */
    }
    int fb = !any_above;                                         /* fallback step: max_k c <= lambda */
    int32_t count = 0;
    for (int64_t r = r0; r < r1; ++r) {
      const row_red* q = &rows[r].red; int64_t at = (int64_t)b * Lt + rows[r].k;
      int bad = (q->status & ORA_ROW_BAD) != 0;
      double c = bad ? 0.0 : 1.0 / q->s;
      int commit = fb ? (r == r0) : (c > lambda);                /* leftmost(M_t) or the threshold set */
      if (!commit) continue;
      A->tokens[at] = q->a; A->mask[at] = 0; ++count;
      if (A->commit_step) A->commit_step[at] = A->step;
      if (A->commit_fallback) A->commit_fallback[at] = (uint8_t)fb;
      if (A->commit_logp) A->commit_logp[at] = bad ? NAN : -log(q->s);
    }
    if (A->n_unmasked) A->n_unmasked[b] = count;
    if (A->is_fallback) A->is_fallback[b] = (uint8_t)fb;
    if (A->fallback_pos) A->fallback_pos[b] = fb ? rows[r0].k : -1;
    if (A->nfe) A->nfe[b] += 1;
    if (A->n_fallback) A->n_fallback[b] += fb;
  }
  free(rows); free(first);
  return ORA_OK;
}

/* ------------------------------------------------------------------------------------------ */
/* Log-likelihood of given tokens at selected positions (the numerator / denominator of the   */
/* ForkGRPO ratio, Section 3.2), per token and summed per sequence in ascending position.     */
typedef struct { int32_t b, k, tok; double lp; uint32_t st; } lp_row;
typedef struct {
  const void* logits; int64_t stride_b, stride_l; int32_t pos0; int32_t V, dtype; size_t es;
  lp_row* rows; int64_t n; int64_t next; pthread_mutex_t mu;
} lp_job;

static void* lp_worker(void* p) {
  lp_job* J = (lp_job*)p;
  for (;;) {
    pthread_mutex_lock(&J->mu); int64_t r = J->next++; pthread_mutex_unlock(&J->mu);
    if (r >= J->n) break;
    lp_row* q = &J->rows[r];
    const char* row = (const char*)J->logits +
        ((int64_t)q->b * J->stride_b + (int64_t)(q->k - J->pos0) * J->stride_l) * (int64_t)J->es;
    q->lp = fork_oracle_row_logp(row, J->V, J->dtype, q->tok, &q->st);
  }
  return NULL;
}

int fork_oracle_logprob(const void* logits, int64_t stride_b, int64_t stride_l, int32_t pos0,
                        int32_t B, int32_t Lt, int32_t Ll, int32_t V, int32_t dtype,
                        const int32_t* tokens, const uint8_t* select,
                        double* logp /*[B,Lt]*/, double* seq_sum /*[B]*/, int32_t* seq_cnt /*[B]*/,
                        uint32_t* row_status /*[B,Lt] or NULL*/, int32_t nthreads) {
  if (!logits || !tokens || !select || B < 0 || Lt <= 0 || V <= 0 || Ll <= 0) return ORA_ERR_ARG;
  lp_row* rows = (lp_row*)malloc(sizeof(lp_row) * (size_t)((int64_t)B * Lt + 1));
  int64_t n = 0;
  for (int32_t b = 0; b < B; ++b)
    for (int32_t k = 0; k < Lt; ++k) {
      int64_t at = (int64_t)b * Lt + k;
      if (logp) logp[at] = 0.0;
      if (!select[at] || k < pos0 || k >= pos0 + Ll) continue;
      rows[n].b = b; rows[n].k = k; rows[n].tok = tokens[at]; ++n;
    }
  lp_job J; J.logits = logits; J.stride_b = stride_b; J.stride_l = stride_l; J.pos0 = pos0; J.V = V;
  J.dtype = dtype; J.es = (dtype == ORA_BF16) ? 2 : 4; J.rows = rows; J.n = n; J.next = 0;
  pthread_mutex_init(&J.mu, NULL);
  int nt = host_threads(nthreads, n);
  pthread_t th[256];
  for (int i = 1; i < nt; ++i) pthread_create(&th[i], NULL, lp_worker, &J);
  lp_worker(&J);
  for (int i = 1; i < nt; ++i) pthread_join(th[i], NULL);
  pthread_mutex_destroy(&J.mu);
  for (int32_t b = 0; b < B; ++b) { if (seq_sum) seq_sum[b] = 0.0; if (seq_cnt) seq_cnt[b] = 0; }
  for (int64_t r = 0; r < n; ++r) {            /* rows are in ascending (b, k) order */
    int64_t at = (int64_t)rows[r].b * Lt + rows[r].k;
    if (logp) logp[at] = rows[r].lp;
    if (row_status) row_status[at] = rows[r].st;
    if (seq_sum) seq_sum[rows[r].b] += rows[r].lp;
    if (seq_cnt) seq_cnt[rows[r].b] += 1;
  }
  free(rows);
  return ORA_OK;
}

/* ------------------------------------------------------------------------------------------ */
/* Block cursor of the semi-autoregressive loop (Section 4.1 Setup: blocks of BL inside the    */
/* generation window): the first block at or after `from` that still holds a masked position. */
static void next_block(const uint8_t* mask_b, int32_t gen_lo, int32_t gen_hi, int32_t block_len,
                       int32_t from, int32_t* lo, int32_t* hi) {
  for (int32_t s = from; s < gen_hi; s += block_len) {
    int32_t e = s + block_len; if (e > gen_hi) e = gen_hi;
    for (int32_t k = s; k < e; ++k) if (mask_b[k]) { *lo = s; *hi = e; return; }
  }
  (void)gen_lo; *lo = gen_hi; *hi = gen_hi;
}

/* Exported helper: the loop's initial / advanced cursors for every sequence. */
void fork_oracle_block_cursors(const uint8_t* mask, int32_t B, int32_t Lt, int32_t gen_lo, int32_t gen_hi,
                               int32_t block_len, int32_t* lo, int32_t* hi) {
  for (int32_t b = 0; b < B; ++b) {
    int32_t from = gen_lo;
    if (lo[b] >= gen_lo && lo[b] < gen_hi) from = lo[b];
    next_block(mask + (int64_t)b * Lt, gen_lo, gen_hi, block_len, from, &lo[b], &hi[b]);
  }
}

typedef int (*fork_oracle_logits_fn)(void* ctx, int32_t step, const int32_t* tokens, const uint8_t* mask,
                                     const int32_t* blk_lo, const int32_t* blk_hi, void* logits_out);

/* Iterated sampling until nothing in [gen_lo, gen_hi) is masked (Section 2: "until all positions
   have been unmasked"), one provider call (= one model evaluation, NFE) per step.  A->blk_lo /
   A->blk_hi are ignored; the loop keeps its own cursors.  A->step is the id of the first step. */
int fork_oracle_decode_loop(fork_oracle_step_args* A, int32_t block_len, int32_t gen_lo, int32_t gen_hi,
                            fork_oracle_logits_fn provider, void* ctx, int32_t max_steps, int32_t* steps_taken) {
  if (!A || !provider || block_len <= 0 || gen_lo < 0 || gen_hi > A->Lt || gen_lo > gen_hi) return ORA_ERR_ARG;
  int32_t B = A->B;
  int32_t* lo = (int32_t*)malloc(sizeof(int32_t) * (size_t)(B + 1));
  int32_t* hi = (int32_t*)malloc(sizeof(int32_t) * (size_t)(B + 1));
  for (int32_t b = 0; b < B; ++b) { lo[b] = gen_lo; hi[b] = gen_lo; }
  fork_oracle_block_cursors(A->mask, B, A->Lt, gen_lo, gen_hi, block_len, lo, hi);
  fork_oracle_step_args S = *A; S.blk_lo = lo; S.blk_hi = hi;
  int32_t n = 0; int rc = ORA_OK;
  for (;;) {
    int live = 0;
    for (int32_t b = 0; b < B; ++b) if (lo[b] < hi[b]) live = 1;
    if (!live) break;
    if (n >= max_steps) { rc = ORA_ERR_MAX_STEPS; break; }
    if (provider(ctx, A->step + n, S.tokens, S.mask, lo, hi, (void*)S.logits) != 0) { rc = ORA_ERR_PROVIDER; break; }
    S.step = A->step + n;
    rc = fork_oracle_step(&S);
    if (rc != ORA_OK) break;
    ++n;
    fork_oracle_block_cursors(S.mask, B, A->Lt, gen_lo, gen_hi, block_len, lo, hi);
  }
  if (steps_taken) *steps_taken = n;
  free(lo); free(hi);
  return rc;
}
