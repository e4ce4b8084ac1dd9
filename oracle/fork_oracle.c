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
 *   - candidates at temperature tau > 0: x_0^k ~ q_theta^k(. | x_t; tau)  (Section 2; Algorithm 2
 *       line 4), drawn by inversion: the vocabulary is laid out in a stated order, the weights
 *       exp((x_v - m)/tau) are summed along it, and the token is the first one at which the running
 *       sum reaches U times the total, U a uniform variate from a stated counter-based generator
 *       (one per position and step).  The paper fixes the distribution, not the method of drawing;
 *       the order and the generator are this build's.  The confidence stays the UNtempered
 *       probability of the drawn token (Algorithm 2 line 5 has no tau).
 *   - the fallback orders the paper compares with: highest confidence (Algorithm 1, Fast-dLLM) and
 *       the lowest-confidence / highest-entropy / random ablations (Section 4.1, ablations).
 *   - top-entropy position selection of JustGRPO-Fast (Section 3.2, last paragraph).
 *   - the ForkGRPO objective (Eq. 2): ratio rho, group-standardised advantage, clipped minimum,
 *       mean over the fallback steps of a rollout, mean over rollouts; and its derivative with
 *       respect to the logits of a selected row.
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
 * AR and whole-block special cases of the loop; for the variants: moments and a chi-square of
 * the uniform stream, scipy's softmax(x/tau) for the drawn candidates, hand-worked fallback choices
 * of Algorithm 1 against Algorithm 2, numpy sorting for both selections, hand-worked advantages
 * and clipping cases of Eq. 2, finite differences for both derivatives.
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
  /* temperature > 0 only */
  int32_t a_s;         /* drawn token */
  double x_s;          /* its logit */
  double key_margin;   /* how far U * total is from the nearer end of the drawn token's stretch of the running sum,
                          as a fraction of the total (with slices: the smaller of that and the same for the slice) */
} row_red;

/* ---- the uniform variates of stochastic candidates ---------------------------------------------
 * One 64-bit key per (seed, step, b, k) from two splitmix finalisers; two uniforms on the 2^-23
 * grid of midpoints taken from disjoint bit fields of the key: U2 = ((key >> 41) + 1/2) 2^-23 draws
 * the token inside a slice of the vocabulary, U1 = (((key >> 18) mod 2^23) + 1/2) 2^-23 picks the slice
 * when the vocabulary is cut into several.  The CUDA path implements the same integer recipe on its own. */
static uint64_t mix64(uint64_t z) {
  z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ULL; z ^= z >> 27; z *= 0x94D049BB133111EBULL; z ^= z >> 31;
  return z;
}
static uint64_t noise_row_key(uint64_t seed, int32_t step, int32_t b, int32_t k) {
  uint64_t z = mix64(seed + 0x9E3779B97F4A7C15ULL * (uint64_t)((uint32_t)step + 1u));
  return mix64(z ^ (((uint64_t)(uint32_t)b << 32) | (uint64_t)(uint32_t)k));
}
static double uniform_token(uint64_t key) { return ((double)(key >> 41) + 0.5) * (1.0 / 8388608.0); }
static double uniform_slice(uint64_t key) { return ((double)((key >> 18) & 0x7FFFFFu) + 0.5) * (1.0 / 8388608.0); }

/* Exported for the pins: the two uniforms of row (seed, step, b, k). */
void fork_oracle_noise(uint64_t seed, int32_t step, int32_t b, int32_t k, double* u_token, double* u_slice) {
  const uint64_t key = noise_row_key(seed, step, b, k);
  if (u_token) *u_token = uniform_token(key);
  if (u_slice) *u_slice = uniform_slice(key);
}

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

/* ---- x_0 ~ q(. ; tau) for tau > 0 (Algorithm 2 line 4), by inversion -----------------------------
 * The order in which the vocabulary is laid out.  A slice of the vocabulary (the whole of it unless
 * the caller says otherwise) is cut into groups of G consecutive entries, G = 16 bytes' worth of
 * logits (8 bf16, 4 fp32); group number j belongs to lane j mod 256.  The order is: lane 0's groups
 * in ascending order, entries ascending inside a group; then lane 1's; ... ; then lane 255's; last the
 * fewer-than-G entries left over at the end of the slice.  Slices follow one another in ascending
 * order.  (Any fixed order gives a sample of the same distribution; this one is the order in which
 * the kernels' threads meet the entries.)
 *
 * One slice: with weights w_v = exp((x_v - m)/tau) (0 for -inf), total W, the token is the first v
 * in the order whose running sum reaches U2 * W.  Several slices: slice r is taken with probability
 * W_r / sum W, by inversion with U1 over the slices in ascending order, and the token inside it as
 * above with U2 and the slice's own total -- a two-stage draw of the same distribution.
 * Rows flagged bad keep the greedy candidate. */
enum { ORA_LANES = 256 };

typedef struct { double total; int32_t tok; double margin; } slice_draw;

static double tempered_weight(double x, double m, double tau) { return isinf(x) ? 0.0 : exp((x - m) / tau); }

/* visit the entries [v0, v1) of the row in the stated order; calls fn(ctx, v) */
static void visit_slice(int32_t v0, int32_t v1, int32_t G, void (*fn)(void*, int32_t), void* ctx) {
  const int32_t n = v1 - v0, ngroups = n / G;
  for (int32_t lane = 0; lane < ORA_LANES; ++lane)
    for (int32_t j = lane; j < ngroups; j += ORA_LANES)
      for (int32_t e = 0; e < G; ++e) fn(ctx, v0 + j * G + e);
  for (int32_t v = v0 + ngroups * G; v < v1; ++v) fn(ctx, v);
}

typedef struct { const void* row; int dtype; double m, tau; nsum acc; double target, before, after; int32_t tok; int found; } draw_ctx;
static void total_fn(void* c, int32_t v) {
  draw_ctx* d = (draw_ctx*)c;
  nsum_add(&d->acc, tempered_weight(load_logit(d->row, v, d->dtype), d->m, d->tau));
}
static void draw_fn(void* c, int32_t v) {
  draw_ctx* d = (draw_ctx*)c;
  if (d->found) return;
  const double w = tempered_weight(load_logit(d->row, v, d->dtype), d->m, d->tau);
  if (w <= 0.0) return;                                /* probability 0: never drawn */
  const double before = nsum_get(&d->acc);
  nsum_add(&d->acc, w);
  d->tok = v; d->before = before; d->after = nsum_get(&d->acc);   /* (the last entry with weight stands if rounding leaves the sum short) */
  if (d->after >= d->target) d->found = 1;
}

static slice_draw draw_in_slice(const void* row, int32_t v0, int32_t v1, int dtype, double m, double tau, double u) {
  const int32_t G = dtype == ORA_BF16 ? 8 : 4;
  draw_ctx d; memset(&d, 0, sizeof(d));
  d.row = row; d.dtype = dtype; d.m = m; d.tau = tau;
  visit_slice(v0, v1, G, total_fn, &d);
  slice_draw out; out.total = nsum_get(&d.acc); out.tok = -1; out.margin = INFINITY;
  if (!(out.total > 0.0)) return out;
  d.acc.sum = d.acc.comp = 0.0; d.target = u * out.total; d.tok = -1;
  visit_slice(v0, v1, G, draw_fn, &d);
  out.tok = d.tok;
  const double lo = d.target - d.before, hi = d.after - d.target;
  out.margin = (lo < hi ? lo : hi) / out.total;
  return out;
}

/* `slice_off`: n_slices + 1 ascending offsets into the row (NULL: the row is one slice) */
static void sample_row(const void* row, int32_t V, int dtype, double tau, uint64_t row_key, const int32_t* slice_off,
                       int32_t n_slices, row_red* out) {
  out->a_s = out->a; out->x_s = out->m; out->key_margin = INFINITY;
  if (out->status & ORA_ROW_BAD) return;
  const int32_t one[2] = {0, V};
  if (!slice_off || n_slices <= 0) { slice_off = one; n_slices = 1; }
  double grand = 0.0;
  slice_draw* d = (slice_draw*)malloc(sizeof(slice_draw) * (size_t)n_slices);
  for (int32_t r = 0; r < n_slices; ++r) {
    d[r] = draw_in_slice(row, slice_off[r], slice_off[r + 1], dtype, out->m, tau, uniform_token(row_key));
    grand += d[r].total;
  }
  const double target = uniform_slice(row_key) * grand;
  double run = 0.0, margin = INFINITY; int32_t pick = -1;
  for (int32_t r = 0; r < n_slices; ++r) {
    if (!(d[r].total > 0.0)) continue;
    const double before = run; run += d[r].total; pick = r;
    if (run >= target) { const double lo = target - before, hi = run - target; margin = (lo < hi ? lo : hi) / grand; break; }
  }
  if (pick >= 0) {
    out->a_s = d[pick].tok; out->x_s = load_logit(row, d[pick].tok, dtype);
    out->key_margin = n_slices > 1 && margin < d[pick].margin ? margin : d[pick].margin;
  }
  free(d);
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
  /* --- the variants the paper compares with; all-zero values give Algorithm 2 at temperature 0 --- */
  int32_t fallback_mode;                                               /* ORA_FB_* */
  const uint32_t* fallback_rand;                                       /* [B], ORA_FB_RANDOM only */
  float temperature;                                                   /* tau; 0 = arg-max candidates */
  uint64_t sample_seed;                                                /* noise stream of tau > 0 */
  double* fallback_margin;   /* [B] test aid: gap between the chosen fallback position's key and the runner-up */
  double* sample_margin;     /* [B,Lt] test aid: distance of the draw from the nearest boundary of the running sum, over the total */
  const int32_t* slice_off;  /* tau > 0: n_slices + 1 ascending offsets cutting the vocabulary into slices (NULL: one slice) */
  int32_t n_slices;
} fork_oracle_step_args;

/* Which position a fallback step commits.  LEFTMOST is Fork-dLLM (Algorithm 2); MAX_CONF is
   Fast-dLLM (Algorithm 1, arg-max_k c); MIN_CONF, MAX_ENTROPY and RANDOM are the ablations of
   Section 4.1.  Ties go to the lowest position; rows flagged bad are passed over unless every
   live row is bad, in which case the leftmost is taken. */
enum { ORA_FB_LEFTMOST = 0, ORA_FB_MAX_CONF = 1, ORA_FB_MIN_CONF = 2, ORA_FB_MAX_ENTROPY = 3, ORA_FB_RANDOM = 4 };

typedef struct { int32_t b, k; row_red red; } live_row;

typedef struct {
  const void* logits; int64_t stride_b, stride_l; int32_t pos0; int32_t V, dtype; size_t es;
  live_row* rows; int64_t n; int64_t next; pthread_mutex_t mu;
  double tau; uint64_t seed; int32_t step; const int32_t* slice_off; int32_t n_slices;
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
    if (J->tau > 0.0)
      sample_row(row, J->V, J->dtype, J->tau, noise_row_key(J->seed, J->step, lr->b, lr->k), J->slice_off, J->n_slices, &lr->red);
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

/* per-row outputs.  The candidate x_0^k is the arg-max (temperature 0) or the drawn token; its
   confidence c_t^k is its probability under the untempered softmax (Algorithm 2 lines 4-5). */
static int32_t row_cand(const row_red* q, int sampled) { return sampled ? q->a_s : q->a; }
static double row_logp(const row_red* q, int sampled) {
  if (q->status & ORA_ROW_BAD) return NAN;
  return (sampled ? q->x_s - q->m : 0.0) - log(q->s);
}
static double row_conf(const row_red* q, int sampled) {
  if (q->status & ORA_ROW_BAD) return 0.0;
  return sampled ? exp(q->x_s - q->m) / q->s : 1.0 / q->s;
}
static double row_entropy(const row_red* q) {
  return (q->status & ORA_ROW_BAD) ? NAN : log(q->s) - q->t / q->s;
}

int fork_oracle_step(const fork_oracle_step_args* A) {
  if (!A || !A->logits || !A->tokens || !A->mask || !A->blk_lo || !A->blk_hi) return ORA_ERR_ARG;
  if (A->B < 0 || A->Lt <= 0 || A->V <= 0 || A->Ll <= 0) return ORA_ERR_ARG;
  if (A->threshold != A->threshold) return ORA_ERR_ARG;
  if (A->fallback_mode < ORA_FB_LEFTMOST || A->fallback_mode > ORA_FB_RANDOM) return ORA_ERR_ARG;
  if (A->fallback_mode == ORA_FB_RANDOM && !A->fallback_rand) return ORA_ERR_ARG;
  if (!(A->temperature >= 0.0f) || isinf(A->temperature)) return ORA_ERR_ARG;
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
  J.tau = (double)A->temperature; J.seed = A->sample_seed; J.step = A->step;
  J.slice_off = A->slice_off; J.n_slices = A->n_slices;
  reduce_rows_parallel(&J, A->nthreads);
  const int sampled = A->temperature > 0.0f;

  const double lambda = (double)A->threshold;
  for (int32_t b = 0; b < B; ++b) {
    int64_t r0 = first[b], r1 = first[b + 1];
    if (r0 == r1) {                       /* nothing masked in the block: the step does nothing here */
      if (A->n_unmasked) A->n_unmasked[b] = 0;
      if (A->is_fallback) A->is_fallback[b] = 0;
      if (A->fallback_pos) A->fallback_pos[b] = -1;
      if (A->fallback_margin) A->fallback_margin[b] = INFINITY;
      continue;
    }
    int any_above = 0;
    for (int64_t r = r0; r < r1; ++r) {
      const row_red* q = &rows[r].red; int64_t at = (int64_t)b * Lt + rows[r].k;
      if (A->conf) A->conf[at] = row_conf(q, sampled);
      if (A->cand) A->cand[at] = row_cand(q, sampled);
      if (A->entropy) A->entropy[at] = row_entropy(q);
      if (A->logp) A->logp[at] = row_logp(q, sampled);
      if (A->row_status) A->row_status[at] = q->status;
      if (A->sample_margin) A->sample_margin[at] = sampled ? q->key_margin : INFINITY;
      if (row_conf(q, sampled) > lambda) any_above = 1;          /* U_t non-empty (line 6) */
    }
    int fb = !any_above;                                         /* fallback step: max_k c <= lambda */
    int64_t pick = r0;                                           /* the row a fallback step commits */
    double margin = INFINITY;
    if (fb && A->fallback_mode == ORA_FB_RANDOM) {
      pick = r0 + (int64_t)(A->fallback_rand[b] % (uint32_t)(r1 - r0));
    } else if (fb && A->fallback_mode != ORA_FB_LEFTMOST) {
      double best = 0.0, second = -INFINITY; int have = 0;
      for (int64_t r = r0; r < r1; ++r) {
        const row_red* q = &rows[r].red;
        if (q->status & ORA_ROW_BAD) continue;
        double key = A->fallback_mode == ORA_FB_MAX_CONF ? row_conf(q, sampled)
                   : A->fallback_mode == ORA_FB_MIN_CONF ? -row_conf(q, sampled) : row_entropy(q);
        if (!have || key > best) { if (have) second = best; best = key; pick = r; have = 1; }   /* strict: ties keep the lower position */
        else if (key > second) second = key;
      }
      if (have) margin = best - second;
    }
    if (A->fallback_margin) A->fallback_margin[b] = fb ? margin : INFINITY;
    int32_t count = 0;
    for (int64_t r = r0; r < r1; ++r) {
      const row_red* q = &rows[r].red; int64_t at = (int64_t)b * Lt + rows[r].k;
      int commit = fb ? (r == pick) : (row_conf(q, sampled) > lambda);   /* the fallback position, or the threshold set */
      if (!commit) continue;
      A->tokens[at] = row_cand(q, sampled); A->mask[at] = 0; ++count;
      if (A->commit_step) A->commit_step[at] = A->step;
      if (A->commit_fallback) A->commit_fallback[at] = (uint8_t)fb;
      if (A->commit_logp) A->commit_logp[at] = row_logp(q, sampled);
    }
    if (A->n_unmasked) A->n_unmasked[b] = count;
    if (A->is_fallback) A->is_fallback[b] = (uint8_t)fb;
    if (A->fallback_pos) A->fallback_pos[b] = fb ? rows[pick].k : -1;
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

/* ------------------------------------------------------------------------------------------ */
/* JustGRPO-Fast position selection (Section 3.2, last paragraph; Section 4.2 Setup): of the   */
/* eligible positions of each rollout keep the fraction `ratio` with the highest token entropy. */
/* Reading: the count is floor(ratio * n) with n the number of eligible positions (at least 1   */
/* when n > 0 and ratio > 0), equal entropies go to the lower position, NaN entropies rank last. */
int fork_oracle_select_top_entropy(const float* entropy, const uint8_t* eligible, int32_t B, int32_t Lt,
                                   float ratio, uint8_t* select, int32_t* n_selected) {
  if (!entropy || !eligible || !select || B < 0 || Lt <= 0 || !(ratio >= 0.0f) || ratio > 1.0f) return ORA_ERR_ARG;
  for (int32_t b = 0; b < B; ++b) {
    const float* H = entropy + (int64_t)b * Lt; const uint8_t* E = eligible + (int64_t)b * Lt;
    uint8_t* S = select + (int64_t)b * Lt;
    int32_t n = 0;
    for (int32_t k = 0; k < Lt; ++k) { S[k] = 0; if (E[k]) ++n; }
    int32_t want = (int32_t)floor((double)ratio * (double)n);
    if (want < 1 && n > 0 && ratio > 0.0f) want = 1;
    for (int32_t pick = 0; pick < want; ++pick) {           /* selection by repeated maximum */
      int32_t arg = -1;
      for (int32_t k = 0; k < Lt; ++k) {
        if (!E[k] || S[k]) continue;
        if (arg < 0) { arg = k; continue; }
        int k_nan = isnan(H[k]), a_nan = isnan(H[arg]);
        if ((a_nan && !k_nan) || (!a_nan && !k_nan && H[k] > H[arg])) arg = k;
      }
      S[arg] = 1;
    }
    if (n_selected) n_selected[b] = want;
  }
  return ORA_OK;
}

/* ------------------------------------------------------------------------------------------ */
/* The ForkGRPO objective (Eq. 2) on a batch of B = P * G rollouts, rollout i = p * G + j.       */
/*   rho_{i,t}  = exp(logp_new - logp_old) at the selected (fallback) positions,                 */
/*   A_i        = (r_i - mean_group) / std_group   (group-standardised; population std; a group  */
/*                with std 0 is skipped: its rollouts contribute nothing),                       */
/*   obj_i      = 1/|F_i| * sum_t min(rho A_i, clip(rho, 1-eps_lo, 1+eps_hi) A_i),               */
/*   J          = 1/B * sum_i obj_i      (1/G sum_i inside the expectation over prompts).        */
/* dlogp = dJ/dlogp_new: rho A_i / (B |F_i|) where the unclipped term is the minimum, else 0.    */
int fork_oracle_grpo_loss(int32_t B, int32_t Lt, int32_t group, const float* logp_new, const float* logp_old,
                          const uint8_t* select, const float* reward, float eps_lo, float eps_hi,
                          double* adv /*[B]*/, double* ratio /*[B,Lt]*/, double* seq_obj /*[B]*/,
                          double* objective /*[1]*/, double* dlogp /*[B,Lt]*/, uint8_t* skipped /*[B/group]*/) {
  if (B < 0 || Lt <= 0 || group <= 0 || B % group != 0 || !logp_new || !logp_old || !select || !reward) return ORA_ERR_ARG;
  double J = 0.0;
  for (int32_t p = 0; p < B / group; ++p) {
    double mean = 0.0, var = 0.0;
    for (int32_t j = 0; j < group; ++j) mean += (double)reward[p * group + j];
    mean /= group;
    for (int32_t j = 0; j < group; ++j) { double d = (double)reward[p * group + j] - mean; var += d * d; }
    double sd = sqrt(var / group);
    int skip = !(sd > 0.0);
    if (skipped) skipped[p] = (uint8_t)skip;
    for (int32_t j = 0; j < group; ++j) {
      int32_t i = p * group + j;
      double A = skip ? 0.0 : ((double)reward[i] - mean) / sd;
      if (adv) adv[i] = A;
      int32_t nf = 0;
      for (int32_t k = 0; k < Lt; ++k) if (select[(int64_t)i * Lt + k]) ++nf;
      double acc = 0.0;
      for (int32_t k = 0; k < Lt; ++k) {
        int64_t at = (int64_t)i * Lt + k;
        if (ratio) ratio[at] = 0.0;
        if (dlogp) dlogp[at] = 0.0;
        if (!select[at]) continue;
        double rho = exp((double)logp_new[at] - (double)logp_old[at]);
        double clipped = rho < 1.0 - (double)eps_lo ? 1.0 - (double)eps_lo : (rho > 1.0 + (double)eps_hi ? 1.0 + (double)eps_hi : rho);
        double u = rho * A, c = clipped * A;
        acc += (u <= c) ? u : c;
        if (ratio) ratio[at] = rho;
        if (dlogp && !skip && u <= c) dlogp[at] = rho * A / ((double)B * (double)nf);
      }
      double obj = nf > 0 ? acc / nf : 0.0;
      if (seq_obj) seq_obj[i] = obj;
      J += obj;
    }
  }
  if (objective) *objective = B > 0 ? J / B : 0.0;
  return ORA_OK;
}

/* Derivative of w * log q(tok) with respect to the logits of one row:                          */
/*   d/dx_v [x_tok - m - ln s] = 1[v = tok] - p_v,   p_v = exp(x_v - m)/s.                       */
int fork_oracle_row_logp_grad(const void* row, int32_t V, int32_t dtype, int32_t tok, double w, double* grad /*[V]*/) {
  if (!row || !grad || V <= 0 || tok < 0 || tok >= V) return ORA_ERR_ARG;
  row_red r; reduce_row(row, V, dtype, &r);
  if (r.status & ORA_ROW_BAD) { for (int32_t v = 0; v < V; ++v) grad[v] = NAN; return ORA_OK; }
  for (int32_t v = 0; v < V; ++v) {
    double x = load_logit(row, v, dtype);
    double p = isinf(x) ? 0.0 : exp(x - r.m) / r.s;
    grad[v] = w * ((v == tok ? 1.0 : 0.0) - p);
  }
  return ORA_OK;
}

/* Log-sum-exp m + ln s of one row (what the scoring pass hands to the backward pass). */
double fork_oracle_row_lse(const void* row, int32_t V, int32_t dtype) {
  row_red r; reduce_row(row, V, dtype, &r);
  return (r.status & ORA_ROW_BAD) ? NAN : r.m + log(r.s);
}
