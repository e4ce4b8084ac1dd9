/*
 * Host side of the synthetic-logit generator: builds the normal-quantile tables
 * and fills rows in host memory.  Input making only; see fork_synth.h.
 * Build: gcc -O2 -ffp-contract=off -fPIC -shared -pthread fork_synth_cpu.c -lm
 */
#include "fork_synth.h"

#include <math.h>
#include <pthread.h>
#include <stdlib.h>
#include <string.h>
#include <unistd.h>

static fs_tab_entry g_main[FS_TAB_N];
static fs_tab_entry g_tail[FS_TAB_N];
static pthread_once_t g_once = PTHREAD_ONCE_INIT;

/* upper-tail quantile: z with P(Z > z) = q, 0 < q <= 0.5, by Newton on erfc in fp64 */
static double upper_quantile(double q) {
  if (q >= 0.5) return 0.0;
  /* start from the leading asymptotic term, then polish */
  double t = sqrt(-2.0 * log(q));
  double z = t - (2.515517 + 0.802853 * t + 0.010328 * t * t) /
                 (1.0 + 1.432788 * t + 0.189269 * t * t + 0.001308 * t * t * t);
  for (int it = 0; it < 60; ++it) {
    double f = 0.5 * erfc(z * M_SQRT1_2) - q;
    double d = -exp(-0.5 * z * z) / sqrt(2.0 * M_PI);
    double step = f / d;
    z -= step;
    if (fabs(step) < 1e-15 * (1.0 + fabs(z))) break;
  }
  return z;
}

static void build_tables(void) {
  /* main: bin i covers upper-tail mass q from 0.5 - i/2^17 down to 0.5 - (i+1)/2^17 */
  double prev = 0.0;
  for (int i = 0; i < FS_TAB_N; ++i) {
    double q_hi = 0.5 - (double)(i + 1) / 131072.0;
    double next = (i + 1 < FS_TAB_N) ? upper_quantile(q_hi) : prev; /* last bin is refined by g_tail */
    g_main[i].q = (float)prev;
    g_main[i].dq = (float)(next - prev);
    prev = next;
  }
  /* tail: the last main bin, upper-tail mass 2^-17 .. 0, split into 2^16 equal-mass sub-bins */
  const double two33 = 8589934592.0;
  prev = upper_quantile(65536.0 / two33);
  for (int j = 0; j < FS_TAB_N; ++j) {
    double q = (double)(FS_TAB_N - j - 1) / two33;
    if (q <= 0.0) q = 0.25 / two33;
    double next = upper_quantile(q);
    g_tail[j].q = (float)prev;
    g_tail[j].dq = (float)(next - prev);
    prev = next;
  }
}

void fork_synth_tables(const fs_tab_entry** tab_main, const fs_tab_entry** tab_tail) {
  pthread_once(&g_once, build_tables);
  if (tab_main) *tab_main = g_main;
  if (tab_tail) *tab_tail = g_tail;
}

void fork_synth_plan_host(const fork_synth_cfg* cfg, int32_t b, int32_t l, fs_row_plan* out) {
  fs_plan_row(cfg, b, l, out);
}

void fork_synth_row_host(const fork_synth_cfg* cfg, uint32_t nonce, int32_t step, int32_t b, int32_t l, void* out) {
  pthread_once(&g_once, build_tables);
  fs_row_plan plan;
  fs_plan_row(cfg, b, l, &plan);
  uint64_t key = fs_row_key(cfg->seed, nonce, step, b, l);
  if (cfg->dtype == FS_BF16) {
    uint16_t* o = (uint16_t*)out;
    for (int32_t v = 0; v < cfg->V; ++v) o[v] = fs_f32_to_bf16(fs_logit(cfg, &plan, key, v, g_main, g_tail));
  } else {
    float* o = (float*)out;
    for (int32_t v = 0; v < cfg->V; ++v) o[v] = fs_logit(cfg, &plan, key, v, g_main, g_tail);
  }
}

typedef struct {
  const fork_synth_cfg* cfg; uint32_t nonce; int32_t step;
  const int32_t* rows_b; const int32_t* rows_k; int64_t n_rows;
  char* logits; int64_t stride_b, stride_l; int32_t pos0; size_t es;
  int64_t next; pthread_mutex_t mu;
} fill_job;

static void* fill_worker(void* p) {
  fill_job* J = (fill_job*)p;
  for (;;) {
    pthread_mutex_lock(&J->mu);
    int64_t r = J->next++;
    pthread_mutex_unlock(&J->mu);
    if (r >= J->n_rows) break;
    int32_t b = J->rows_b[r], k = J->rows_k[r];
    char* dst = J->logits + ((int64_t)b * J->stride_b + (int64_t)(k - J->pos0) * J->stride_l) * (int64_t)J->es;
    fork_synth_row_host(J->cfg, J->nonce, J->step, b, k, dst);
  }
  return NULL;
}

int64_t fork_synth_fill_host(const fork_synth_cfg* cfg, uint32_t nonce, int32_t step,
                             const uint8_t* mask, const int32_t* lo, const int32_t* hi,
                             void* logits, int64_t stride_b, int64_t stride_l, int32_t pos0, int32_t Ll,
                             int32_t nthreads) {
  pthread_once(&g_once, build_tables);
  int64_t cap = (int64_t)cfg->B * cfg->Lt;
  int32_t* rb = (int32_t*)malloc(sizeof(int32_t) * (size_t)(cap > 0 ? cap : 1));
  int32_t* rk = (int32_t*)malloc(sizeof(int32_t) * (size_t)(cap > 0 ? cap : 1));
  int64_t n = 0;
  for (int32_t b = 0; b < cfg->B; ++b) {
    int32_t a = lo[b] < 0 ? 0 : lo[b], e = hi[b] > cfg->Lt ? cfg->Lt : hi[b];
    for (int32_t k = a; k < e; ++k) {
      if (k < pos0 || k >= pos0 + Ll) continue;
      if (mask[(int64_t)b * cfg->Lt + k]) { rb[n] = b; rk[n] = k; ++n; }
    }
  }
  fill_job J;
  J.cfg = cfg; J.nonce = nonce; J.step = step; J.rows_b = rb; J.rows_k = rk; J.n_rows = n;
  J.logits = (char*)logits; J.stride_b = stride_b; J.stride_l = stride_l; J.pos0 = pos0;
  J.es = (cfg->dtype == FS_BF16) ? 2 : 4; J.next = 0;
  pthread_mutex_init(&J.mu, NULL);
  int nt = nthreads > 0 ? nthreads : (int)sysconf(_SC_NPROCESSORS_ONLN);
  if (nt < 1) nt = 1;
  if (nt > 256) nt = 256;
  if ((int64_t)nt > n) nt = (int)(n > 0 ? n : 1);
  pthread_t th[256];
  for (int i = 1; i < nt; ++i) pthread_create(&th[i], NULL, fill_worker, &J);
  fill_worker(&J);
  for (int i = 1; i < nt; ++i) pthread_join(th[i], NULL);
  pthread_mutex_destroy(&J.mu);
  free(rb); free(rk);
  return n;
}
