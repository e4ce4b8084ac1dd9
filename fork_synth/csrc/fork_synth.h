/*
 * fork_synth — seeded synthetic logits for the Fork-dLLM confidence pass.
 *
 * This module only MAKES inputs.  It holds none of the sampler's arithmetic
 * (no softmax, no max/sum-exp, no threshold rule): it draws a Gaussian
 * background per vocabulary entry and plants peaks / near-tied "fork" tops.
 * The same inline core compiles for the host (gcc) and for the device (nvcc),
 * and every floating-point step is a single correctly-rounded operation
 * (fmaf / one multiply / one add), so the host and the device produce
 * bit-identical rows from the same (seed, nonce, step, b, l, v).
 *
 * Stand-in for: logits of LLaDA-8B-Instruct / Dream-7B on the paper's suites
 * (Section 4.1 Setup), which need weights and datasets that are not available.
 */
#ifndef FORK_SYNTH_H
#define FORK_SYNTH_H

#include <stdint.h>

#ifdef __CUDACC__
#define FS_HD __host__ __device__ __forceinline__
#else
#define FS_HD static inline
#endif

#ifdef __cplusplus
extern "C" {
#endif

enum { FS_BF16 = 0, FS_F32 = 1 };
enum { FS_PEAK_ADD = 0, /* planted logit = background draw + h   ("literal" reading)   */
       FS_PEAK_SET = 1  /* planted logit = peak_base + h          ("calibrated" reading) */ };

/* Table of the standard-normal quantile function, built once on the host. */
#define FS_TAB_N 65536
typedef struct { float q; float dq; } fs_tab_entry; /* value at the bin's low edge, width of the bin */

typedef struct fork_synth_cfg {
  uint64_t seed;
  int32_t  B, Lt, V;
  int32_t  dtype;        /* FS_BF16 / FS_F32 */
  float    sigma;        /* background std */
  int32_t  peak_mode;    /* FS_PEAK_ADD / FS_PEAK_SET */
  float    peak_base;    /* used by FS_PEAK_SET and by fork rows */
  float    peak_prob;    /* P(position carries a single planted peak), keyed by (seed,b,l) */
  float    h_lo, h_span; /* peak height h = h_lo + u * h_span, u in [0,1) */
  float    fork_prob;    /* P(position is a "fork" row with 2..4 near-equal tops), keyed by (seed,b,l) */
  float    fork_h;       /* fork tops sit at peak_base + fork_h - gap_j */
  float    fork_gap;     /* gap_0 = 0, gap_j = u_j * fork_gap */
} fork_synth_cfg;

/* Per-row planting decisions, a pure function of (cfg, b, l). */
typedef struct fs_row_plan {
  int32_t n_planted;     /* 0, 1 (peak) or 2..4 (fork) */
  int32_t is_fork;
  int32_t tok[4];
  float   val[4];        /* FS_PEAK_ADD single peak: the height h to add; otherwise the value to set */
} fs_row_plan;

FS_HD uint64_t fs_mix64(uint64_t x) {
  x ^= x >> 30; x *= 0xbf58476d1ce4e5b9ULL;
  x ^= x >> 27; x *= 0x94d049bb133111ebULL;
  x ^= x >> 31; return x;
}

FS_HD float fs_u01(uint64_t h) {            /* 24 random bits -> [0,1), exact */
  return (float)(uint32_t)(h >> 40) * 5.9604644775390625e-08f;
}

FS_HD float fs_fma(float a, float b, float c) {
#ifdef __CUDA_ARCH__
  return __fmaf_rn(a, b, c);
#else
  return __builtin_fmaf(a, b, c);
#endif
}
FS_HD float fs_mul(float a, float b) {
#ifdef __CUDA_ARCH__
  return __fmul_rn(a, b);
#else
  return a * b;   /* built with -ffp-contract=off: never fused with a following add */
#endif
}
FS_HD float fs_add(float a, float b) {
#ifdef __CUDA_ARCH__
  return __fadd_rn(a, b);
#else
  return a + b;
#endif
}

/* key of one logits row's background: fresh per (nonce, step, b, l) */
FS_HD uint64_t fs_row_key(uint64_t seed, uint32_t nonce, int32_t step, int32_t b, int32_t l) {
  uint64_t k = fs_mix64(seed ^ 0x5851f42d4c957f2dULL);
  k = fs_mix64(k + (((uint64_t)(uint32_t)step) << 32 | (uint64_t)nonce));
  k = fs_mix64(k + (((uint64_t)(uint32_t)b) << 32 | (uint64_t)(uint32_t)l));
  return k;
}

/* standard normal draw from a 64-bit hash: sign bit, 16-bit bin, 24-bit position in the bin;
   the outermost bin is refined by a second table over the next 16 bits. */
FS_HD float fs_normal(uint64_t h, const fs_tab_entry* tab_main, const fs_tab_entry* tab_tail) {
  uint32_t i = (uint32_t)(h >> 47) & 0xFFFFu;
  float z;
  if (i != 0xFFFFu) {
    float f = (float)((uint32_t)(h >> 23) & 0xFFFFFFu) * 5.9604644775390625e-08f;
    z = fs_fma(f, tab_main[i].dq, tab_main[i].q);
  } else {
    uint32_t j = (uint32_t)(h >> 31) & 0xFFFFu;
    float f = (float)((uint32_t)(h >> 7) & 0xFFFFFFu) * 5.9604644775390625e-08f;
    z = fs_fma(f, tab_tail[j].dq, tab_tail[j].q);
  }
  return (h >> 63) ? -z : z;
}

FS_HD float fs_background(const fork_synth_cfg* c, uint64_t row_key, int32_t v,
                          const fs_tab_entry* tab_main, const fs_tab_entry* tab_tail) {
  uint64_t h = fs_mix64(row_key + (uint64_t)(uint32_t)v * 0x9E3779B97F4A7C15ULL);
  return fs_mul(c->sigma, fs_normal(h, tab_main, tab_tail));
}

/* float -> bf16 bits, round to nearest even, integer arithmetic only (inputs are finite) */
FS_HD uint16_t fs_f32_to_bf16(float x) {
  union { float f; uint32_t u; } cv; cv.f = x;
  uint32_t u = cv.u;
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

FS_HD void fs_plan_row(const fork_synth_cfg* c, int32_t b, int32_t l, fs_row_plan* p) {
  uint64_t k = fs_mix64(c->seed ^ 0xda942042e4dd58b5ULL);
  k = fs_mix64(k + (((uint64_t)(uint32_t)b) << 32 | (uint64_t)(uint32_t)l));
  uint64_t h0 = fs_mix64(k + 1), h1 = fs_mix64(k + 2), h2 = fs_mix64(k + 3), h3 = fs_mix64(k + 4);
  float u_kind = fs_u01(h0);
  int32_t V = c->V;
  p->n_planted = 0; p->is_fork = 0;
  for (int j = 0; j < 4; ++j) { p->tok[j] = -1; p->val[j] = 0.f; }
  if (u_kind < c->fork_prob && V >= 16) {
    int32_t n = 2 + (int32_t)((h0 & 0xFFFFu) % 3u);
    int32_t t0 = (int32_t)(h1 % (uint64_t)V);
    int32_t st = 1 + (int32_t)((h1 >> 32) % (uint64_t)(V / 8));
    p->is_fork = 1; p->n_planted = n;
    for (int j = 0; j < n; ++j) {
      p->tok[j] = (int32_t)(((int64_t)t0 + (int64_t)j * st) % V);
      float gap = (j == 0) ? 0.f : fs_mul(fs_u01(fs_mix64(h2 + (uint64_t)j)), c->fork_gap);
      p->val[j] = fs_add(fs_add(c->peak_base, c->fork_h), -gap);
    }
  } else if (u_kind < fs_add(c->fork_prob, c->peak_prob)) {
    float h = fs_fma(fs_u01(h3), c->h_span, c->h_lo);
    p->n_planted = 1;
    p->tok[0] = (int32_t)(h1 % (uint64_t)V);
    p->val[0] = (c->peak_mode == FS_PEAK_SET) ? fs_add(c->peak_base, h) : h;
  }
}

/* The logit at vocabulary entry v of one row, before rounding to the storage type. */
FS_HD float fs_logit(const fork_synth_cfg* c, const fs_row_plan* p, uint64_t row_key, int32_t v,
                     const fs_tab_entry* tab_main, const fs_tab_entry* tab_tail) {
  float x = fs_background(c, row_key, v, tab_main, tab_tail);
  for (int j = 0; j < p->n_planted; ++j) {
    if (v == p->tok[j]) {
      if (!p->is_fork && c->peak_mode == FS_PEAK_ADD) x = fs_add(x, p->val[j]);
      else x = p->val[j];
    }
  }
  return x;
}

/* ---- host library (fork_synth_cpu.c) ---- */
/* Builds (once) and returns the two quantile tables; each has FS_TAB_N entries. */
void fork_synth_tables(const fs_tab_entry** tab_main, const fs_tab_entry** tab_tail);
/* Writes row (step,b,l) as V elements of cfg->dtype into out (host memory). */
void fork_synth_row_host(const fork_synth_cfg* cfg, uint32_t nonce, int32_t step, int32_t b, int32_t l, void* out);
/* Fills every live row (mask[b,k]!=0, lo[b]<=k<hi[b]) of a host logits buffer laid out
   [B, Ll, V] with strides (elements) and window origin pos0; other rows are left untouched.
   nthreads<=0 uses all host cores. Returns the number of rows written. */
int64_t fork_synth_fill_host(const fork_synth_cfg* cfg, uint32_t nonce, int32_t step,
                             const uint8_t* mask, const int32_t* lo, const int32_t* hi,
                             void* logits, int64_t stride_b, int64_t stride_l, int32_t pos0, int32_t Ll,
                             int32_t nthreads);
void fork_synth_plan_host(const fork_synth_cfg* cfg, int32_t b, int32_t l, fs_row_plan* out);

#ifdef __cplusplus
}
#endif
#endif /* FORK_SYNTH_H */
