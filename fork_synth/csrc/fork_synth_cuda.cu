/*
 * Device side of the synthetic-logit generator (input making only; see fork_synth.h).
 * The rows written here are bit-identical to fork_synth_row_host(): same inline core, same
 * host-built quantile tables, every floating-point step a single correctly rounded operation.
 * Also provides the generator as a `fork_logits_fn`-shaped callback for a decode loop.
 * Build: nvcc -O3 -fmad=false -gencode arch=compute_100a,code=sm_100a -shared -Xcompiler -fPIC
 */
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "fork_synth.h"

static __device__ fs_tab_entry d_tab_main[FS_TAB_N];
static __device__ fs_tab_entry d_tab_tail[FS_TAB_N];
static bool g_inited[64];

extern "C" int fork_synth_cuda_init(const fs_tab_entry* tab_main, const fs_tab_entry* tab_tail) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return (int)e;
  if (dev >= 0 && dev < 64 && g_inited[dev]) return 0;
  e = cudaMemcpyToSymbol(d_tab_main, tab_main, sizeof(fs_tab_entry) * FS_TAB_N);
  if (e != cudaSuccess) return (int)e;
  e = cudaMemcpyToSymbol(d_tab_tail, tab_tail, sizeof(fs_tab_entry) * FS_TAB_N);
  if (e != cudaSuccess) return (int)e;
  e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return (int)e;
  if (dev >= 0 && dev < 64) g_inited[dev] = true;
  return 0;
}

#define FS_SPLIT 8   /* CTAs per row */

__global__ void __launch_bounds__(256) fill_kernel(fork_synth_cfg cfg, uint32_t nonce, int32_t step,
                                                   const uint8_t* __restrict__ mask, const int32_t* __restrict__ lo,
                                                   const int32_t* __restrict__ hi, void* logits, long long stride_b,
                                                   long long stride_l, int32_t pos0, int32_t Ll) {
  const int b = blockIdx.z, j = blockIdx.y, k = pos0 + j;
  if (k >= cfg.Lt) return;
  const int l0 = lo ? lo[b] : 0, h0 = hi ? hi[b] : cfg.Lt;
  if (k < l0 || k >= h0 || !mask[(size_t)b * cfg.Lt + k]) return;
  __shared__ fs_row_plan plan;
  if (threadIdx.x == 0) fs_plan_row(&cfg, b, k, &plan);
  __syncthreads();
  const uint64_t key = fs_row_key(cfg.seed, nonce, step, b, k);
  const long long base = (long long)b * stride_b + (long long)j * stride_l;
  const int per = (cfg.V + FS_SPLIT - 1) / FS_SPLIT;
  const int v0 = blockIdx.x * per;
  int v1 = v0 + per; if (v1 > cfg.V) v1 = cfg.V;
  if (cfg.dtype == FS_BF16) {
    uint16_t* o = (uint16_t*)logits + base;
    for (int v = v0 + threadIdx.x; v < v1; v += blockDim.x)
      o[v] = fs_f32_to_bf16(fs_logit(&cfg, &plan, key, v, d_tab_main, d_tab_tail));
  } else {
    float* o = (float*)logits + base;
    for (int v = v0 + threadIdx.x; v < v1; v += blockDim.x)
      o[v] = fs_logit(&cfg, &plan, key, v, d_tab_main, d_tab_tail);
  }
}

/* Fill every live row of a device logits buffer; all pointers are device pointers. */
extern "C" int fork_synth_cuda_fill(const fork_synth_cfg* cfg, uint32_t nonce, int32_t step, const uint8_t* mask,
                                    const int32_t* lo, const int32_t* hi, void* logits, int64_t stride_b,
                                    int64_t stride_l, int32_t pos0, int32_t Ll, void* stream) {
  if (cfg->B <= 0 || Ll <= 0) return 0;
  if (cfg->B > 65535 || Ll > 65535) return (int)cudaErrorInvalidValue;
  dim3 grid(FS_SPLIT, (unsigned)Ll, (unsigned)cfg->B);
  fill_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(*cfg, nonce, step, mask, lo, hi, logits, (long long)stride_b,
                                                      (long long)stride_l, pos0, Ll);
  return (int)cudaGetLastError();
}

__global__ void canary_kernel(void* p, long long n, int dtype) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long stride = (long long)gridDim.x * blockDim.x;
  if (dtype == FS_BF16) { uint16_t* o = (uint16_t*)p; for (; i < n; i += stride) o[i] = 0x7FC0; }
  else { uint32_t* o = (uint32_t*)p; for (; i < n; i += stride) o[i] = 0x7FC00000u; }
}

/* NaN in every element: a read of a row that is not live then poisons the result. */
extern "C" int fork_synth_cuda_canary(void* logits, int64_t n_elems, int32_t dtype, void* stream) {
  if (n_elems <= 0) return 0;
  canary_kernel<<<148 * 8, 256, 0, (cudaStream_t)stream>>>(logits, (long long)n_elems, dtype);
  return (int)cudaGetLastError();
}

/* ---- the generator as the decode loop's model-forward callback ---------------------------- */
struct fork_synth_provider_ctx {
  fork_synth_cfg cfg;
  int64_t stride_b, stride_l;
  int32_t pos0, Ll;
  uint32_t* nonce;      /* per-step nonce (host), may be NULL */
  int32_t n_nonce;
  int64_t calls;
  int32_t fail_at;      /* step at which the callback reports failure, -1 = never */
};

extern "C" void* fork_synth_provider_create(const fork_synth_cfg* cfg, int64_t stride_b, int64_t stride_l,
                                            int32_t pos0, int32_t Ll, const uint32_t* nonce, int32_t n_nonce) {
  fork_synth_provider_ctx* c = (fork_synth_provider_ctx*)calloc(1, sizeof(fork_synth_provider_ctx));
  if (!c) return NULL;
  c->cfg = *cfg; c->stride_b = stride_b; c->stride_l = stride_l; c->pos0 = pos0; c->Ll = Ll;
  c->n_nonce = 0; c->nonce = NULL; c->calls = 0; c->fail_at = -1;
  if (nonce && n_nonce > 0) {
    c->nonce = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)n_nonce);
    memcpy(c->nonce, nonce, sizeof(uint32_t) * (size_t)n_nonce);
    c->n_nonce = n_nonce;
  }
  return c;
}

extern "C" void fork_synth_provider_destroy(void* ctx) {
  fork_synth_provider_ctx* c = (fork_synth_provider_ctx*)ctx;
  if (!c) return;
  free(c->nonce);
  free(c);
}

extern "C" int64_t fork_synth_provider_calls(void* ctx) { return ((fork_synth_provider_ctx*)ctx)->calls; }
extern "C" void fork_synth_provider_fail_at(void* ctx, int32_t step) { ((fork_synth_provider_ctx*)ctx)->fail_at = step; }

/* Signature of fork_logits_fn (include/fork_dllm.h). */
extern "C" int fork_synth_provider(void* ctx, int32_t step, const int32_t* tokens, const uint8_t* mask,
                                   const int32_t* blk_lo, const int32_t* blk_hi, void* logits_out, void* stream) {
  fork_synth_provider_ctx* c = (fork_synth_provider_ctx*)ctx;
  (void)tokens;
  c->calls += 1;
  if (c->fail_at >= 0 && step >= c->fail_at) return 7;
  uint32_t nonce = (c->nonce && step >= 0 && step < c->n_nonce) ? c->nonce[step] : 0u;
  return fork_synth_cuda_fill(&c->cfg, nonce, step, mask, blk_lo, blk_hi, logits_out, c->stride_b, c->stride_l,
                              c->pos0, c->Ll, stream);
}
