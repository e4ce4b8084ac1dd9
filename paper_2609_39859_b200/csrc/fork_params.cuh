/*
 * Workspace layout, kernel parameters and the work partition as the kernels of the Fork-dLLM
 * confidence pass see them.
 */
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/fork_dllm.h"
#include "fork_partition.h"
#include "fork_reduce.cuh"

namespace forkd {


constexpr int kNT = 256;             /* threads per CTA of the streaming kernel */
constexpr int kUnroll = 4;           /* 128-bit loads in flight per thread */
constexpr int kSetupNT = 1024;       /* threads of the one-CTA set-up kernels */

enum Mode { kModeStep = 0, kModeLogprob = 1, kModeSample = 2 };   /* kModeSample: a step with stochastic candidates (tau > 0) */
__host__ __device__ constexpr bool mode_is_step(int mode) { return mode != kModeLogprob; }

/* ---- workspace ---------------------------------------------------------------------------- */
struct WsHeader {                    /* 256 bytes at the start of the workspace */
  int32_t R;                         /* live rows of the current call */
  int32_t C;                         /* units per row */
  int32_t G;                         /* grid size the partition was computed for */
  uint32_t dev_status;               /* FORK_DEV_* bits */
  int32_t remaining;                 /* decode loop: sequences that still hold a masked position */
  int32_t pad[59];
};
static_assert(sizeof(WsHeader) == 256, "header size");

struct WsView {
  WsHeader* hdr;
  int32_t* seq_off;                  /* [B+1] first row of each sequence */
  int32_t* expected;                 /* [B] parts the sequence will receive */
  int32_t* ticket;                   /* [B] parts received so far */
  int32_t* loop_lo;                  /* [B] decode-loop block cursors */
  int32_t* loop_hi;                  /* [B] */
  int2* rows;                        /* [B*Lt] (b, k) of each live row, ascending */
  float4* final_rec;                 /* [B*Lt] per-row results kept between the finaliser's passes */
  float4* parts;                     /* [B*Lt + FORK_MAX_GRID] partial results, slot r+g */
  float2* kparts;                    /* [B*Lt + FORK_MAX_GRID] best perturbed key of each part (stochastic candidates) */
  size_t bytes;
};

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static WsView ws_view(void* base, int32_t B, int32_t Lt) {
  WsView v;
  char* p = (char*)base;
  size_t off = 0;
  const size_t nb = (size_t)(B > 0 ? B : 1), rows = nb * (size_t)(Lt > 0 ? Lt : 1);
  v.hdr = (WsHeader*)(p + off); off += sizeof(WsHeader);
  v.seq_off = (int32_t*)(p + off); off = align_up(off + (nb + 1) * 4, 256);
  v.expected = (int32_t*)(p + off); off = align_up(off + nb * 4, 256);
  v.ticket = (int32_t*)(p + off); off = align_up(off + nb * 4, 256);
  v.loop_lo = (int32_t*)(p + off); off = align_up(off + nb * 4, 256);
  v.loop_hi = (int32_t*)(p + off); off = align_up(off + nb * 4, 256);
  v.rows = (int2*)(p + off); off = align_up(off + rows * sizeof(int2), 256);
  v.final_rec = (float4*)(p + off); off = align_up(off + rows * sizeof(float4), 256);
  v.parts = (float4*)(p + off); off = align_up(off + (rows + FORK_MAX_GRID) * sizeof(float4), 256);
  v.kparts = (float2*)(p + off); off = align_up(off + (rows + FORK_MAX_GRID) * sizeof(float2), 256);
  v.bytes = off;
  return v;
}

/* ---- kernel parameters -------------------------------------------------------------------- */
struct RowSource {                   /* where the logits rows are */
  const void* logits;
  long long stride_b, stride_l;
  int pos0, Ll, V;
};

struct ReduceParams {
  RowSource src;
  int B, Lt, C, fast;
  /* workspace */
  const WsHeader* hdr; const int32_t* seq_off; const int32_t* expected; int32_t* ticket;
  const int2* rows; float4* final_rec; float4* parts; float2* kparts;
  /* step mode */
  int32_t* tokens; uint8_t* mask; float threshold; int32_t step;
  float* conf; int32_t* cand; float* entropy; float* logp; uint32_t* row_status;
  int32_t* commit_step; uint8_t* commit_fallback; float* commit_logp;
  int32_t* n_unmasked; uint8_t* is_fallback; int32_t* fallback_pos; int32_t* nfe; int32_t* n_fallback;
  int fallback_mode; const uint32_t* fallback_rand;
  float noise_c; unsigned long long sample_seed;      /* stochastic candidates: log2(e)/tau and the noise stream */
  /* vocabulary-parallel slices */
  int vocab_offset;                  /* global index of entry 0 of this buffer */
  float4* vp_part; float4* vp_key;   /* [B,Lt] local phase: per-position results for the exchange instead of the unmask rule */
  const float4* vp_parts_in; const float4* vp_keys_in; int vp_ranks;   /* select phase: gathered [ranks][B,Lt] */
  /* log-probability mode */
  const int32_t* lp_tokens; float* lp_out; float* seq_sum; int32_t* seq_cnt; float* lse_out;
};

template <typename T>
__device__ __forceinline__ const T* row_ptr(const RowSource& s, int b, int k) {
  return reinterpret_cast<const T*>(s.logits) + ((long long)b * s.stride_b + (long long)(k - s.pos0) * s.stride_l);
}

__device__ __forceinline__ float4 ld_cg_f4(const float4* p) { return __ldcg(p); }

/* ---- the partition as the kernels see it ---------------------------------------------------- */
struct PartitionCtx {
  long long U; int G; int C;
  bool small;                                    /* (U+1)*G < 2^32: 32-bit division is exact */
  __device__ __forceinline__ int owner(long long x) const {
    if (small) return (int)((((uint32_t)x + 1u) * (uint32_t)G - 1u) / (uint32_t)U);
    return fork_part_owner(U, G, x);
  }
};

__device__ __forceinline__ PartitionCtx make_partition(int R, int C, int grid) {
  PartitionCtx c;
  c.U = (long long)R * C;
  c.G = fork_effective_grid(c.U, grid);
  c.C = C;
  c.small = (unsigned long long)(c.U + 1) * (unsigned long long)c.G < 0xffffffffull;
  return c;
}

}  // namespace forkd
