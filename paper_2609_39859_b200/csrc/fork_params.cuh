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

/* kModeSample: a step with stochastic candidates (tau > 0); kModeVp / kModeVpSample: the local phase
   of the vocabulary-parallel step (per-position parts for the exchange instead of the unmask rule).
   Instances of their own, so that no kernel carries finalisation code it never runs: the
   streaming loops share the SM's instruction cache with whatever else the kernel contains. */
enum Mode { kModeStep = 0, kModeLogprob = 1, kModeSample = 2, kModeVp = 3, kModeVpSample = 4, kModeCount = 5 };
__host__ __device__ constexpr bool mode_is_step(int mode) { return mode != kModeLogprob; }
__host__ __device__ constexpr bool mode_is_sample(int mode) { return mode == kModeSample || mode == kModeVpSample; }
__host__ __device__ constexpr bool mode_is_vp(int mode) { return mode == kModeVp || mode == kModeVpSample; }

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

/* ---- decode loop: state the steps of a loop hand on to one another on the device -------------
 * The block cursors are double buffered: step i of a loop reads lo/hi[i & 1] (they are the step's
 * block bounds) and writes lo/hi[(i + 1) & 1] -- every sequence's finaliser its own cursor, after
 * its commits (the same block, or the next block that still holds a masked position), and whoever
 * handles the sequences without a live row copies theirs -- so nothing a CTA of the step still has
 * to read is ever modified.  `remaining` counts the sequences that still hold a masked position;
 * `seq_done` counts the sequences dealt with in the current step, and whoever brings it to B puts
 * it back to zero and reports (ticket0 + i, remaining) to the host through flags[i % kLoopFlags],
 * eight bytes of pinned host memory that the host polls instead of synchronising the stream. */
constexpr int kLoopFlags = 8;
struct LoopCtl {
  int32_t remaining, seq_done;
  int32_t gen_lo, gen_hi, block_len, step0;
  uint32_t ticket0; int32_t pad;
  unsigned long long* flags;
  int32_t* lo[2]; int32_t* hi[2];
};

struct VpPeerTable { float4* part[FORK_VP_MAX_RANKS]; float4* key[FORK_VP_MAX_RANKS]; };

/* splits x row blocks of the fused LM-head step never exceed max(SMs, row blocks): room for 160 SMs */
constexpr size_t kHeadPartsExtra = 128 * 161;

struct WsView {
  WsHeader* hdr;
  int32_t* seq_off;                  /* [B+1] first row of each sequence */
  int32_t* expected;                 /* [B] parts the sequence will receive */
  int32_t* ticket;                   /* [B] parts received so far */
  int32_t* loop_lo[2];               /* [B] decode-loop block cursors, double buffered */
  int32_t* loop_hi[2];               /* [B] */
  LoopCtl* loop;                     /* decode-loop state */
  int2* rows;                        /* [B*Lt] (b, k) of each live row, ascending */
  float4* final_rec;                 /* [B*Lt] per-row results kept between the finaliser's passes */
  float4* parts;                     /* [B*Lt + FORK_MAX_GRID] partial results, slot r+g */
  uint32_t* commit_bits;             /* [B * ceil(Lt/32)] positions committed by a step whose mask update was handed on */
  VpPeerTable* vp_peer_tab;          /* gather-buffer addresses of a vocabulary-parallel reduction with the exchange fused in */
  float4* head_parts;                /* [splits][row blocks * 128] per-row results of the fused LM-head step, one per vocabulary split */
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
  for (int i = 0; i < 2; ++i) {
    v.loop_lo[i] = (int32_t*)(p + off); off = align_up(off + nb * 4, 256);
    v.loop_hi[i] = (int32_t*)(p + off); off = align_up(off + nb * 4, 256);
  }
  v.loop = (LoopCtl*)(p + off); off = align_up(off + sizeof(LoopCtl), 256);
  v.rows = (int2*)(p + off); off = align_up(off + rows * sizeof(int2), 256);
  v.final_rec = (float4*)(p + off); off = align_up(off + rows * sizeof(float4), 256);
  v.parts = (float4*)(p + off); off = align_up(off + (rows + FORK_MAX_GRID) * sizeof(float4), 256);
  v.commit_bits = (uint32_t*)(p + off); off = align_up(off + nb * (size_t)(((Lt > 0 ? Lt : 1) + 31) / 32) * 4, 256);
  v.vp_peer_tab = (VpPeerTable*)(p + off); off = align_up(off + sizeof(VpPeerTable), 256);
  v.head_parts = (float4*)(p + off); off = align_up(off + (rows + kHeadPartsExtra) * sizeof(float4), 256);
  v.bytes = off;
  return v;
}

/* ---- one-kernel step: control block ------------------------------------------------------------
 * A step whose batch is small enough runs as ONE kernel: every virtual CTA of the streaming kernel
 * derives the active set itself from `mask` and the block bounds when it starts (its snapshot),
 * instead of reading the lists a set-up kernel would have written.  That needs state that is clean
 * when the kernel starts without a kernel before it to clean it: it lives in a control block that
 * the library owns (zero when the library is loaded, left clean by every launch), never in the
 * caller's workspace, whose bytes may be anything.
 *   started  : virtual CTAs that have taken their snapshot, summed over all launches.  Every virtual
 *              CTA of a launch adds one, so between launches it is a multiple of the launch size and
 *              "all of this launch have their snapshot" reads started % size == 0.  No sequence's
 *              mask is modified before that holds (a CTA that starts late must still see M_t).
 *   ticket   : parts received per sequence; the last arriver puts it back to zero.
 *   deferred : set by a finaliser that found snapshots still missing: its mask update (positions in
 *              WsView::commit_bits) is applied by the CTA that counts itself last, or by itself if
 *              that has happened in the meantime; applying twice is harmless. */
constexpr int kFuseMaxB = 256;        /* sequences */
constexpr int kFuseMaxWords = 1024;   /* 32-position words of block window over all sequences */
constexpr int kFuseMaxSeqWords = 64;  /* ... and per sequence (a row look-up walks a sequence's words) */
struct FusedCtl {
  unsigned long long started;
  unsigned long long pad;
  int32_t ticket[kFuseMaxB];
  uint32_t deferred[kFuseMaxB];
};

/* ---- kernel parameters -------------------------------------------------------------------- */
struct RowSource {                   /* where the logits rows are */
  const void* logits;
  long long stride_b, stride_l;
  int pos0, Ll, V;
};

/* Every kernel of the library takes this block, and at the start of a launch -- cold caches, the
   critical path of every CTA -- each 64-byte line of it that is touched costs a trip to the constant
   cache's backing store: what the start of the streaming kernels reads comes first and together;
   what only the finalisation reads comes last. */
struct ReduceParams {
  /* read on the way to the first copy */
  RowSource src;
  int B, Lt, C, fast;
  FusedCtl* ctl; uint8_t* mask; const int32_t* blk_lo; const int32_t* blk_hi;   /* one-kernel step (ctl != NULL): control block, block bounds */
  int W, Gv, late_g;                 /* ... words per sequence of the window bitmaps, virtual CTAs of the launch, and
                                        late_g - 1 = a virtual CTA that dawdles before its snapshot (read by the test-only
                                        instance of the kernel alone; 0 = none) */
  int l2_evict_first;                /* bulk copies of logits carry the L2 "evict first" hint */
  const int32_t* vp_pos0_seq;        /* fused LM-head step: NULL, or [B] the position of row 0 of each sequence's window */
  const float4* head_draw;           /* fused LM-head step with drawn candidates: [window rows] (token, its logit, total, 0) */
  int min_units;                     /* small steps: units per participating CTA (fork_effective_grid) */
  LoopCtl* loop;                     /* a step of fork_decode_loop: where the cursors of the next step go (else NULL) */
  int vocab_offset;                  /* vocabulary-parallel slices: global index of entry 0 of this buffer */
  WsHeader* hdr; const int2* rows; const int32_t* seq_off; const int32_t* expected; int32_t* ticket;   /* workspace */
  float noise_c; int32_t step; unsigned long long sample_seed;   /* stochastic candidates: log2(e)/tau and the stream of uniforms */
  float inv_tau, raise_nats;         /* ... 1/tau, and how far above a thread's reference the running maximum may rise
                                        before the reference follows (keeps the tempered exponents in range) */
  /* read at segment ends and in the finalisation */
  float4* parts; float4* final_rec; uint32_t* commit_bits;
  /* candidates drawn at a temperature; all three in the caller's sample scratch */
  float* sslots;                     /* [B*Lt + FORK_MAX_GRID][kSlotStride] lane sums of the tempered weights of every part */
  int32_t* row_ticket;               /* [B*Lt] parts of a row that have arrived; zero between launches */
  float4* row_draw;                  /* [B*Lt] per live row: (drawn token, its logit, total of the tempered weights, -) */
  int32_t* tokens; float threshold; int fallback_mode; const uint32_t* fallback_rand;
  float* conf; int32_t* cand; float* entropy; float* logp; uint32_t* row_status;
  int32_t* commit_step; uint8_t* commit_fallback; float* commit_logp;
  int32_t* n_unmasked; uint8_t* is_fallback; int32_t* fallback_pos; int32_t* nfe; int32_t* n_fallback;
  /* vocabulary-parallel slices */
  float4* vp_part; float4* vp_key;   /* [B,Lt] local phase: per-position results for the exchange instead of the unmask rule */
  const float4* vp_parts_in; const float4* vp_keys_in; int vp_ranks;   /* select phase: gathered [ranks][B,Lt] */
  int vp_row_stride;                 /* > 0: the gathered parts are indexed [rank][b * Ll + (k - pos0)] with this many rows
                                        per rank (the fused LM-head step), not [rank][b * Lt + k] */
  /* local phase with the exchange fused in (vp_peers > 0): the gather buffers [vp_peers][B,Lt] of all
     ranks as this GPU addresses them (its own, and peer-mapped memory); slot vp_rank of each is
     written.  The addresses sit in the workspace, not here: the size of this block is felt at
     every launch. */
  const VpPeerTable* vp_peer_tab; int vp_rank, vp_peers;
  /* log-probability mode */
  const int32_t* lp_tokens; float* lp_out; float* seq_sum; int32_t* seq_cnt; float* lse_out;
};

/* Row r of the step -> (sequence, position).  Two-kernel step: the lists the set-up kernel wrote.
   One-kernel step: this group's snapshot in shared memory -- off[b] = first row of sequence b,
   bits[b*W + i] = live positions pos0 + 32 i .. pos0 + 32 i + 31 of sequence b. */
/* the snapshot lookups are rare (once per row segment) and kept out of line: inlined at every use
   they lengthen the streaming loops' code, which is what the instruction cache has to hold */
__device__ __noinline__ int snap_seq_of(const int32_t* off, int B, int r) {       /* the last b with off[b] <= r */
  int lo = 0, hi = B;
  while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (off[mid] <= r) lo = mid; else hi = mid; }
  return lo;
}
__device__ __noinline__ int snap_pos_of(const uint32_t* w, int W, int pos0, int j) {   /* position of live row j of a sequence */
  for (int i = 0; i < W; ++i) {
    const uint32_t x = w[i];
    const int n = __popc(x);
    if (j < n) return pos0 + 32 * i + (int)__fns(x, 0u, j + 1);
    j -= n;
  }
  return pos0;
}
struct RowMap {
  const int2* rows; const int32_t* seq_off;
  const int32_t* off; const uint32_t* bits; int B, W, pos0;
  const int* win_lo; const int* win_hi;   /* one-kernel step: the block windows as the snapshot holds them, or NULL when one of them had to be clipped */
  __device__ __forceinline__ int seq_of(int r) const { return snap_seq_of(off, B, r); }
  __device__ __forceinline__ int pos_of(int b, int j) const { return snap_pos_of(bits + b * W, W, pos0, j); }
  __device__ __forceinline__ int2 bk(int r) const {
    if (!off) return rows[r];
    const int b = seq_of(r);
    return make_int2(b, pos_of(b, r - off[b]));
  }
  __device__ __forceinline__ int k_of(int b, int r) const { return off ? pos_of(b, r - off[b]) : rows[r].y; }
  __device__ __forceinline__ void seq_range(int b, int& r0, int& r1) const {
    if (off) { r0 = off[b]; r1 = off[b + 1]; } else { r0 = seq_off[b]; r1 = seq_off[b + 1]; }
  }
};
__device__ __forceinline__ RowMap row_map_lists(const ReduceParams& p) {
  return RowMap{p.rows, p.seq_off, nullptr, nullptr, p.B, 0, p.src.pos0, nullptr, nullptr};
}

template <typename T>
__device__ __forceinline__ const T* row_ptr(const RowSource& s, int b, int k) {
  return reinterpret_cast<const T*>(s.logits) + ((long long)b * s.stride_b + (long long)(k - s.pos0) * s.stride_l);
}

__device__ __forceinline__ float4 ld_cg_f4(const float4* p) { return __ldcg(p); }

/* ---- decode loop: cursors of the next step, termination ------------------------------------- */
/* `n` more sequences of step p.step have been dealt with (by one thread).  The one that completes
   the batch leaves the counter clean and tells the host how many sequences still hold a masked
   position: one 8-byte store (ticket, remaining) into pinned host memory. */
__device__ __forceinline__ void loop_sequences_done(LoopCtl* L, int step, int B, int n) {
  int old;
  asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(&L->seq_done), "r"(n) : "memory");
  if (old + n == B) {
    L->seq_done = 0;
    int rem;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(rem) : "l"(&L->remaining) : "memory");
    const uint32_t i = (uint32_t)(step - L->step0);
    const unsigned long long v = ((unsigned long long)(uint32_t)rem << 32) | (unsigned long long)(L->ticket0 + i);
    *reinterpret_cast<volatile unsigned long long*>(L->flags + (i % kLoopFlags)) = v;   /* posted; nothing else for the host depends on it */
  }
}

/* The sequences without a live row in this step keep their cursors; `idle` of them, handled by
   the calling warp (lanes stride over b). */
__device__ __forceinline__ void loop_copy_idle_cursor(LoopCtl* L, int step, const int32_t* lo, const int32_t* hi, int b) {
  const int nxt = ((step - L->step0) + 1) & 1;
  L->lo[nxt][b] = lo[b]; L->hi[nxt][b] = hi[b];
}

/* ---- the partition as the kernels see it ---------------------------------------------------- */
struct PartitionCtx {
  long long U; int G; int C;
  bool small;                                    /* (U+1)*G < 2^32: 32-bit division is exact */
  __device__ __forceinline__ int owner(long long x) const {
    if (small) return (int)((((uint32_t)x + 1u) * (uint32_t)G - 1u) / (uint32_t)U);
    return fork_part_owner(U, G, x);
  }
};

__device__ __forceinline__ PartitionCtx make_partition(int R, int C, int grid, int min_units) {
  PartitionCtx c;
  c.U = (long long)R * C;
  c.G = fork_effective_grid(c.U, grid, min_units);
  c.C = C;
  c.small = (unsigned long long)(c.U + 1) * (unsigned long long)c.G < 0xffffffffull;
  return c;
}

}  // namespace forkd
