/*
 * Kernels and C ABI of the Fork-dLLM confidence pass (see include/fork_dllm.h for the contract).
 *
 * A step is two launches on the caller's stream:
 *   1. active_set_kernel (one CTA): M_t restricted to each sequence's block (Algorithm 2, line 3)
 *      compacted into a row list, per-sequence row offsets, and the number of partial results each
 *      sequence will receive.  The row list is the step's snapshot of the mask: the second kernel
 *      never reads `mask` (which it modifies).
 *   2. reduce_select_kernel (persistent grid): streams every live row once (lines 4-5: arg-max
 *      candidate and its softmax probability, plus entropy), and the CTA that delivers the last
 *      partial result of a sequence applies the unmask rule for it (lines 6-9: threshold set, or
 *      the leftmost masked position when that set is empty) and writes tokens, mask and records.
 * Cross-CTA hand-over uses "last one to arrive" ticket counters (fence + atomic): nothing in
 * here ever waits for another CTA.
 *
 * The same two kernels serve the log-likelihood scoring (Section 3.2), the step with candidates
 * drawn at a temperature (a third instance of the streaming kernels that also tracks the largest
 * Gumbel-perturbed key) and the local phase of the vocabulary-parallel step (the finaliser writes
 * per-position parts instead of applying the rule).  Small kernels of their own: block cursors of the
 * decode loop, the select phase on gathered parts, top-entropy position selection, the ForkGRPO
 * objective (Eq. 2) and the log-softmax backward at the scored rows.
 */
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <cstdio>
#include <cstring>

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

/* ---- kernel 1: the active set -------------------------------------------------------------- */
/* One CTA.  live(b,k) = flags[b,k] != 0 and k inside the sequence's window (block bounds clipped
   to the sequence buffer and to the positions the logits buffer covers). */
struct SetupParams {
  const uint8_t* flags;              /* mask (step) or select (log-probability) */
  const int32_t* lo; const int32_t* hi;   /* NULL: the whole sequence */
  int B, Lt, pos0, Ll, C, G;
  WsHeader* hdr; int32_t* seq_off; int32_t* expected; int32_t* ticket; int2* rows;
  /* outputs for sequences without a live row */
  int32_t* n_unmasked; uint8_t* is_fallback; int32_t* fallback_pos;   /* step mode */
  float* seq_sum; int32_t* seq_cnt;                                   /* log-probability mode */
};

__device__ __forceinline__ void seq_window(const SetupParams& p, int b, int& lo, int& hi, bool& clipped) {
  int l0 = p.lo ? p.lo[b] : 0, h0 = p.hi ? p.hi[b] : p.Lt;
  lo = l0; hi = h0;
  if (lo < 0) lo = 0;
  if (hi > p.Lt) hi = p.Lt;
  if (lo < p.pos0) lo = p.pos0;
  if (hi > p.pos0 + p.Ll) hi = p.pos0 + p.Ll;
  clipped = (h0 > l0) && (lo != l0 || hi != h0);
  if (hi < lo) hi = lo;
}

constexpr int kSetupMaxB = 4096;     /* sequences whose counts fit in shared memory (more: counts go through global memory) */

__global__ void __launch_bounds__(kSetupNT, 1) active_set_kernel(SetupParams p) {
  /* with programmatic dependent launch this grid may already be resident while the kernel before
     it in the stream (normally the previous step) is still running: nothing is read or written
     before that kernel has completed; the streaming kernel of this step may be made resident now */
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;");
  __shared__ int sh_cnt[kSetupMaxB + 1];          /* sh_cnt[b+1] = live rows of b, then their inclusive scan */
  __shared__ int sh_warp[kSetupNT / 32];
  __shared__ int sh_carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = kSetupNT / 32;
  int* cnt = (p.B <= kSetupMaxB) ? sh_cnt : p.seq_off;       /* cnt[0..B] */
  unsigned clipped_any = 0;

  /* pass 1: live rows per sequence */
  for (int b = warp; b < p.B; b += nwarp) {
    int lo, hi; bool clipped;
    seq_window(p, b, lo, hi, clipped);
    clipped_any |= clipped ? 1u : 0u;
    int n = 0;
    for (int k0 = lo; k0 < hi; k0 += 32) {
      int k = k0 + lane;
      bool live = (k < hi) && p.flags[(size_t)b * p.Lt + k] != 0;
      n += __popc(__ballot_sync(0xffffffffu, live));
    }
    if (lane == 0) { cnt[b + 1] = n; p.ticket[b] = 0; }
  }
  if (tid == 0) { cnt[0] = 0; sh_carry = 0; }
  __syncthreads();

  /* pass 2: inclusive scan of the counts, kSetupNT sequences at a time */
  for (int base = 0; base < p.B; base += kSetupNT) {
    int b = base + tid;
    int x = (b < p.B) ? cnt[b + 1] : 0;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { int y = __shfl_up_sync(0xffffffffu, x, o); if (lane >= o) x += y; }
    if (lane == 31) sh_warp[warp] = x;
    __syncthreads();
    if (warp == 0) {
      int w = sh_warp[lane];
      int xs = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { int y = __shfl_up_sync(0xffffffffu, xs, o); if (lane >= o) xs += y; }
      sh_warp[lane] = xs - w;                       /* exclusive prefix of the warp totals */
    }
    __syncthreads();
    int incl = sh_carry + sh_warp[warp] + x;
    if (b < p.B) cnt[b + 1] = incl;
    __syncthreads();
    if (tid == kSetupNT - 1) sh_carry = incl;
    __syncthreads();
  }
  const int R = sh_carry;
  const PartitionCtx c = make_partition(R, p.C, p.G);
  if (tid == 0) {
    p.hdr->R = R; p.hdr->C = p.C; p.hdr->G = c.G;
  }

  /* pass 3: row list, expected part counts, outputs of idle sequences */
  for (int b = warp; b < p.B; b += nwarp) {
    int lo, hi; bool clipped;
    seq_window(p, b, lo, hi, clipped);
    const int r0 = cnt[b], r1 = cnt[b + 1];
    int run = r0;
    for (int k0 = lo; k0 < hi; k0 += 32) {
      int k = k0 + lane;
      bool live = (k < hi) && p.flags[(size_t)b * p.Lt + k] != 0;
      unsigned bal = __ballot_sync(0xffffffffu, live);
      if (live) p.rows[run + __popc(bal & ((1u << lane) - 1u))] = make_int2(b, k);
      run += __popc(bal);
    }
    int parts = 0;
    for (int r = r0 + lane; r < r1; r += 32)
      parts += c.owner((long long)(r + 1) * c.C - 1) - c.owner((long long)r * c.C) + 1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) parts += __shfl_down_sync(0xffffffffu, parts, o);
    if (lane == 0) {
      p.expected[b] = parts;
      if (cnt == sh_cnt) { p.seq_off[b + 1] = r1; if (b == 0) p.seq_off[0] = 0; }
      if (r0 == r1) {
        if (p.n_unmasked) p.n_unmasked[b] = 0;
        if (p.is_fallback) p.is_fallback[b] = 0;
        if (p.fallback_pos) p.fallback_pos[b] = -1;
        if (p.seq_sum) p.seq_sum[b] = 0.f;
        if (p.seq_cnt) p.seq_cnt[b] = 0;
      }
    }
  }
  clipped_any = __syncthreads_or((int)clipped_any);
  if (tid == 0) p.hdr->dev_status = clipped_any ? FORK_DEV_WINDOW_CLAMPED : 0u;
}

/* ---- shared by both streaming kernels: merging parts, the unmask rule, scoring ------------- */
__device__ __forceinline__ Part part_from(const float4& v) { return Part{v.x, v.y, v.z, __float_as_int(v.w)}; }

constexpr int kLaneMergeMax = 24;
/* Parts of row r, by one lane, loaded four at a time and merged in ascending CTA order.  `n`
   returns how many parts the row has; rows with more than kLaneMergeMax (very few live rows, the
   whole grid on them) are merged by merge_row_parts_warp instead. */
__device__ __forceinline__ Part merge_row_parts(const ReduceParams& p, const PartitionCtx& c, int r, int& g0, int& n) {
  g0 = c.owner((long long)r * c.C);
  const int g1 = c.owner((long long)(r + 1) * c.C - 1);
  n = g1 - g0 + 1;
  const float4* q = p.parts + (r + g0);
  const float4 v0 = ld_cg_f4(q);
  float4 v1 = v0, v2 = v0, v3 = v0;
  if (n > 1) v1 = ld_cg_f4(q + 1);
  if (n > 2) v2 = ld_cg_f4(q + 2);
  if (n > 3) v3 = ld_cg_f4(q + 3);
  Part acc = part_from(v0);
  if (n > 1) acc = part_merge(acc, part_from(v1));
  if (n > 2) acc = part_merge(acc, part_from(v2));
  if (n > 3) acc = part_merge(acc, part_from(v3));
  if (n <= kLaneMergeMax) {                                  /* a moderate number: this lane goes on, four loads at a time */
    for (int j = 4; j < n; j += 4) {
      const float4 w0 = ld_cg_f4(q + j);
      float4 w1 = w0, w2 = w0, w3 = w0;
      if (j + 1 < n) w1 = ld_cg_f4(q + j + 1);
      if (j + 2 < n) w2 = ld_cg_f4(q + j + 2);
      if (j + 3 < n) w3 = ld_cg_f4(q + j + 3);
      acc = part_merge(acc, part_from(w0));
      if (j + 1 < n) acc = part_merge(acc, part_from(w1));
      if (j + 2 < n) acc = part_merge(acc, part_from(w2));
      if (j + 3 < n) acc = part_merge(acc, part_from(w3));
    }
  }
  return acc;
}

/* A row cut into many parts (few live rows, many CTAs): the whole warp loads 32 parts at a time
   and tree-merges them; every lane returns the same Part. */
__device__ __forceinline__ Part merge_row_parts_warp(const ReduceParams& p, int r, int g0, int n) {
  const int lane = threadIdx.x & 31;
  const float4* q = p.parts + (r + g0);
  Part acc = part_empty();
  for (int j0 = 0; j0 < n; j0 += 32) {
    Part x = (j0 + lane < n) ? part_from(ld_cg_f4(q + j0 + lane)) : part_empty();
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      Part y;
      y.m = __shfl_xor_sync(0xffffffffu, x.m, o); y.s = __shfl_xor_sync(0xffffffffu, x.s, o);
      y.t = __shfl_xor_sync(0xffffffffu, x.t, o); y.idx = __shfl_xor_sync(0xffffffffu, x.idx, o);
      const bool low = (lane & o) == 0;                      /* both partners compute merge(lower, upper) */
      x = low ? part_merge(x, y) : part_merge(y, x);
    }
    acc = part_merge(acc, x);
  }
  return acc;
}

/* Guarded scalar reduction of a whole row by ONE warp (every lane returns the same Part). */
template <typename T>
__device__ Part careful_row_warp(const T* row, int V, bool& bad, bool* nonfinite = nullptr) {
  const int lane = threadIdx.x & 31;
  float m = -INFINITY;
  int idx = -1, isbad = 0;
  for (int i = lane; i < V; i += 32) {
    const float x = to_f32(row[i]);
    if (x != x) { isbad = 1; continue; }
    if (x == INFINITY) isbad = 1;
    if (idx < 0 || x > m) { m = x; idx = i; }
  }
  if (idx < 0) idx = kIdxNone;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, m, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    const bool take = (oi != kIdxNone) && (idx == kIdxNone || om > m || (om == m && oi < idx));
    if (take) { m = om; idx = oi; }
  }
  isbad = __any_sync(0xffffffffu, isbad);
  if (nonfinite) *nonfinite = isbad != 0;                    /* NaN or +inf seen (as opposed to nothing but -inf) */
  if (isbad || idx == kIdxNone || m == -INFINITY) {
    bad = true;
    return Part{m, __int_as_float(0x7fc00000), __int_as_float(0x7fc00000), idx == kIdxNone ? 0 : idx};
  }
  bad = false;
  float s = 0.f, t = 0.f;
  for (int i = lane; i < V; i += 32) {
    const float x = to_f32(row[i]);
    if (x == -INFINITY) continue;
    const float y = (x - m) * kLog2e;
    const float e = exp2f(y);
    s += e;
    if (e > 0.f) t = fmaf(y, e, t);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { s += __shfl_xor_sync(0xffffffffu, s, o); t += __shfl_xor_sync(0xffffffffu, t, o); }
  return Part{m, s, t, idx};
}

__device__ __forceinline__ KeyPart key_from(const float2& v) { return KeyPart{v.x, __float_as_int(v.y)}; }

/* Largest perturbed key of row r over its n parts (slots r+g0 ...), by one lane. */
__device__ __forceinline__ KeyPart merge_row_keys(const ReduceParams& p, int r, int g0, int n) {
  const float2* q = p.kparts + (r + g0);
  KeyPart acc = key_empty();
#pragma unroll 4
  for (int j = 0; j < n; ++j) acc = key_merge(acc, key_from(__ldcg(q + j)));
  return acc;
}

/* Final statistics of up to 32 rows (one per lane) of sequence b starting at row `base`.
   Rows whose streamed result is not finite are re-read by the whole warp with the guarded routine.
   With SAMPLE the candidate is the drawn token (the element holding the row's largest perturbed
   key) and confidence / log-probability are those of that token; flagged rows keep the arg-max. */
/* Rows base .. base+31 of sequence b, one per lane: the row's parts merged, rows whose streamed
   result is not finite re-read by the whole warp with the guarded routine. */
struct MergedRow {
  Part merged; int k, g0, nparts; bool valid, bad, nonfinite;
};
template <typename T>
__device__ __forceinline__ MergedRow merge_rows_warp(const ReduceParams& p, const PartitionCtx& c, int b, int base, int r1,
                                                     int k_hint) {
  const int lane = threadIdx.x & 31;
  const int r = base + lane;
  MergedRow m;
  m.valid = r < r1; m.bad = false; m.nonfinite = false;
  m.merged = part_empty();
  m.k = 0; m.g0 = 0; m.nparts = 0;
  bool redo = false;
  if (m.valid) { m.k = (k_hint >= 0) ? k_hint : p.rows[r].y; m.merged = merge_row_parts(p, c, r, m.g0, m.nparts); }
  unsigned many = __ballot_sync(0xffffffffu, m.valid && m.nparts > kLaneMergeMax);
  while (many) {                                             /* rows cut into very many parts: all lanes help */
    const int src = __ffs(many) - 1;
    many &= many - 1;
    const Part w = merge_row_parts_warp(p, __shfl_sync(0xffffffffu, r, src), __shfl_sync(0xffffffffu, m.g0, src),
                                        __shfl_sync(0xffffffffu, m.nparts, src));
    if (lane == src) m.merged = w;
  }
  if (m.valid) redo = part_needs_careful(m.merged);
  unsigned todo = __ballot_sync(0xffffffffu, m.valid && redo);
  while (todo) {
    const int src = __ffs(todo) - 1;
    todo &= todo - 1;
    const int kk = __shfl_sync(0xffffffffu, m.k, src);
    bool bd, nf;
    const Part cp = careful_row_warp<T>(row_ptr<T>(p.src, b, kk), p.src.V, bd, &nf);
    if (lane == src) { m.merged = cp; m.bad = bd; m.nonfinite = nf; }
  }
  return m;
}

template <typename T, bool WANT_INDEX, bool SAMPLE>
__device__ __forceinline__ RowOut finalize_rows_warp(const ReduceParams& p, const PartitionCtx& c, int b, int base,
                                                     int r1, Part& merged, int& k, int k_hint) {
  const int lane = threadIdx.x & 31;
  const int r = base + lane;
  MergedRow m = merge_rows_warp<T>(p, c, b, base, r1, k_hint);
  k = m.k;
  if (SAMPLE) {
    float xs = 0.f;
    if (m.valid && !m.bad) {
      const KeyPart kp = merge_row_keys(p, r, m.g0, m.nparts);
      const NoiseRow nz = noise_row(p.sample_seed, p.step, b, k, p.noise_c, (uint32_t)p.vocab_offset);
      m.merged.idx = resolve_sample<T>(row_ptr<T>(p.src, b, k), nz, kp.vec, p.src.V, kp.key, xs);
    }
    merged = m.merged;
    return row_out_sampled(merged, m.bad, xs);
  }
  if (m.valid && WANT_INDEX && !m.bad) m.merged.idx = resolve_index<T>(row_ptr<T>(p.src, b, k), m.merged.idx, p.src.V, m.merged.m);
  merged = m.merged;
  return row_out_from(merged, m.bad);
}

/* What a finaliser can load about a sequence BEFORE its last part arrives (it idles until then):
   the sequence's row range and this lane's position among its first 32 rows. */
struct SeqHint { int r0, r1, k; };
__device__ __forceinline__ SeqHint load_seq_hint(const ReduceParams& p, int b) {
  SeqHint h;
  h.r0 = p.seq_off[b]; h.r1 = p.seq_off[b + 1];
  const int r = h.r0 + (int)(threadIdx.x & 31);
  h.k = (r < h.r1) ? p.rows[r].y : -1;
  return h;
}

/* ---- vocabulary-parallel slices ------------------------------------------------------------- */
/* Local phase: what this slice contributes to every live row of sequence b, written per position
   for the exchange: (m, s, t2, global index of the lowest arg-max), s = NaN when the slice holds
   NaN or +inf, the neutral element (m = -inf, s = t2 = 0) when it holds nothing but -inf; with
   stochastic candidates also (largest perturbed key, global index of its entry, that logit). */
template <typename T, bool SAMPLE>
__device__ void finalize_vp_local(const ReduceParams& p, const PartitionCtx& c, int b, const SeqHint& h) {
  const int lane = threadIdx.x & 31;
  const float qnan = __int_as_float(0x7fc00000);
  for (int base = h.r0; base < h.r1; base += 32) {
    const int r = base + lane;
    MergedRow m = merge_rows_warp<T>(p, c, b, base, h.r1, base == h.r0 ? h.k : -1);
    if (!m.valid) continue;
    const size_t at = (size_t)b * p.Lt + m.k;
    const T* row = row_ptr<T>(p.src, b, m.k);
    float4 out, kout = make_float4(-INFINITY, __int_as_float(kIdxNone), 0.f, 0.f);
    if (m.bad && !m.nonfinite) {
      out = make_float4(-INFINITY, 0.f, 0.f, __int_as_float(p.vocab_offset));
    } else if (m.bad) {
      out = make_float4(m.merged.m, qnan, qnan, __int_as_float(p.vocab_offset + m.merged.idx));
    } else {
      const int idx = resolve_index<T>(row, m.merged.idx, p.src.V, m.merged.m);
      out = make_float4(m.merged.m, m.merged.s, m.merged.t, __int_as_float(p.vocab_offset + idx));
      if (SAMPLE) {
        const KeyPart kp = merge_row_keys(p, r, m.g0, m.nparts);
        const NoiseRow nz = noise_row(p.sample_seed, p.step, b, m.k, p.noise_c, (uint32_t)p.vocab_offset);
        float xs;
        const int si = resolve_sample<T>(row, nz, kp.vec, p.src.V, kp.key, xs);
        kout = make_float4(kp.key, __int_as_float(p.vocab_offset + si), xs, 0.f);
      }
    }
    p.vp_part[at] = out;
    if (SAMPLE) p.vp_key[at] = kout;
  }
}

/* Select phase: the statistics of rows base .. base+31 of sequence b from the gathered slices,
   merged in rank order (ascending vocabulary offset; ties keep the lowest global index). */
template <bool SAMPLE>
__device__ __forceinline__ RowOut gathered_rows_warp(const ReduceParams& p, int b, int base, int r1, int& k, int k_hint) {
  const int lane = threadIdx.x & 31;
  const int r = base + lane;
  k = 0;
  if (r >= r1) return row_out_from(part_empty(), true);
  k = (k_hint >= 0) ? k_hint : p.rows[r].y;
  const size_t at = (size_t)b * p.Lt + k, n = (size_t)p.B * p.Lt;
  Part acc = part_empty();
  for (int j = 0; j < p.vp_ranks; ++j) acc = part_merge(acc, part_from(__ldg(p.vp_parts_in + j * n + at)));
  const bool bad = !(isfinite(acc.s) && isfinite(acc.t)) || !(acc.m > -INFINITY) || acc.m == INFINITY;
  if (!SAMPLE || bad) return row_out_from(acc, bad);
  float best = -INFINITY, xs = 0.f;
  int bidx = kIdxNone;
  for (int j = 0; j < p.vp_ranks; ++j) {
    const float4 q = __ldg(p.vp_keys_in + j * n + at);
    const int qi = __float_as_int(q.y);
    if (q.x > best || (q.x == best && qi < bidx)) { best = q.x; bidx = qi; xs = q.z; }
  }
  acc.idx = bidx;
  return row_out_sampled(acc, false, xs);
}

/* Key by which a fallback step ranks a row under the orders other than "leftmost" (the largest key
   wins, equal keys go to the lower row): the confidence (Algorithm 1), its negative, or the token
   entropy (the ablations of Section 4.1).  Flagged rows rank below every other row. */
__device__ __forceinline__ float fallback_key(int mode, float conf, float entropy, bool bad) {
  if (bad) return -INFINITY;
  return mode == FORK_FALLBACK_MAX_CONF ? conf : (mode == FORK_FALLBACK_MIN_CONF ? -conf : entropy);
}

/* The unmask rule for one sequence, run by one warp once every part of the sequence has arrived
   (Algorithm 2 lines 6-9): commit every live position whose confidence exceeds lambda, or one
   position when none does -- the leftmost live one (Fork-dLLM), or the one the requested
   comparison order picks; write tokens, mask and the per-token records. */
template <typename T, bool SAMPLE, bool GATHERED = false>
__device__ void finalize_step_sequence(const ReduceParams& p, const PartitionCtx& c, int b, const SeqHint& h) {
  const int lane = threadIdx.x & 31;
  const int r0 = h.r0, r1 = h.r1;
  const bool one_batch = (r1 - r0) <= 32;                    /* the usual case: results stay in registers */
  const bool ranked = p.fallback_mode >= FORK_FALLBACK_MAX_CONF && p.fallback_mode <= FORK_FALLBACK_MAX_ENTROPY;
  int any = 0;
  float4 keep = make_float4(0.f, 0.f, 0.f, 0.f);
  int keep_k = 0;
  float best_key = -INFINITY;                                /* this lane's best row under a ranked order */
  int best_r = 0x7fffffff;
  for (int base = r0; base < r1; base += 32) {
    Part merged; int k;
    const RowOut o = GATHERED ? gathered_rows_warp<SAMPLE>(p, b, base, r1, k, base == r0 ? h.k : -1)
                              : finalize_rows_warp<T, true, SAMPLE>(p, c, b, base, r1, merged, k, base == r0 ? h.k : -1);
    const int r = base + lane;
    if (r < r1) {
      const size_t at = (size_t)b * p.Lt + k;
      if (p.conf) p.conf[at] = o.conf;
      if (p.cand) p.cand[at] = o.cand;
      if (p.entropy) p.entropy[at] = o.entropy;
      if (p.logp) p.logp[at] = o.logp;
      if (p.row_status) p.row_status[at] = o.status;
      keep = make_float4(o.conf, o.logp, __int_as_float(o.cand), 0.f);
      keep_k = k;
      if (!one_batch) p.final_rec[r] = keep;
      any |= (o.conf > p.threshold) ? 1 : 0;                 /* U_t non-empty (Algorithm 2, line 6) */
      if (ranked) {
        const float key = fallback_key(p.fallback_mode, o.conf, o.entropy, o.status != 0u);
        if (key > best_key) { best_key = key; best_r = r; }  /* rows ascend within a lane: strict > keeps the lower */
      }
    }
  }
  any = __any_sync(0xffffffffu, any);
  const int fb = any ? 0 : 1;                                /* fallback step: max_k c <= lambda */
  int pick = r0;                                             /* leftmost(M_t) inside the block */
  if (fb && ranked) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ok = __shfl_xor_sync(0xffffffffu, best_key, o);
      const int orow = __shfl_xor_sync(0xffffffffu, best_r, o);
      if (ok > best_key || (ok == best_key && orow < best_r)) { best_key = ok; best_r = orow; }
    }
    if (best_key > -INFINITY) pick = best_r;                 /* every row flagged: stay with the leftmost */
  } else if (fb && p.fallback_mode == FORK_FALLBACK_RANDOM) {
    pick = r0 + (int)(p.fallback_rand[b] % (uint32_t)(r1 - r0));
  }
  int count = 0, pick_k = -1;
  for (int base = r0; base < r1; base += 32) {
    const int r = base + lane;
    bool commit = false;
    if (r < r1) {
      const float4 f = one_batch ? keep : p.final_rec[r];    /* written by this same lane above */
      commit = fb ? (r == pick) : (f.x > p.threshold);       /* the fallback position, or the threshold set */
      if (commit) {
        const int k = one_batch ? keep_k : p.rows[r].y;
        const size_t at = (size_t)b * p.Lt + k;
        if (fb) pick_k = k;
        p.tokens[at] = __float_as_int(f.z);
        p.mask[at] = 0;
        if (p.commit_step) p.commit_step[at] = p.step;
        if (p.commit_fallback) p.commit_fallback[at] = (uint8_t)fb;
        if (p.commit_logp) p.commit_logp[at] = f.y;
      }
    }
    count += __popc(__ballot_sync(0xffffffffu, commit));
  }
  if (fb) {                                                  /* exactly one lane committed: tell lane 0 where */
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) pick_k = max(pick_k, __shfl_xor_sync(0xffffffffu, pick_k, o));
  }
  if (lane == 0) {
    if (p.n_unmasked) p.n_unmasked[b] = count;
    if (p.is_fallback) p.is_fallback[b] = (uint8_t)fb;
    if (p.fallback_pos) p.fallback_pos[b] = pick_k;
    /* reductions without a return value: no load at the very end of the step to wait for */
    if (p.nfe) atomicAdd(p.nfe + b, 1);
    if (p.n_fallback && fb) atomicAdd(p.n_fallback + b, 1);
  }
}

/* Scoring for one sequence by one warp: log q(token) = x_tok - m - ln s at every selected position
   and their sum (Section 3.2 of the paper: the likelihood terms of the ForkGRPO ratio). */
template <typename T>
__device__ void finalize_logprob_sequence(const ReduceParams& p, const PartitionCtx& c, int b, const SeqHint& h) {
  const int lane = threadIdx.x & 31;
  const int r0 = h.r0, r1 = h.r1;
  float local = 0.f;
  for (int base = r0; base < r1; base += 32) {
    Part merged; int k;
    const RowOut o = finalize_rows_warp<T, false, false>(p, c, b, base, r1, merged, k, base == r0 ? h.k : -1);
    const int r = base + lane;
    if (r < r1) {
      const size_t at = (size_t)b * p.Lt + k;
      const int tok = p.lp_tokens[at];
      uint32_t st = o.status;
      float lp;
      if (tok < 0 || tok >= p.src.V) { st |= FORK_ROW_BAD_TOKEN; lp = 0.f; }
      else if (o.status) lp = o.logp;                        /* NaN for a non-finite row */
      else lp = (to_f32(row_ptr<T>(p.src, b, k)[tok]) - merged.m) + o.logp;   /* x_tok - m - ln s */
      p.lp_out[at] = lp;
      if (p.lse_out) p.lse_out[at] = o.status ? o.logp : merged.m - o.logp;   /* m + ln s; NaN for a flagged row */
      if (p.row_status) p.row_status[at] = st;
      local += lp;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) local += __shfl_xor_sync(0xffffffffu, local, o);
  if (lane == 0) {
    if (p.seq_sum) p.seq_sum[b] = local;
    if (p.seq_cnt) p.seq_cnt[b] = r1 - r0;
  }
}

/* Lane 0 of the calling warp publishes one part of row r (sequence b) and takes a ticket; returns
   (to every lane) whether this was the last part the sequence was waiting for. */
__device__ __forceinline__ bool publish_part(const ReduceParams& p, const Part& part, int r, int g, int b, int want,
                                             const KeyPart* kp = nullptr) {
  int last = 0;
  if ((threadIdx.x & 31) == 0) {
    p.parts[r + g] = make_float4(part.m, part.s, part.t, __int_as_float(part.idx));
    if (kp) p.kparts[r + g] = make_float2(kp->key, __int_as_float(kp->vec));
    int old;                                 /* release our part, acquire everybody else's */
    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(p.ticket + b) : "memory");
    last = (old + 1 == want) ? 1 : 0;
  }
  return __shfl_sync(0xffffffffu, last, 0) != 0;
}

/* The rows a CTA works on: its contiguous unit range cut at row boundaries. */
struct Segment { int r, e0, e1; };
struct SegmentIter {
  long long u, u1; int C, V;
  __device__ __forceinline__ void init(const PartitionCtx& c, int g, int V_) {
    u = fork_part_begin(c.U, c.G, g); u1 = fork_part_begin(c.U, c.G, g + 1); C = c.C; V = V_;
  }
  __device__ __forceinline__ bool next(Segment& s) {
    if (u >= u1) return false;
    s.r = (u < 0x7fffffffLL) ? (int)((uint32_t)u / (uint32_t)C) : (int)(u / C);
    const int c0 = (int)(u - (long long)s.r * C);
    long long uend = (long long)(s.r + 1) * C;
    if (uend > u1) uend = u1;
    const int c1 = (int)(uend - (long long)s.r * C);
    s.e0 = c0 * FORK_CHUNK;
    s.e1 = c1 * FORK_CHUNK;
    if (s.e1 > V) s.e1 = V;
    u = uend;
    return true;
  }
};

/* ---- kernel 2a: direct 128-bit loads (also the path for buffers that are not 16-byte aligned) -- */
struct Smem {
  Part parts[kNT / 32];
  KeyPart keys[kNT / 32];
  float fl[kNT / 32];
  int flag;
};

template <typename T, int MODE>
__global__ void __launch_bounds__(kNT, 4) reduce_select_kernel(ReduceParams p) {
  constexpr bool WITH_T = mode_is_step(MODE);
  constexpr bool SAMPLE = (MODE == kModeSample);
  __shared__ Smem sm;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;");
  const int R = p.hdr->R;
  if (R <= 0) return;
  const PartitionCtx c = make_partition(R, p.C, (int)gridDim.x);
  const int g = blockIdx.x;
  if (g >= c.G) return;                                     /* CTAs beyond the number of units have no work */
  SegmentIter it;
  it.init(c, g, p.src.V);
  Segment sg;
  bool sticky = false;
  while (it.next(sg)) {
    const int2 bk = p.rows[sg.r];
    const T* row = row_ptr<T>(p.src, bk.x, bk.y);
    Part part;
    KeyTrack kt;
    kt.init();
    NoiseRow nz = NoiseRow{0u, 0u, 0.f, 0u};
    if (SAMPLE) nz = noise_row(p.sample_seed, p.step, bk.x, bk.y, p.noise_c, (uint32_t)p.vocab_offset);
    if (p.fast) {
      part = part_block_reduce<kNT>(
          stream_thread<T, WITH_T, kNT, kUnroll, SAMPLE>(row, sg.e0, sg.e1, threadIdx.x, threadIdx.x == 0, sticky, &kt, &nz),
          sm.parts);
    } else {
      bool bad;
      part = careful_segment<T, kNT>(row, sg.e0, sg.e1, sm.parts, sm.fl, bad);
      if (SAMPLE)
        for (int i = sg.e0 + (int)threadIdx.x; i < sg.e1; i += kNT) kt.one(nz, to_f32(row[i]), i);
    }
    KeyPart kp = key_empty();
    if (SAMPLE) kp = key_block_reduce<kNT>(kt.best, sm.keys);
    if (threadIdx.x < 32) {
      const bool last = publish_part(p, part, sg.r, g, bk.x, p.expected[bk.x], SAMPLE ? &kp : nullptr);
      if (last) {                                           /* every part of sequence b has been delivered */
        const SeqHint h = load_seq_hint(p, bk.x);
        if (MODE == kModeLogprob) finalize_logprob_sequence<T>(p, c, bk.x, h);
        else if (p.vp_part) finalize_vp_local<T, SAMPLE>(p, c, bk.x, h);
        else finalize_step_sequence<T, SAMPLE>(p, c, bk.x, h);
      }
    }
  }
}

/* ---- kernel 2b: bulk-copy (TMA) shared-memory ring, warp-specialised --------------------------
 * Warps 0..kCW-1 consume, warp kCW produces, warp kCW+1 finalises.
 *   producer : one lane walks the CTA's segments and issues cp.async.bulk copies of up to one stage
 *              (kStageBytes) into a ring of shared-memory stages, each guarded by a full/empty
 *              mbarrier pair; it runs ahead of the consumers by the depth of the ring, across row
 *              boundaries, so HBM requests never drain while rows are being wrapped up.
 *   consumers: wait for a stage, read their 128-bit vectors from shared memory, accumulate, release
 *              the stage; at the end of a row segment each warp shuffle-reduces its threads' Parts
 *              and hands ONE Part to the finaliser through a small mbarrier-guarded mailbox, then
 *              goes straight on to the next segment.
 *   finaliser: merges the kCW warp Parts, publishes the CTA's part of the row, takes the sequence's
 *              ticket and, if it was the last, applies the unmask rule for that sequence.
 * Every mbarrier wait is bounded: after kSpinLimit failed polls the thread records
 * FORK_DEV_TIMEOUT in the workspace header and leaves its loop.                                   */
constexpr int kCW = 8;                                     /* consumer warps per CTA */
constexpr int kMaxCW = kCW;
constexpr int kMail = 4;                                   /* mailbox depth (row segments in flight to the finaliser) */
constexpr int kMaxStages = 13;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr int ring_stage_bytes() { return kCW * 32 * kUnroll * 16; }     /* 16 KB */

struct RingSmem {
  unsigned long long full[kMaxStages], empty[kMaxStages], mfull[kMail], mempty[kMail];
  Part mail[kMail][kMaxCW];
  KeyPart kmail[kMail][kMaxCW];
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
/* bounded wait; false (and a status bit in the workspace header) if the phase never completed */
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity, const ReduceParams& p) {
  for (uint32_t i = 0; i < kSpinLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  atomicOr(const_cast<uint32_t*>(&p.hdr->dev_status), FORK_DEV_TIMEOUT);
  return false;
}
__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, uint32_t bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               :: "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}


template <typename T, int MODE, int kPerSM>
__global__ void __launch_bounds__((kCW + 2) * 32, kPerSM) reduce_select_ring_kernel(ReduceParams p, int n_stages) {
  constexpr bool WITH_T = mode_is_step(MODE);
  constexpr bool SAMPLE = (MODE == kModeSample);
  constexpr int VEC = 16 / (int)sizeof(T);
  constexpr int kCT = kCW * 32;                              /* consumer threads */
  constexpr int kStageVecs = kCT * kUnroll;                  /* 128-bit vectors per stage */
  constexpr int kStageBytes = kStageVecs * 16;
  extern __shared__ __align__(1024) unsigned char dyn_smem[];
  unsigned char* ring = dyn_smem;
  RingSmem& rs = *reinterpret_cast<RingSmem*>(dyn_smem + (size_t)n_stages * kStageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) { mbar_init(&rs.full[s], 1); mbar_init(&rs.empty[s], kCW); }
    for (int d = 0; d < kMail; ++d) { mbar_init(&rs.mfull[d], kCW); mbar_init(&rs.mempty[d], 1); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;");          /* the next kernel in the stream may take free SM slots */
  const int R = p.hdr->R;
  if (R <= 0) return;
  const PartitionCtx c = make_partition(R, p.C, (int)gridDim.x);
  const int g = blockIdx.x;
  if (g >= c.G) return;
  SegmentIter it;
  it.init(c, g, p.src.V);
  Segment sg;

  if (warp == kCW) {
    /* ---------------- producer ---------------- */
    if (lane != 0) return;
    uint32_t n = 0, s = 0, ph = 0;                           /* stages issued, ring slot, its phase */
    bool ok = true;
    while (ok && it.next(sg)) {
      const int2 bk = p.rows[sg.r];
      const char* src = reinterpret_cast<const char*>(row_ptr<T>(p.src, bk.x, bk.y) + sg.e0);
      const uint32_t total = (uint32_t)((sg.e1 - sg.e0) / VEC) * 16u;
      for (uint32_t off = 0; off < total; off += kStageBytes, ++n) {
        const uint32_t bytes = (total - off < (uint32_t)kStageBytes) ? (total - off) : (uint32_t)kStageBytes;
        if (!mbar_wait(&rs.empty[s], ph ^ 1u, p)) { ok = false; break; }
        mbar_arrive_expect_tx(&rs.full[s], bytes);
        bulk_copy_g2s(ring + (size_t)s * kStageBytes, src + off, bytes, &rs.full[s]);
        if (++s == (uint32_t)n_stages) { s = 0; ph ^= 1u; }
      }
    }
    if (!ok) {                                               /* do not leave with copies still landing */
      const uint32_t first = n > (uint32_t)n_stages ? n - (uint32_t)n_stages : 0u;
      for (uint32_t q = first; q < n; ++q)
        mbar_wait(&rs.full[q % (uint32_t)n_stages], (q / (uint32_t)n_stages) & 1u, p);
    }
    return;
  }

  if (warp < kCW) {
    /* ---------------- consumers ---------------- */
    const int ctid = threadIdx.x;                           /* 0 .. kCT-1 */
    uint32_t s = 0, ph = 0, nseg = 0;                       /* ring slot, its phase, segments done */
    bool sticky = false;                                    /* this thread has met a -inf logit before */
    while (it.next(sg)) {
      Acc<T, WITH_T, false> a;
      a.init();
      KeyTrack kt;                                            /* stochastic candidates: largest perturbed key */
      kt.init();
      NoiseRow nz = NoiseRow{0u, 0u, 0.f, 0u};
      if (SAMPLE) { const int2 bk = p.rows[sg.r]; nz = noise_row(p.sample_seed, p.step, bk.x, bk.y, p.noise_c, (uint32_t)p.vocab_offset); }
      const int nvec = (sg.e1 - sg.e0) / VEC;
      for (int voff = 0; voff < nvec; voff += kStageVecs) {
        if (!mbar_wait(&rs.full[s], ph, p)) return;
        const uint4* sp = reinterpret_cast<const uint4*>(ring + (size_t)s * kStageBytes);
        const int nv = nvec - voff;
        if (nv >= kStageVecs) {
          /* a full stage: kUnroll vectors per thread; the stage is handed back to the producer as
             soon as the values sit in registers (track() has consumed every loaded word) */
          uint4 v[kUnroll];
#pragma unroll
          for (int j = 0; j < kUnroll; ++j) v[j] = sp[ctid + j * kCT];
          if (!sticky) a.template track<kUnroll>(v, sg.e0 + (voff + ctid) * VEC, kCT * VEC);
          __syncwarp();
          if (lane == 0) mbar_arrive(&rs.empty[s]);
          if (!sticky) a.template accumulate<kUnroll>(v);
          if (SAMPLE) kt.template update<kUnroll>(T{}, nz, v, sg.e0 + (voff + ctid) * VEC, kCT * VEC);
        } else {
          /* the last, partly filled stage of a segment: same unrolled code, vectors past the end
             replaced by the clamp value (contributes 2^-huge = 0 and never wins the maximum
             against a finite logit; an all -inf row is re-read by the finaliser anyway) */
          uint4 v[kUnroll];
#pragma unroll
          for (int j = 0; j < kUnroll; ++j)
            v[j] = (ctid + j * kCT < nv) ? sp[ctid + j * kCT] : neutral_vector(T{});
          if (!sticky) a.template track<kUnroll>(v, sg.e0 + (voff + ctid) * VEC, kCT * VEC);
          __syncwarp();
          if (lane == 0) mbar_arrive(&rs.empty[s]);
          if (!sticky) a.template accumulate<kUnroll>(v);
          if (SAMPLE) {                                       /* only the vectors that exist draw noise */
#pragma unroll
            for (int j = 0; j < kUnroll; ++j)
              if (ctid + j * kCT < nv) {
                const uint4 one[1] = {v[j]};
                kt.template update<1>(T{}, nz, one, sg.e0 + (voff + ctid + j * kCT) * VEC, kCT * VEC);
              }
          }
        }
        if (++s == (uint32_t)n_stages) { s = 0; ph ^= 1u; }
      }
      const bool tail = (ctid == 0) && (sg.e0 + nvec * VEC < sg.e1);   /* fewer than VEC trailing elements */
      Part pt;
      if (tail && (SAMPLE || !sticky)) {
        const int2 bk = p.rows[sg.r];
        const T* row = row_ptr<T>(p.src, bk.x, bk.y);
        for (int e = sg.e0 + nvec * VEC; e < sg.e1; ++e) {
          const float x = to_f32(row[e]);
          if (!sticky) a.one(x, e);
          if (SAMPLE) kt.one(nz, x, e);
        }
      }
      if (!sticky) {
        pt = a.part();
        if (!part_is_finite(pt)) sticky = true;
      }
      /* a thread that met -inf (now or earlier) takes its own vectors again from global memory, clamped */
      if (sticky) {
        const int2 bk = p.rows[sg.r];
        pt = stream_thread_clamped<T, WITH_T, kCT>(row_ptr<T>(p.src, bk.x, bk.y), sg.e0, sg.e1, ctid, ctid == 0);
      }
      __syncwarp();
      pt = part_warp_reduce(pt);
      KeyPart kp = key_empty();
      if (SAMPLE) kp = key_warp_reduce(kt.best);
      if (lane == 0) {
        const uint32_t d = nseg % kMail, mph = (nseg / kMail) & 1u;
        if (mbar_wait(&rs.mempty[d], mph ^ 1u, p)) {
          rs.mail[d][warp] = pt;
          if (SAMPLE) rs.kmail[d][warp] = kp;
          mbar_arrive(&rs.mfull[d]);
        }
      }
      ++nseg;
    }
    return;
  }

  /* ---------------- finaliser ---------------- */
  uint32_t nseg = 0;
  while (it.next(sg)) {
    /* everything that does not depend on the parts is fetched while the consumers still stream */
    const int b = p.rows[sg.r].x;
    const int want = p.expected[b];
    const SeqHint h = load_seq_hint(p, b);
    const uint32_t d = nseg % kMail, ph = (nseg / kMail) & 1u;
    if (!mbar_wait(&rs.mfull[d], ph, p)) return;
    Part pt = (lane < kCW) ? rs.mail[d][lane] : part_empty();
    KeyPart kp = key_empty();
    if (SAMPLE && lane < kCW) kp = rs.kmail[d][lane];
    __syncwarp();
    if (lane == 0) mbar_arrive(&rs.mempty[d]);
    pt = part_warp_reduce(pt);
    if (SAMPLE) kp = key_warp_reduce(kp);
    if (publish_part(p, pt, sg.r, g, b, want, SAMPLE ? &kp : nullptr)) {
      if (MODE == kModeLogprob) finalize_logprob_sequence<T>(p, c, b, h);
      else if (p.vp_part) finalize_vp_local<T, SAMPLE>(p, c, b, h);
      else finalize_step_sequence<T, SAMPLE>(p, c, b, h);
    }
    ++nseg;
  }
}

/* ---- vocabulary-parallel select phase: one warp per sequence on the gathered slices ---------- */
constexpr int kVpNT = 256;
template <bool SAMPLE>
__global__ void __launch_bounds__(kVpNT) vp_select_kernel(ReduceParams p) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int b = (int)blockIdx.x * (kVpNT / 32) + (int)(threadIdx.x >> 5);
  if (b >= p.B) return;
  const SeqHint h = load_seq_hint(p, b);
  if (h.r1 <= h.r0) return;                                  /* no live row: the active-set kernel wrote its outputs */
  PartitionCtx c;
  c.U = 0; c.G = 1; c.C = 1; c.small = true;
  finalize_step_sequence<float, SAMPLE, true>(p, c, b, h);
}

/* ---- decode-loop helpers ------------------------------------------------------------------- */
struct CursorParams {
  const uint8_t* mask; int B, Lt, gen_lo, gen_hi, block_len;
  int32_t* lo; int32_t* hi; WsHeader* hdr; int init;
};

/* One warp per sequence: the first block at or after the current one that holds a masked
   position; lo = hi = gen_hi when there is none.  hdr->remaining counts unfinished sequences. */
__global__ void __launch_bounds__(kSetupNT, 1) block_cursor_kernel(CursorParams p) {
  __shared__ int sh_remaining;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = kSetupNT / 32;
  if (tid == 0) sh_remaining = 0;
  __syncthreads();
  for (int b = warp; b < p.B; b += nwarp) {
    int from = p.gen_lo;
    if (!p.init) { int cur = p.lo[b]; if (cur >= p.gen_lo && cur < p.gen_hi) from = cur; }
    int found_lo = p.gen_hi, found_hi = p.gen_hi;
    for (int s = from; s < p.gen_hi; s += p.block_len) {
      int e = s + p.block_len; if (e > p.gen_hi) e = p.gen_hi;
      unsigned any = 0;
      for (int k0 = s; k0 < e; k0 += 32) {
        int k = k0 + lane;
        any |= __ballot_sync(0xffffffffu, (k < e) && p.mask[(size_t)b * p.Lt + k] != 0);
      }
      if (any) { found_lo = s; found_hi = e; break; }
    }
    if (lane == 0) {
      p.lo[b] = found_lo; p.hi[b] = found_hi;
      if (found_lo < found_hi) atomicAdd(&sh_remaining, 1);
    }
  }
  __syncthreads();
  if (tid == 0) p.hdr->remaining = sh_remaining;
}

}  // namespace forkd

/* =============================================================================================
 *  Host side: argument checks, launch configuration, the C ABI
 * ============================================================================================= */
using namespace forkd;

static std::atomic<long long> g_launches{0};
static std::atomic<int> g_tune[FORK_TUNE_COUNT_];

static size_t ring_smem_bytes(int n_stages) { return (size_t)n_stages * ring_stage_bytes() + sizeof(RingSmem); }

/* The bulk-copy kernel runs two CTAs per SM (8 consumer warps and 6 stages of 16 KB each).  Three
   CTAs with registers capped at 64 and 4 stages, or two with 12 consumer warps, measured the same
   on the large shapes and slightly worse on the small one. */
constexpr int kRingPerSM = 2;
static void ring_config(int* n_stages) {
  int st = g_tune[FORK_TUNE_STAGES].load();
  const int max_st = (int)((220 * 1024 / kRingPerSM - sizeof(RingSmem) - 1024) / ring_stage_bytes());
  if (st <= 0 || st > max_st) st = max_st;
  if (st > kMaxStages) st = kMaxStages;
  if (st < 2) st = 2;
  *n_stages = st;
}

struct DeviceInfo { int sms = 0; int occ[2][3] = {{0, 0, 0}, {0, 0, 0}}; bool ring_ready = false; };
static DeviceInfo g_dev[64];

template <typename T, int MODE>
static int occupancy_of() {
  int n = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, reduce_select_kernel<T, MODE>, kNT, 0) != cudaSuccess) n = 0;
  return n;
}

static bool device_info(DeviceInfo** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
  DeviceInfo& d = g_dev[dev];
  if (d.sms == 0) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return false;
    d.occ[0][0] = occupancy_of<bf16_t, kModeStep>();
    d.occ[0][1] = occupancy_of<bf16_t, kModeLogprob>();
    d.occ[1][0] = occupancy_of<float, kModeStep>();
    d.occ[1][1] = occupancy_of<float, kModeLogprob>();
    d.occ[0][2] = occupancy_of<bf16_t, kModeSample>();
    d.occ[1][2] = occupancy_of<float, kModeSample>();
    const int max_dyn = 220 * 1024;
    auto allow = [&](const void* fn) { return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, max_dyn) == cudaSuccess; };
    d.ring_ready =
        allow((const void*)reduce_select_ring_kernel<bf16_t, kModeStep, kRingPerSM>) &&
        allow((const void*)reduce_select_ring_kernel<bf16_t, kModeLogprob, kRingPerSM>) &&
        allow((const void*)reduce_select_ring_kernel<bf16_t, kModeSample, kRingPerSM>) &&
        allow((const void*)reduce_select_ring_kernel<float, kModeStep, kRingPerSM>) &&
        allow((const void*)reduce_select_ring_kernel<float, kModeLogprob, kRingPerSM>) &&
        allow((const void*)reduce_select_ring_kernel<float, kModeSample, kRingPerSM>);
    if (!d.ring_ready) return false;
    d.sms = sms;
  }
  *out = &d;
  return true;
}

static int grid_size(const DeviceInfo& d, int dtype, int mode, bool fast) {
  const int variant = g_tune[FORK_TUNE_VARIANT].load();
  if (fast && (variant == 0 || variant == 2)) {
    return d.sms * kRingPerSM;
  }
  int per_sm = g_tune[FORK_TUNE_CTAS_PER_SM].load();
  int occ = d.occ[dtype][mode];
  if (occ <= 0) occ = 1;
  if (per_sm <= 0 || per_sm > occ) per_sm = occ;
  long long G = (long long)d.sms * per_sm;
  if (G > FORK_MAX_GRID) G = FORK_MAX_GRID;
  return (int)G;
}

static bool bad_source(const void* logits, int64_t sb, int64_t sl, int32_t pos0, int32_t B, int32_t Lt,
                       int32_t Ll, int32_t V, int32_t dtype) {
  if (!logits || B < 0 || Lt <= 0 || Ll <= 0 || V <= 0 || pos0 < 0) return true;
  if (dtype != FORK_BF16 && dtype != FORK_F32) return true;
  if (sl < V || sb < 0) return true;
  if ((int64_t)B * Lt > (int64_t)1 << 30) return true;
  return false;
}

static bool source_is_vector_aligned(const void* logits, int64_t sb, int64_t sl, int32_t dtype) {
  const int64_t es = dtype == FORK_BF16 ? 2 : 4;
  return ((uintptr_t)logits % 16 == 0) && ((sb * es) % 16 == 0) && ((sl * es) % 16 == 0);
}

template <typename KernelT, typename ParamT>
static cudaError_t launch(KernelT kernel, dim3 grid, dim3 block, cudaStream_t st, bool pdl, const ParamT& prm) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = 0; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  if (pdl) {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
  }
  cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, prm);
  if (e == cudaSuccess) g_launches.fetch_add(1);
  return e;
}

static thread_local cudaEvent_t t_ev_start = nullptr, t_ev_stop = nullptr;

static cudaError_t launch_reduce_inner(const ReduceParams& rp, int dtype, int mode, int G, cudaStream_t st);

/* the streaming kernel, bracketed by the caller's events when fork_set_timing_events armed them */
static cudaError_t launch_reduce(const ReduceParams& rp, int dtype, int mode, int G, cudaStream_t st) {
  cudaEvent_t e0 = t_ev_start, e1 = t_ev_stop;
  t_ev_start = t_ev_stop = nullptr;
  if (e0 && cudaEventRecord(e0, st) != cudaSuccess) return cudaErrorUnknown;
  cudaError_t e = launch_reduce_inner(rp, dtype, mode, G, st);
  if (e == cudaSuccess && e1 && cudaEventRecord(e1, st) != cudaSuccess) return cudaErrorUnknown;
  return e;
}

template <typename T, int MODE, int PER_SM>
static cudaError_t launch_ring(const ReduceParams& rp, int G, int n_stages, bool pdl, cudaStream_t st) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(G); cfg.blockDim = dim3((kCW + 2) * 32); cfg.dynamicSmemBytes = ring_smem_bytes(n_stages);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  if (pdl) {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
  }
  cudaError_t e = cudaLaunchKernelEx(&cfg, reduce_select_ring_kernel<T, MODE, PER_SM>, rp, n_stages);
  if (e == cudaSuccess) g_launches.fetch_add(1);
  return e;
}

template <typename T, int PER_SM>
static cudaError_t launch_ring_mode(const ReduceParams& rp, int mode, int G, int n_stages, bool pdl, cudaStream_t st) {
  if (mode == kModeSample) return launch_ring<T, kModeSample, PER_SM>(rp, G, n_stages, pdl, st);
  if (mode == kModeStep) return launch_ring<T, kModeStep, PER_SM>(rp, G, n_stages, pdl, st);
  return launch_ring<T, kModeLogprob, PER_SM>(rp, G, n_stages, pdl, st);
}

/* variant 2 (bulk-copy ring) needs 16-byte aligned rows; everything else takes variant 1 */
static bool use_ring(const ReduceParams& rp) {
  const int v = g_tune[FORK_TUNE_VARIANT].load();
  return rp.fast && (v == 0 || v == 2);
}

static cudaError_t launch_reduce_inner(const ReduceParams& rp, int dtype, int mode, int G, cudaStream_t st) {
  const bool pdl = g_tune[FORK_TUNE_PDL].load() >= 0;
  if (use_ring(rp)) {
    int n_stages;
    ring_config(&n_stages);
    if (dtype == FORK_BF16) return launch_ring_mode<bf16_t, kRingPerSM>(rp, mode, G, n_stages, pdl, st);
    return launch_ring_mode<float, kRingPerSM>(rp, mode, G, n_stages, pdl, st);
  }
  if (mode == kModeSample) {
    if (dtype == FORK_BF16) return launch(reduce_select_kernel<bf16_t, kModeSample>, dim3(G), dim3(kNT), st, pdl, rp);
    return launch(reduce_select_kernel<float, kModeSample>, dim3(G), dim3(kNT), st, pdl, rp);
  }
  if (dtype == FORK_BF16) {
    if (mode == kModeStep) return launch(reduce_select_kernel<bf16_t, kModeStep>, dim3(G), dim3(kNT), st, pdl, rp);
    return launch(reduce_select_kernel<bf16_t, kModeLogprob>, dim3(G), dim3(kNT), st, pdl, rp);
  }
  if (mode == kModeStep) return launch(reduce_select_kernel<float, kModeStep>, dim3(G), dim3(kNT), st, pdl, rp);
  return launch(reduce_select_kernel<float, kModeLogprob>, dim3(G), dim3(kNT), st, pdl, rp);
}

extern "C" size_t fork_workspace_bytes(int32_t B, int32_t Lt) {
  if (B < 0 || Lt <= 0) return 0;
  return ws_view(nullptr, B, Lt).bytes;
}

extern "C" const char* fork_status_string(int s) {
  switch (s) {
    case FORK_OK: return "FORK_OK";
    case FORK_ERR_INVALID_ARG: return "FORK_ERR_INVALID_ARG";
    case FORK_ERR_CUDA: return "FORK_ERR_CUDA";
    case FORK_ERR_WORKSPACE: return "FORK_ERR_WORKSPACE";
    case FORK_ERR_MAX_STEPS: return "FORK_ERR_MAX_STEPS";
    case FORK_ERR_PROVIDER: return "FORK_ERR_PROVIDER";
    default: return "FORK_UNKNOWN_STATUS";
  }
}

extern "C" int32_t fork_set_tuning(int32_t key, int32_t value) {
  if (key < 0 || key >= FORK_TUNE_COUNT_) return -1;
  return g_tune[key].exchange(value);
}

extern "C" int64_t fork_kernel_launches(void) { return g_launches.load(); }

extern "C" void fork_set_timing_events(void* start, void* stop) {
  t_ev_start = (cudaEvent_t)start;
  t_ev_stop = (cudaEvent_t)stop;
}

static fork_status check_workspace(void* ws, size_t bytes, int32_t B, int32_t Lt) {
  if (!ws || ((uintptr_t)ws % 256) != 0) return FORK_ERR_WORKSPACE;
  if (bytes < fork_workspace_bytes(B, Lt)) return FORK_ERR_WORKSPACE;
  return FORK_OK;
}

struct VpLocal { int32_t vocab_offset; float4* part; float4* key; };

static fork_status step_impl(const fork_step_args* a, const int32_t* lo, const int32_t* hi, void* ws,
                             cudaStream_t st, const VpLocal* vp = nullptr) {
  DeviceInfo* dev;
  if (!device_info(&dev)) return FORK_ERR_CUDA;
  WsView w = ws_view(ws, a->B, a->Lt);
  const int mode = a->temperature > 0.f ? kModeSample : kModeStep;
  const bool fast = source_is_vector_aligned(a->logits, a->stride_b, a->stride_l, a->dtype);
  const int G = grid_size(*dev, a->dtype, mode, fast);
  const int C = (a->V + FORK_CHUNK - 1) / FORK_CHUNK;

  SetupParams sp;
  memset(&sp, 0, sizeof(sp));
  sp.flags = a->mask; sp.lo = lo; sp.hi = hi;
  sp.B = a->B; sp.Lt = a->Lt; sp.pos0 = a->pos0; sp.Ll = a->Ll; sp.C = C; sp.G = G;
  sp.hdr = w.hdr; sp.seq_off = w.seq_off; sp.expected = w.expected; sp.ticket = w.ticket; sp.rows = w.rows;
  if (!vp) { sp.n_unmasked = a->n_unmasked; sp.is_fallback = a->is_fallback; sp.fallback_pos = a->fallback_pos; }
  if (launch(active_set_kernel, dim3(1), dim3(kSetupNT), st, g_tune[FORK_TUNE_PDL].load() >= 0, sp) != cudaSuccess) return FORK_ERR_CUDA;

  ReduceParams rp;
  memset(&rp, 0, sizeof(rp));
  rp.src = RowSource{a->logits, (long long)a->stride_b, (long long)a->stride_l, a->pos0, a->Ll, a->V};
  rp.B = a->B; rp.Lt = a->Lt; rp.C = C;
  rp.fast = fast ? 1 : 0;
  rp.hdr = w.hdr; rp.seq_off = w.seq_off; rp.expected = w.expected; rp.ticket = w.ticket;
  rp.rows = w.rows; rp.final_rec = w.final_rec; rp.parts = w.parts; rp.kparts = w.kparts;
  rp.noise_c = mode == kModeSample ? (float)(1.4426950408889634 / (double)a->temperature) : 0.f;
  rp.sample_seed = a->sample_seed;
  rp.tokens = a->tokens; rp.mask = a->mask; rp.threshold = a->threshold; rp.step = a->step;
  rp.conf = a->conf; rp.cand = a->cand; rp.entropy = a->entropy; rp.logp = a->logp; rp.row_status = a->row_status;
  rp.commit_step = a->commit_step; rp.commit_fallback = a->commit_fallback; rp.commit_logp = a->commit_logp;
  rp.n_unmasked = a->n_unmasked; rp.is_fallback = a->is_fallback; rp.fallback_pos = a->fallback_pos;
  rp.nfe = a->nfe; rp.n_fallback = a->n_fallback;
  rp.fallback_mode = a->fallback_mode; rp.fallback_rand = a->fallback_rand;
  if (vp) { rp.vocab_offset = vp->vocab_offset; rp.vp_part = vp->part; rp.vp_key = vp->key; }
  if (launch_reduce(rp, a->dtype, mode, G, st) != cudaSuccess) return FORK_ERR_CUDA;
  return FORK_OK;
}

static fork_status check_step_args(const fork_step_args* a, bool need_bounds) {
  if (!a) return FORK_ERR_INVALID_ARG;
  if (bad_source(a->logits, a->stride_b, a->stride_l, a->pos0, a->B, a->Lt, a->Ll, a->V, a->dtype))
    return FORK_ERR_INVALID_ARG;
  if (!a->tokens || !a->mask) return FORK_ERR_INVALID_ARG;
  if (need_bounds && (!a->blk_lo || !a->blk_hi)) return FORK_ERR_INVALID_ARG;
  if (a->threshold != a->threshold) return FORK_ERR_INVALID_ARG;      /* NaN threshold */
  if (a->fallback_mode < FORK_FALLBACK_LEFTMOST || a->fallback_mode > FORK_FALLBACK_RANDOM) return FORK_ERR_INVALID_ARG;
  if (a->fallback_mode == FORK_FALLBACK_RANDOM && !a->fallback_rand) return FORK_ERR_INVALID_ARG;
  if (!(a->temperature >= 0.f) || a->temperature > 3.0e38f) return FORK_ERR_INVALID_ARG;
  return FORK_OK;
}

extern "C" fork_status fork_step(const fork_step_args* a, void* ws, size_t ws_bytes, void* stream) {
  fork_status s = check_step_args(a, true);
  if (s != FORK_OK) return s;
  s = check_workspace(ws, ws_bytes, a->B, a->Lt);
  if (s != FORK_OK) return s;
  if (a->B == 0) return FORK_OK;
  return step_impl(a, a->blk_lo, a->blk_hi, ws, (cudaStream_t)stream);
}

extern "C" fork_status fork_logprob(const fork_logprob_args* a, void* ws, size_t ws_bytes, void* stream) {
  if (!a) return FORK_ERR_INVALID_ARG;
  if (bad_source(a->logits, a->stride_b, a->stride_l, a->pos0, a->B, a->Lt, a->Ll, a->V, a->dtype))
    return FORK_ERR_INVALID_ARG;
  if (!a->tokens || !a->select || !a->logp) return FORK_ERR_INVALID_ARG;
  fork_status s = check_workspace(ws, ws_bytes, a->B, a->Lt);
  if (s != FORK_OK) return s;
  if (a->B == 0) return FORK_OK;
  cudaStream_t st = (cudaStream_t)stream;
  DeviceInfo* dev;
  if (!device_info(&dev)) return FORK_ERR_CUDA;
  WsView w = ws_view(ws, a->B, a->Lt);
  const int mode = kModeLogprob;
  const bool fast = source_is_vector_aligned(a->logits, a->stride_b, a->stride_l, a->dtype);
  const int G = grid_size(*dev, a->dtype, mode, fast);
  const int C = (a->V + FORK_CHUNK - 1) / FORK_CHUNK;
  if (cudaMemsetAsync(a->logp, 0, sizeof(float) * (size_t)a->B * a->Lt, st) != cudaSuccess) return FORK_ERR_CUDA;

  SetupParams sp;
  memset(&sp, 0, sizeof(sp));
  sp.flags = a->select; sp.lo = nullptr; sp.hi = nullptr;
  sp.B = a->B; sp.Lt = a->Lt; sp.pos0 = a->pos0; sp.Ll = a->Ll; sp.C = C; sp.G = G;
  sp.hdr = w.hdr; sp.seq_off = w.seq_off; sp.expected = w.expected; sp.ticket = w.ticket; sp.rows = w.rows;
  sp.seq_sum = a->seq_sum; sp.seq_cnt = a->seq_cnt;
  if (launch(active_set_kernel, dim3(1), dim3(kSetupNT), st, g_tune[FORK_TUNE_PDL].load() >= 0, sp) != cudaSuccess) return FORK_ERR_CUDA;

  ReduceParams rp;
  memset(&rp, 0, sizeof(rp));
  rp.src = RowSource{a->logits, (long long)a->stride_b, (long long)a->stride_l, a->pos0, a->Ll, a->V};
  rp.B = a->B; rp.Lt = a->Lt; rp.C = C;
  rp.fast = fast ? 1 : 0;
  rp.hdr = w.hdr; rp.seq_off = w.seq_off; rp.expected = w.expected; rp.ticket = w.ticket;
  rp.rows = w.rows; rp.final_rec = w.final_rec; rp.parts = w.parts;
  rp.lp_tokens = a->tokens; rp.lp_out = a->logp; rp.seq_sum = a->seq_sum; rp.seq_cnt = a->seq_cnt;
  rp.lse_out = a->lse;
  rp.row_status = a->row_status;
  if (launch_reduce(rp, a->dtype, mode, G, st) != cudaSuccess) return FORK_ERR_CUDA;
  return FORK_OK;
}

extern "C" fork_status fork_decode_loop(const fork_step_args* proto, int32_t block_len, int32_t gen_lo,
                                        int32_t gen_hi, fork_logits_fn provider, void* ctx, int32_t max_steps,
                                        int32_t* steps_taken, void* ws, size_t ws_bytes, void* stream) {
  if (steps_taken) *steps_taken = 0;
  fork_status s = check_step_args(proto, false);
  if (s != FORK_OK) return s;
  if (!provider || block_len <= 0 || gen_lo < 0 || gen_hi > proto->Lt || gen_lo > gen_hi || max_steps < 0)
    return FORK_ERR_INVALID_ARG;
  s = check_workspace(ws, ws_bytes, proto->B, proto->Lt);
  if (s != FORK_OK) return s;
  if (proto->B == 0) return FORK_OK;
  cudaStream_t st = (cudaStream_t)stream;
  WsView w = ws_view(ws, proto->B, proto->Lt);

  CursorParams cp{proto->mask, proto->B, proto->Lt, gen_lo, gen_hi, block_len, w.loop_lo, w.loop_hi, w.hdr, 1};
  if (launch(block_cursor_kernel, dim3(1), dim3(kSetupNT), st, false, cp) != cudaSuccess) return FORK_ERR_CUDA;
  cp.init = 0;
  int32_t n = 0;
  fork_status rc = FORK_OK;
  for (;;) {
    int32_t remaining = 0;
    if (cudaMemcpyAsync(&remaining, &w.hdr->remaining, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) { rc = FORK_ERR_CUDA; break; }
    if (remaining == 0) break;
    if (n >= max_steps) { rc = FORK_ERR_MAX_STEPS; break; }
    if (provider(ctx, proto->step + n, proto->tokens, proto->mask, w.loop_lo, w.loop_hi,
                 const_cast<void*>(proto->logits), stream) != 0) { rc = FORK_ERR_PROVIDER; break; }
    fork_step_args a = *proto;
    a.step = proto->step + n;
    rc = step_impl(&a, w.loop_lo, w.loop_hi, ws, st);
    if (rc != FORK_OK) break;
    ++n;
    if (launch(block_cursor_kernel, dim3(1), dim3(kSetupNT), st, false, cp) != cudaSuccess) { rc = FORK_ERR_CUDA; break; }
  }
  if (steps_taken) *steps_taken = n;
  return rc;
}

extern "C" fork_status fork_device_status(const void* ws, uint32_t* host_out, void* stream) {
  if (!ws || !host_out) return FORK_ERR_INVALID_ARG;
  const WsHeader* h = (const WsHeader*)ws;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(host_out, &h->dev_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) return FORK_ERR_CUDA;
  return FORK_OK;
}

/* ---- fork_step on the library's own scratch ------------------------------------------------- */
/* The scratch that fork_step normally receives from its caller, held instead in a fixed array that
   is part of this library's device image: every GPU that loads the library carries these bytes
   until the process exits.  In host code the NAME of a __device__ array is only a host-side
   stand-in, not a device address, so the address the kernels get is looked up once per device with
   cudaGetSymbolAddress and cached. */
static __device__ __align__(256) unsigned char g_static_scratch[FORK_STATIC_SCRATCH_BYTES];
static void* g_static_scratch_ptr[64];
static std::atomic<int> g_static_scratch_ready[64];

static fork_status static_scratch(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FORK_ERR_CUDA;
  if (!g_static_scratch_ready[dev].load(std::memory_order_acquire)) {
    void* ptr = nullptr;                       /* set-up, once per device, with that device current */
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return FORK_ERR_CUDA;
    g_static_scratch_ptr[dev] = ptr;           /* every thread that gets here stores the same address */
    g_static_scratch_ready[dev].store(1, std::memory_order_release);
  }
  *out = g_static_scratch_ptr[dev];
  return FORK_OK;
}

extern "C" fork_status fork_step_static(const fork_step_args* a, void* stream) {
  fork_status s = check_step_args(a, true);
  if (s != FORK_OK) return s;
  if (fork_workspace_bytes(a->B, a->Lt) > (size_t)FORK_STATIC_SCRATCH_BYTES) return FORK_ERR_WORKSPACE;
  if (a->B == 0) return FORK_OK;
  void* ws = nullptr;
  s = static_scratch(&ws);
  if (s != FORK_OK) return s;
  /* nothing in the scratch has to survive from call to call: the active-set kernel rewrites the
     row list and offsets and clears the per-sequence ticket counters at the start of every step */
  return step_impl(a, a->blk_lo, a->blk_hi, ws, (cudaStream_t)stream);
}

/* ---- top-entropy position selection (JustGRPO-Fast; Section 3.2, last paragraph) ------------ */
/* One CTA per rollout.  Keys sit in shared memory: the entropy of an eligible position (-inf when it
   is NaN, so that it ranks last), NaN for a position that is not eligible.  Position i is selected
   when fewer than `want` eligible positions rank before it (higher entropy, or equal entropy and a
   lower position). */
constexpr int kSelectNT = 256;
constexpr int kSelectMaxLt = 32768;

__global__ void __launch_bounds__(kSelectNT) select_top_entropy_kernel(const float* __restrict__ entropy,
                                                                      const uint8_t* __restrict__ eligible, int Lt,
                                                                      float ratio, uint8_t* __restrict__ select,
                                                                      int32_t* __restrict__ n_selected) {
  extern __shared__ float sel_key[];
  __shared__ int sh_n;
  const int b = blockIdx.x, tid = threadIdx.x;
  if (tid == 0) sh_n = 0;
  __syncthreads();
  int mine = 0;
  for (int k = tid; k < Lt; k += kSelectNT) {
    const size_t at = (size_t)b * Lt + k;
    float key = __int_as_float(0x7fc00000);
    if (eligible[at]) { const float h = entropy[at]; key = (h != h) ? -INFINITY : h; ++mine; }
    sel_key[k] = key;
  }
  if (mine) atomicAdd(&sh_n, mine);
  __syncthreads();
  const int n = sh_n;
  int want = (int)floor((double)ratio * (double)n);
  if (want < 1 && n > 0 && ratio > 0.f) want = 1;
  for (int i = tid; i < Lt; i += kSelectNT) {
    const float ki = sel_key[i];
    uint8_t out = 0;
    if (ki == ki && want > 0) {
      int before = 0;
      for (int j = 0; j < Lt; ++j) {
        const float kj = sel_key[j];                          /* a comparison with NaN is false: not eligible */
        before += (kj > ki || (kj == ki && j < i)) ? 1 : 0;
      }
      out = before < want ? 1 : 0;
    }
    select[(size_t)b * Lt + i] = out;
  }
  if (tid == 0 && n_selected) n_selected[b] = want;
}

extern "C" fork_status fork_select_top_entropy(const float* entropy, const uint8_t* eligible, int32_t B, int32_t Lt,
                                               float ratio, uint8_t* select, int32_t* n_selected, void* stream) {
  if (!entropy || !eligible || !select || B < 0 || Lt <= 0 || Lt > kSelectMaxLt) return FORK_ERR_INVALID_ARG;
  if (!(ratio >= 0.f) || ratio > 1.f) return FORK_ERR_INVALID_ARG;
  if (B == 0) return FORK_OK;
  const size_t smem = (size_t)Lt * sizeof(float);
  static std::atomic<int> raised[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return FORK_ERR_CUDA;
  if (smem > 48 * 1024 && (dev >= 64 || !raised[dev].load())) {
    if (cudaFuncSetAttribute(select_top_entropy_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kSelectMaxLt * (int)sizeof(float)) != cudaSuccess) return FORK_ERR_CUDA;
    if (dev < 64) raised[dev].store(1);
  }
  select_top_entropy_kernel<<<B, kSelectNT, smem, (cudaStream_t)stream>>>(entropy, eligible, Lt, ratio, select, n_selected);
  if (cudaGetLastError() != cudaSuccess) return FORK_ERR_CUDA;
  g_launches.fetch_add(1);
  return FORK_OK;
}

/* ---- ForkGRPO objective (Eq. 2) ------------------------------------------------------------- */
/* One CTA per prompt group.  Group statistics in fp64 (a handful of values), the per-position terms
   in fp32; one warp per rollout walks its positions twice (count of fallback steps, then the
   terms).  A second one-CTA kernel sums the per-rollout objectives in a fixed order. */
constexpr int kGrpoNT = 256;

__global__ void __launch_bounds__(kGrpoNT) grpo_group_kernel(fork_grpo_args a) {
  __shared__ double sh_mean, sh_sd;
  const int p = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = kGrpoNT / 32;
  const int G = a.group, B = a.B, Lt = a.Lt;
  if (tid == 0) {
    double mean = 0.0, var = 0.0;
    for (int j = 0; j < G; ++j) mean += (double)a.reward[p * G + j];
    mean /= G;
    for (int j = 0; j < G; ++j) { const double d = (double)a.reward[p * G + j] - mean; var += d * d; }
    sh_mean = mean; sh_sd = sqrt(var / G);
    if (a.skipped) a.skipped[p] = (uint8_t)(!(sh_sd > 0.0));
  }
  __syncthreads();
  const bool skip = !(sh_sd > 0.0);
  for (int j = warp; j < G; j += nwarp) {
    const int i = p * G + j;
    const float A = skip ? 0.f : (float)(((double)a.reward[i] - sh_mean) / sh_sd);
    int nf = 0;
    for (int k0 = 0; k0 < Lt; k0 += 32) {
      const int k = k0 + lane;
      nf += __popc(__ballot_sync(0xffffffffu, k < Lt && a.select[(size_t)i * Lt + k] != 0));
    }
    const float scale = nf > 0 ? 1.f / ((float)B * (float)nf) : 0.f;
    float acc = 0.f;
    for (int k = lane; k < Lt; k += 32) {
      const size_t at = (size_t)i * Lt + k;
      float rho = 0.f, d = 0.f;
      if (a.select[at]) {
        rho = expf(a.logp_new[at] - a.logp_old[at]);
        const float clipped = fminf(fmaxf(rho, 1.f - a.eps_lo), 1.f + a.eps_hi);
        const float u = rho * A, c = clipped * A;
        acc += (u <= c) ? u : c;                             /* the clipped minimum of Eq. 2 */
        if (!skip && u <= c) d = rho * A * scale;            /* the unclipped term is active */
      }
      if (a.ratio) a.ratio[at] = rho;
      if (a.dlogp) a.dlogp[at] = d;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) {
      if (a.adv) a.adv[i] = A;
      a.seq_obj[i] = nf > 0 ? acc / (float)nf : 0.f;
    }
  }
}

__global__ void __launch_bounds__(kGrpoNT) grpo_sum_kernel(const float* seq_obj, int B, float* objective) {
  __shared__ double sh[kGrpoNT];
  double acc = 0.0;
  for (int i = threadIdx.x; i < B; i += kGrpoNT) acc += (double)seq_obj[i];
  sh[threadIdx.x] = acc;
  __syncthreads();
  for (int o = kGrpoNT / 2; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *objective = B > 0 ? (float)(sh[0] / B) : 0.f;
}

extern "C" fork_status fork_grpo_loss(const fork_grpo_args* a, void* stream) {
  if (!a || a->B < 0 || a->Lt <= 0 || a->group <= 0 || a->B % a->group != 0) return FORK_ERR_INVALID_ARG;
  if (!a->logp_new || !a->logp_old || !a->select || !a->reward || !a->seq_obj) return FORK_ERR_INVALID_ARG;
  if (!(a->eps_lo >= 0.f) || !(a->eps_hi >= 0.f)) return FORK_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (a->B > 0) {
    grpo_group_kernel<<<a->B / a->group, kGrpoNT, 0, st>>>(*a);
    if (cudaGetLastError() != cudaSuccess) return FORK_ERR_CUDA;
    g_launches.fetch_add(1);
  }
  if (a->objective) {
    grpo_sum_kernel<<<1, kGrpoNT, 0, st>>>(a->seq_obj, a->B, a->objective);
    if (cudaGetLastError() != cudaSuccess) return FORK_ERR_CUDA;
    g_launches.fetch_add(1);
  }
  return FORK_OK;
}

/* ---- derivative of the scored log-likelihoods with respect to the logits -------------------- */
/* d/dx_v [w (x_tok - lse)] = w (1[v = tok] - p_v), p_v = exp(x_v - lse): one read of the row, one
   write of the same size.  Work is cut into units of kBwdNT * kBwdVecs * kBwdIters 128-bit vectors of one row;
   the rows are those of the row list the active-set kernel built from `select`. */
constexpr int kBwdNT = 256;
constexpr int kBwdVecs = 2;
constexpr int kBwdIters = 8;          /* a unit = kBwdIters inner iterations of one row (64 KB): per-row values are fetched once per unit */

struct BwdParams {
  RowSource src; void* grad; long long gstride_b, gstride_l;
  const WsHeader* hdr; const int2* rows;
  const int32_t* tokens; const float* lse; const float* dlogp; int Lt, vector_ok;
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ void store_grad(bf16_t* p, float g) {
  p->bits = (uint16_t)(pack_bf16x2(g, 0.f) & 0xffffu);
}
__device__ __forceinline__ void store_grad(float* p, float g) { *p = g; }

template <typename T>
__global__ void __launch_bounds__(kBwdNT) logprob_backward_kernel(BwdParams p) {
  constexpr int VEC = 16 / (int)sizeof(T);
  constexpr int kStepElems = kBwdNT * kBwdVecs * VEC;          /* elements per inner iteration */
  constexpr int kUnitElems = kStepElems * kBwdIters;           /* elements of one row per unit */
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int R = p.hdr->R;
  const int V = p.src.V;
  const int units_per_row = (V + kUnitElems - 1) / kUnitElems;
  const long long U = (long long)R * units_per_row;
  for (long long u = blockIdx.x; u < U; u += gridDim.x) {
    const int r = (int)(u / units_per_row);
    const int u0 = (int)(u - (long long)r * units_per_row) * kUnitElems;
    const int u1 = min(u0 + kUnitElems, V);
    const int2 bk = p.rows[r];
    const size_t at = (size_t)bk.x * p.Lt + bk.y;
    const int tok = p.tokens[at];
    if (tok < 0 || tok >= V) continue;                       /* scored as FORK_ROW_BAD_TOKEN: no gradient */
    const float w = p.dlogp[at];
    const float nl = -p.lse[at] * kLog2e;
    const T* row = row_ptr<T>(p.src, bk.x, bk.y);
    T* grow = reinterpret_cast<T*>(p.grad) + ((long long)bk.x * p.gstride_b + (long long)(bk.y - p.src.pos0) * p.gstride_l);
    if (!p.vector_ok) {
      for (int q = u0 + (int)threadIdx.x; q < u1; q += kBwdNT) {
        const float pr = exp2f(fmaf(to_f32(row[q]), kLog2e, nl));
        store_grad(grow + q, w * ((q == tok ? 1.f : 0.f) - pr));
      }
      continue;
    }
    for (int e0 = u0; e0 < u1; e0 += kStepElems) {
      uint4 v[kBwdVecs];
      int e[kBwdVecs];
#pragma unroll
      for (int j = 0; j < kBwdVecs; ++j) {
        e[j] = e0 + ((int)threadIdx.x + j * kBwdNT) * VEC;
        if (e[j] + VEC <= V) v[j] = ld_stream(reinterpret_cast<const uint4*>(row + e[j]));
      }
#pragma unroll
      for (int j = 0; j < kBwdVecs; ++j) {
        if (e[j] + VEC <= V) {
          float x[VEC];
          if (sizeof(T) == 2) {
            x[0] = bf16_lo(v[j].x); x[1] = bf16_hi(v[j].x); x[2 % VEC] = bf16_lo(v[j].y); x[3 % VEC] = bf16_hi(v[j].y);
            x[4 % VEC] = bf16_lo(v[j].z); x[5 % VEC] = bf16_hi(v[j].z); x[6 % VEC] = bf16_lo(v[j].w); x[7 % VEC] = bf16_hi(v[j].w);
          } else {
            x[0] = __uint_as_float(v[j].x); x[1] = __uint_as_float(v[j].y); x[2] = __uint_as_float(v[j].z); x[3] = __uint_as_float(v[j].w);
          }
          float gr[VEC];
#pragma unroll
          for (int q = 0; q < VEC; ++q) {
            const float pr = ex2_approx(fmaf(x[q], kLog2e, nl));
            gr[q] = w * ((e[j] + q == tok ? 1.f : 0.f) - pr);
          }
          uint4 o;
          if (sizeof(T) == 2) {
            o.x = pack_bf16x2(gr[0], gr[1]); o.y = pack_bf16x2(gr[2 % VEC], gr[3 % VEC]);
            o.z = pack_bf16x2(gr[4 % VEC], gr[5 % VEC]); o.w = pack_bf16x2(gr[6 % VEC], gr[7 % VEC]);
          } else {
            o.x = __float_as_uint(gr[0]); o.y = __float_as_uint(gr[1]); o.z = __float_as_uint(gr[2]); o.w = __float_as_uint(gr[3]);
          }
          __stcs(reinterpret_cast<uint4*>(grow + e[j]), o);
        } else {
          for (int q = e[j]; q < V && q < e[j] + VEC; ++q) {  /* the ragged end of the row */
            const float pr = exp2f(fmaf(to_f32(row[q]), kLog2e, nl));
            store_grad(grow + q, w * ((q == tok ? 1.f : 0.f) - pr));
          }
        }
      }
    }
  }
}

extern "C" fork_status fork_logprob_backward(const fork_logprob_bwd_args* a, void* ws, size_t ws_bytes, void* stream) {
  if (!a) return FORK_ERR_INVALID_ARG;
  if (bad_source(a->logits, a->stride_b, a->stride_l, a->pos0, a->B, a->Lt, a->Ll, a->V, a->dtype))
    return FORK_ERR_INVALID_ARG;
  if (!a->tokens || !a->select || !a->lse || !a->dlogp || !a->grad) return FORK_ERR_INVALID_ARG;
  if (a->grad_stride_l < a->V || a->grad_stride_b < 0) return FORK_ERR_INVALID_ARG;
  fork_status s = check_workspace(ws, ws_bytes, a->B, a->Lt);
  if (s != FORK_OK) return s;
  if (a->B == 0) return FORK_OK;
  cudaStream_t st = (cudaStream_t)stream;
  DeviceInfo* dev;
  if (!device_info(&dev)) return FORK_ERR_CUDA;
  WsView w = ws_view(ws, a->B, a->Lt);
  SetupParams sp;
  memset(&sp, 0, sizeof(sp));
  sp.flags = a->select; sp.lo = nullptr; sp.hi = nullptr;
  sp.B = a->B; sp.Lt = a->Lt; sp.pos0 = a->pos0; sp.Ll = a->Ll; sp.C = 1; sp.G = 1;
  sp.hdr = w.hdr; sp.seq_off = w.seq_off; sp.expected = w.expected; sp.ticket = w.ticket; sp.rows = w.rows;
  const bool pdl = g_tune[FORK_TUNE_PDL].load() >= 0;
  if (launch(active_set_kernel, dim3(1), dim3(kSetupNT), st, pdl, sp) != cudaSuccess) return FORK_ERR_CUDA;
  BwdParams bp;
  memset(&bp, 0, sizeof(bp));
  bp.src = RowSource{a->logits, (long long)a->stride_b, (long long)a->stride_l, a->pos0, a->Ll, a->V};
  bp.grad = a->grad; bp.gstride_b = a->grad_stride_b; bp.gstride_l = a->grad_stride_l;
  bp.hdr = w.hdr; bp.rows = w.rows; bp.tokens = a->tokens; bp.lse = a->lse; bp.dlogp = a->dlogp; bp.Lt = a->Lt;
  bp.vector_ok = (source_is_vector_aligned(a->logits, a->stride_b, a->stride_l, a->dtype) &&
                  source_is_vector_aligned(a->grad, a->grad_stride_b, a->grad_stride_l, a->dtype)) ? 1 : 0;
  const int grid = dev->sms * 8;
  cudaError_t e = a->dtype == FORK_BF16 ? launch(logprob_backward_kernel<bf16_t>, dim3(grid), dim3(kBwdNT), st, pdl, bp)
                                        : launch(logprob_backward_kernel<float>, dim3(grid), dim3(kBwdNT), st, pdl, bp);
  return e == cudaSuccess ? FORK_OK : FORK_ERR_CUDA;
}

/* ---- vocabulary-parallel entry points ------------------------------------------------------- */
extern "C" fork_status fork_vp_reduce(const fork_step_args* a, int32_t vocab_offset, void* part_out, void* key_out,
                                      void* ws, size_t ws_bytes, void* stream) {
  fork_status s = check_step_args(a, true);
  if (s != FORK_OK) return s;
  if (!part_out || vocab_offset < 0 || (int64_t)vocab_offset + a->V > 0x7fffffffLL) return FORK_ERR_INVALID_ARG;
  if (a->temperature > 0.f && !key_out) return FORK_ERR_INVALID_ARG;
  if (((uintptr_t)part_out % 16) != 0 || ((uintptr_t)key_out % 16) != 0) return FORK_ERR_INVALID_ARG;
  s = check_workspace(ws, ws_bytes, a->B, a->Lt);
  if (s != FORK_OK) return s;
  if (a->B == 0) return FORK_OK;
  VpLocal vp{vocab_offset, (float4*)part_out, (float4*)key_out};
  return step_impl(a, a->blk_lo, a->blk_hi, ws, (cudaStream_t)stream, &vp);
}

extern "C" fork_status fork_vp_select(const fork_step_args* a, const void* parts, const void* keys, int32_t n_ranks,
                                      void* ws, size_t ws_bytes, void* stream) {
  if (!a || a->B < 0 || a->Lt <= 0 || !a->tokens || !a->mask || !a->blk_lo || !a->blk_hi) return FORK_ERR_INVALID_ARG;
  if ((int64_t)a->B * a->Lt > (int64_t)1 << 30) return FORK_ERR_INVALID_ARG;
  if (a->threshold != a->threshold) return FORK_ERR_INVALID_ARG;
  if (a->fallback_mode < FORK_FALLBACK_LEFTMOST || a->fallback_mode > FORK_FALLBACK_RANDOM) return FORK_ERR_INVALID_ARG;
  if (a->fallback_mode == FORK_FALLBACK_RANDOM && !a->fallback_rand) return FORK_ERR_INVALID_ARG;
  if (!(a->temperature >= 0.f) || a->temperature > 3.0e38f) return FORK_ERR_INVALID_ARG;
  if (!parts || n_ranks <= 0 || (a->temperature > 0.f && !keys)) return FORK_ERR_INVALID_ARG;
  if (((uintptr_t)parts % 16) != 0 || ((uintptr_t)keys % 16) != 0) return FORK_ERR_INVALID_ARG;
  fork_status s = check_workspace(ws, ws_bytes, a->B, a->Lt);
  if (s != FORK_OK) return s;
  if (a->B == 0) return FORK_OK;
  cudaStream_t st = (cudaStream_t)stream;
  WsView w = ws_view(ws, a->B, a->Lt);
  const bool pdl = g_tune[FORK_TUNE_PDL].load() >= 0;
  SetupParams sp;
  memset(&sp, 0, sizeof(sp));
  sp.flags = a->mask; sp.lo = a->blk_lo; sp.hi = a->blk_hi;
  sp.B = a->B; sp.Lt = a->Lt; sp.pos0 = 0; sp.Ll = a->Lt; sp.C = 1; sp.G = 1;
  if (a->Ll > 0) { sp.pos0 = a->pos0; sp.Ll = a->Ll; }      /* the window the slices covered */
  sp.hdr = w.hdr; sp.seq_off = w.seq_off; sp.expected = w.expected; sp.ticket = w.ticket; sp.rows = w.rows;
  sp.n_unmasked = a->n_unmasked; sp.is_fallback = a->is_fallback; sp.fallback_pos = a->fallback_pos;
  if (launch(active_set_kernel, dim3(1), dim3(kSetupNT), st, pdl, sp) != cudaSuccess) return FORK_ERR_CUDA;
  ReduceParams rp;
  memset(&rp, 0, sizeof(rp));
  rp.B = a->B; rp.Lt = a->Lt; rp.C = 1;
  rp.hdr = w.hdr; rp.seq_off = w.seq_off; rp.expected = w.expected; rp.ticket = w.ticket;
  rp.rows = w.rows; rp.final_rec = w.final_rec; rp.parts = w.parts; rp.kparts = w.kparts;
  rp.tokens = a->tokens; rp.mask = a->mask; rp.threshold = a->threshold; rp.step = a->step;
  rp.conf = a->conf; rp.cand = a->cand; rp.entropy = a->entropy; rp.logp = a->logp; rp.row_status = a->row_status;
  rp.commit_step = a->commit_step; rp.commit_fallback = a->commit_fallback; rp.commit_logp = a->commit_logp;
  rp.n_unmasked = a->n_unmasked; rp.is_fallback = a->is_fallback; rp.fallback_pos = a->fallback_pos;
  rp.nfe = a->nfe; rp.n_fallback = a->n_fallback;
  rp.fallback_mode = a->fallback_mode; rp.fallback_rand = a->fallback_rand;
  rp.vp_parts_in = (const float4*)parts; rp.vp_keys_in = (const float4*)keys; rp.vp_ranks = n_ranks;
  const dim3 grid((unsigned)((a->B + kVpNT / 32 - 1) / (kVpNT / 32)));
  cudaError_t e = a->temperature > 0.f ? launch(vp_select_kernel<true>, grid, dim3(kVpNT), st, pdl, rp)
                                       : launch(vp_select_kernel<false>, grid, dim3(kVpNT), st, pdl, rp);
  return e == cudaSuccess ? FORK_OK : FORK_ERR_CUDA;
}

/* ---- host-buffer entry point --------------------------------------------------------------- */
struct StagingView {
  char* logits; int32_t* tokens; uint8_t* mask; int32_t* lo; int32_t* hi;
  float* conf; int32_t* cand; float* entropy; float* logp; uint32_t* row_status;
  int32_t* commit_step; uint8_t* commit_fallback; float* commit_logp;
  int32_t* n_unmasked; uint8_t* is_fallback; int32_t* fallback_pos; int32_t* nfe; int32_t* n_fallback;
  uint32_t* fallback_rand;
  size_t logits_bytes, bytes;
};

static StagingView staging_view(void* base, const fork_step_args* a) {
  StagingView v;
  char* p = (char*)base;
  size_t off = 0;
  const size_t es = a->dtype == FORK_BF16 ? 2 : 4;
  const size_t nb = (size_t)(a->B > 0 ? a->B : 1), n = nb * (size_t)a->Lt;
  /* the window is re-packed densely on the device side: [B, Ll, stride_l] */
  v.logits_bytes = nb * (size_t)a->Ll * (size_t)a->stride_l * es;
  auto take = [&](size_t bytes) { char* q = p + off; off = align_up(off + bytes, 256); return q; };
  v.logits = take(v.logits_bytes);
  v.tokens = (int32_t*)take(n * 4); v.mask = (uint8_t*)take(n);
  v.lo = (int32_t*)take(nb * 4); v.hi = (int32_t*)take(nb * 4);
  v.conf = (float*)take(n * 4); v.cand = (int32_t*)take(n * 4); v.entropy = (float*)take(n * 4);
  v.logp = (float*)take(n * 4); v.row_status = (uint32_t*)take(n * 4);
  v.commit_step = (int32_t*)take(n * 4); v.commit_fallback = (uint8_t*)take(n); v.commit_logp = (float*)take(n * 4);
  v.n_unmasked = (int32_t*)take(nb * 4); v.is_fallback = (uint8_t*)take(nb); v.fallback_pos = (int32_t*)take(nb * 4);
  v.nfe = (int32_t*)take(nb * 4); v.n_fallback = (int32_t*)take(nb * 4);
  v.fallback_rand = (uint32_t*)take(nb * 4);
  v.bytes = off;
  return v;
}

extern "C" size_t fork_staging_bytes(const fork_step_args* a) {
  if (!a || a->B < 0 || a->Lt <= 0 || a->Ll <= 0 || a->stride_l <= 0) return 0;
  return staging_view(nullptr, a).bytes;
}

extern "C" fork_status fork_step_host(const fork_step_args* h, void* staging, size_t staging_bytes, void* ws,
                                      size_t ws_bytes, void* stream) {
  fork_status s = check_step_args(h, true);
  if (s != FORK_OK) return s;
  if (h->stride_b != (int64_t)h->Ll * h->stride_l) return FORK_ERR_INVALID_ARG;   /* host window must be dense in b */
  s = check_workspace(ws, ws_bytes, h->B, h->Lt);
  if (s != FORK_OK) return s;
  if (!staging || ((uintptr_t)staging % 256) != 0 || staging_bytes < fork_staging_bytes(h)) return FORK_ERR_WORKSPACE;
  if (h->B == 0) return FORK_OK;
  cudaStream_t st = (cudaStream_t)stream;
  StagingView v = staging_view(staging, h);
  const size_t n = (size_t)h->B * h->Lt, nb = (size_t)h->B;
#define FORK_H2D(dst, src, bytes) \
  if ((src) && cudaMemcpyAsync((dst), (src), (bytes), cudaMemcpyHostToDevice, st) != cudaSuccess) return FORK_ERR_CUDA
#define FORK_D2H(dst, src, bytes) \
  if ((dst) && cudaMemcpyAsync((dst), (src), (bytes), cudaMemcpyDeviceToHost, st) != cudaSuccess) return FORK_ERR_CUDA
  FORK_H2D(v.logits, h->logits, v.logits_bytes);
  FORK_H2D(v.tokens, h->tokens, n * 4); FORK_H2D(v.mask, h->mask, n);
  FORK_H2D(v.lo, h->blk_lo, nb * 4); FORK_H2D(v.hi, h->blk_hi, nb * 4);
  FORK_H2D(v.nfe, h->nfe, nb * 4); FORK_H2D(v.n_fallback, h->n_fallback, nb * 4);
  FORK_H2D(v.fallback_rand, h->fallback_rand, nb * 4);
  fork_step_args d = *h;
  d.logits = v.logits; d.tokens = v.tokens; d.mask = v.mask; d.blk_lo = v.lo; d.blk_hi = v.hi;
  d.conf = h->conf ? v.conf : nullptr; d.cand = h->cand ? v.cand : nullptr;
  d.entropy = h->entropy ? v.entropy : nullptr; d.logp = h->logp ? v.logp : nullptr;
  d.row_status = h->row_status ? v.row_status : nullptr;
  d.commit_step = h->commit_step ? v.commit_step : nullptr;
  d.commit_fallback = h->commit_fallback ? v.commit_fallback : nullptr;
  d.commit_logp = h->commit_logp ? v.commit_logp : nullptr;
  d.n_unmasked = h->n_unmasked ? v.n_unmasked : nullptr; d.is_fallback = h->is_fallback ? v.is_fallback : nullptr;
  d.fallback_pos = h->fallback_pos ? v.fallback_pos : nullptr;
  d.nfe = h->nfe ? v.nfe : nullptr; d.n_fallback = h->n_fallback ? v.n_fallback : nullptr;
  d.fallback_rand = h->fallback_rand ? v.fallback_rand : nullptr;
  /* per-position outputs are written only on the live / committed set: start from the host's values */
  FORK_H2D(v.conf, h->conf, n * 4); FORK_H2D(v.cand, h->cand, n * 4); FORK_H2D(v.entropy, h->entropy, n * 4);
  FORK_H2D(v.logp, h->logp, n * 4); FORK_H2D(v.row_status, h->row_status, n * 4);
  FORK_H2D(v.commit_step, h->commit_step, n * 4); FORK_H2D(v.commit_fallback, h->commit_fallback, n);
  FORK_H2D(v.commit_logp, h->commit_logp, n * 4);
  s = step_impl(&d, d.blk_lo, d.blk_hi, ws, st);
  if (s != FORK_OK) return s;
  FORK_D2H(h->tokens, v.tokens, n * 4); FORK_D2H(h->mask, v.mask, n);
  FORK_D2H(h->conf, v.conf, n * 4); FORK_D2H(h->cand, v.cand, n * 4); FORK_D2H(h->entropy, v.entropy, n * 4);
  FORK_D2H(h->logp, v.logp, n * 4); FORK_D2H(h->row_status, v.row_status, n * 4);
  FORK_D2H(h->commit_step, v.commit_step, n * 4); FORK_D2H(h->commit_fallback, v.commit_fallback, n);
  FORK_D2H(h->commit_logp, v.commit_logp, n * 4);
  FORK_D2H(h->n_unmasked, v.n_unmasked, nb * 4); FORK_D2H(h->is_fallback, v.is_fallback, nb);
  FORK_D2H(h->fallback_pos, v.fallback_pos, nb * 4);
  FORK_D2H(h->nfe, v.nfe, nb * 4); FORK_D2H(h->n_fallback, v.n_fallback, nb * 4);
#undef FORK_H2D
#undef FORK_D2H
  if (cudaStreamSynchronize(st) != cudaSuccess) return FORK_ERR_CUDA;
  return FORK_OK;
}

/* ---- read-only streaming probe ---------------------------------------------------------------- */
/* The rate at which this GPU delivers a buffer that is only read (128-bit streaming loads, a
   persistent grid, nothing computed but an XOR): the practical ceiling for the reduction kernels,
   which never write more than a few bytes per row.  The benchmark reports it beside the measured
   copy rate. */
__global__ void __launch_bounds__(256, 4) read_probe_kernel(const uint4* __restrict__ p, long long nvec, uint32_t* sink) {
  /* every CTA reads one contiguous share, like the reduction kernels */
  const long long per = (nvec + gridDim.x - 1) / gridDim.x;
  const long long lo = (long long)blockIdx.x * per, hi = (lo + per < nvec) ? lo + per : nvec;
  uint32_t x = 0;
  long long i = lo + threadIdx.x;
  for (; i + 3 * 256 < hi; i += 256 * 4) {
    uint4 v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = ld_stream(p + i + j * 256);
#pragma unroll
    for (int j = 0; j < 4; ++j) x ^= v[j].x ^ v[j].y ^ v[j].z ^ v[j].w;
  }
  for (; i < hi; i += 256) { const uint4 v = ld_stream(p + i); x ^= v.x ^ v.y ^ v.z ^ v.w; }
  if (x == 0x9e3779b9u) *sink = x;                           /* practically never: keeps the loads alive */
}

extern "C" fork_status fork_read_probe(const void* buffer, size_t bytes, void* sink4, void* stream) {
  if (!buffer || !sink4 || (reinterpret_cast<uintptr_t>(buffer) & 15u) != 0) return FORK_ERR_INVALID_ARG;
  DeviceInfo* dev;
  if (!device_info(&dev)) return FORK_ERR_CUDA;
  read_probe_kernel<<<dev->sms * 4, 256, 0, (cudaStream_t)stream>>>((const uint4*)buffer, (long long)(bytes / 16), (uint32_t*)sink4);
  if (cudaGetLastError() != cudaSuccess) return FORK_ERR_CUDA;
  g_launches.fetch_add(1);
  return FORK_OK;
}

/* ---- host-side view of the partition, for tests ------------------------------------------- */
extern "C" int64_t fork_debug_part_begin(int64_t U, int32_t G, int32_t g) { return fork_part_begin(U, G, g); }
extern "C" int32_t fork_debug_part_owner(int64_t U, int32_t G, int64_t x) { return fork_part_owner(U, G, x); }
extern "C" int32_t fork_debug_row_parts(int64_t U, int32_t G, int32_t C, int64_t r) { return fork_row_parts(U, G, C, r); }
extern "C" int32_t fork_debug_chunk(void) { return FORK_CHUNK; }
extern "C" int32_t fork_debug_effective_grid(int64_t U, int32_t G) { return fork_effective_grid(U, G); }
