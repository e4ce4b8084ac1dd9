/*
 * Kernels and C ABI of the Fork-dLLM confidence pass (see include/fork_dllm.h for the contract).
 *
 * A step is two launches on the caller's stream:
 *   1. active_set_kernel (one CTA): M_t restricted to each sequence's block (Algorithm 2, line 3)
 *      compacted into a row list, per-sequence row offsets, and the number of partial results each
 *      sequence will receive.  It snapshots the mask, so the second kernel never reads `mask`
 *      (which it modifies).
 *   2. reduce_select_kernel (persistent grid): streams every live row once (lines 4-5: arg-max
 *      candidate and its softmax probability, plus entropy), and the CTA that delivers the last
 *      partial result of a sequence applies the unmask rule for it (lines 6-9: threshold set, or
 *      the leftmost masked position when that set is empty) and writes tokens, mask and records.
 * Cross-CTA hand-over uses "last one to arrive" ticket counters (fence + atomic): nothing in
 * here ever waits for another CTA.
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

enum Mode { kModeStep = 0, kModeLogprob = 1 };

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
  const int2* rows; float4* final_rec; float4* parts;
  /* step mode */
  int32_t* tokens; uint8_t* mask; float threshold; int32_t step;
  float* conf; int32_t* cand; float* entropy; float* logp; uint32_t* row_status;
  int32_t* commit_step; uint8_t* commit_fallback; float* commit_logp;
  int32_t* n_unmasked; uint8_t* is_fallback; int32_t* fallback_pos; int32_t* nfe; int32_t* n_fallback;
  /* log-probability mode */
  const int32_t* lp_tokens; float* lp_out; float* seq_sum; int32_t* seq_cnt;
};

template <typename T>
__device__ __forceinline__ const T* row_ptr(const RowSource& s, int b, int k) {
  return reinterpret_cast<const T*>(s.logits) + ((long long)b * s.stride_b + (long long)(k - s.pos0) * s.stride_l);
}

__device__ __forceinline__ float4 ld_cg_f4(const float4* p) { return __ldcg(p); }

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

__global__ void __launch_bounds__(kSetupNT, 1) active_set_kernel(SetupParams p) {
  asm volatile("griddepcontrol.launch_dependents;");
  __shared__ int sh_warp[kSetupNT / 32];
  __shared__ int sh_carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = kSetupNT / 32;
  unsigned clipped_any = 0;

  /* pass 1: live rows per sequence */
  for (int b = warp; b < p.B; b += nwarp) {
    int lo, hi; bool clipped;
    seq_window(p, b, lo, hi, clipped);
    clipped_any |= clipped ? 1u : 0u;
    int cnt = 0;
    for (int k0 = lo; k0 < hi; k0 += 32) {
      int k = k0 + lane;
      bool live = (k < hi) && p.flags[(size_t)b * p.Lt + k] != 0;
      cnt += __popc(__ballot_sync(0xffffffffu, live));
    }
    if (lane == 0) { p.seq_off[b + 1] = cnt; p.expected[b] = 0; p.ticket[b] = 0; }
  }
  if (tid == 0) { p.seq_off[0] = 0; sh_carry = 0; }
  __syncthreads();

  /* pass 2: inclusive scan of the counts, kSetupNT sequences at a time */
  for (int base = 0; base < p.B; base += kSetupNT) {
    int b = base + tid;
    int v = (b < p.B) ? p.seq_off[b + 1] : 0;
    int x = v;
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
    if (b < p.B) p.seq_off[b + 1] = incl;
    __syncthreads();
    if (tid == kSetupNT - 1) sh_carry = incl;
    __syncthreads();
  }
  const int R = sh_carry;
  const long long U = (long long)R * p.C;
  const int G = fork_effective_grid(U, p.G);
  if (tid == 0) {
    p.hdr->R = R; p.hdr->C = p.C; p.hdr->G = G;
  }

  /* pass 3: row list, expected part counts, outputs of idle sequences */
  for (int b = warp; b < p.B; b += nwarp) {
    int lo, hi; bool clipped;
    seq_window(p, b, lo, hi, clipped);
    const int r0 = p.seq_off[b], r1 = p.seq_off[b + 1];
    int run = r0;
    for (int k0 = lo; k0 < hi; k0 += 32) {
      int k = k0 + lane;
      bool live = (k < hi) && p.flags[(size_t)b * p.Lt + k] != 0;
      unsigned bal = __ballot_sync(0xffffffffu, live);
      if (live) p.rows[run + __popc(bal & ((1u << lane) - 1u))] = make_int2(b, k);
      run += __popc(bal);
    }
    int parts = 0;
    for (int r = r0 + lane; r < r1; r += 32) parts += fork_row_parts(U, G, p.C, r);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) parts += __shfl_down_sync(0xffffffffu, parts, o);
    if (lane == 0) {
      p.expected[b] = parts;
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

/* ---- kernel 2: stream, reduce, select, commit --------------------------------------------- */
struct Smem {
  Part parts[kNT / 32];
  float fl[kNT / 32];
  int flag;
  int pick;
  int count;
};

/* all parts of row r, merged in ascending CTA order */
__device__ __forceinline__ Part merge_row_parts(const ReduceParams& p, long long U, int G, int r) {
  const int g0 = fork_part_owner(U, G, (long long)r * p.C);
  const int g1 = fork_part_owner(U, G, (long long)(r + 1) * p.C - 1);
  Part acc = part_empty();
  for (int g = g0; g <= g1; ++g) {
    float4 v = ld_cg_f4(p.parts + (r + g));
    Part q{v.x, v.y, v.z, __float_as_int(v.w)};
    acc = (g == g0) ? q : part_merge(acc, q);
  }
  return acc;
}

/* Row statistics of a batch of up to kNT rows starting at `base`, one row per thread; rows whose
   streamed result is not finite are re-read by the whole CTA with the guarded routine. */
template <typename T>
__device__ __forceinline__ RowOut finalize_rows(const ReduceParams& p, Smem& sm, long long U, int G,
                                                int base, int r1, Part& merged) {
  const int r = base + threadIdx.x;
  const bool valid = r < r1;
  bool redo = false;
  merged = part_empty();
  if (valid) { merged = merge_row_parts(p, U, G, r); redo = part_needs_careful(merged); }
  RowOut o = row_out_from(merged, false);
  if (__syncthreads_or(redo ? 1 : 0)) {
    for (;;) {
      if (threadIdx.x == 0) sm.pick = kIdxNone;
      __syncthreads();
      if (redo) atomicMin(&sm.pick, r);
      __syncthreads();
      const int pick = sm.pick;
      if (pick == kIdxNone) break;
      const int2 bk = p.rows[pick];
      bool bad;
      Part c = careful_segment<T, kNT>(row_ptr<T>(p.src, bk.x, bk.y), 0, p.src.V, sm.parts, sm.fl, bad);
      if (r == pick) { merged = c; o = row_out_from(c, bad); redo = false; }
      __syncthreads();
    }
  }
  return o;
}

template <typename T>
__device__ void finalize_step_sequence(const ReduceParams& p, Smem& sm, long long U, int G, int b) {
  const int r0 = p.seq_off[b], r1 = p.seq_off[b + 1];
  int any = 0;
  for (int base = r0; base < r1; base += kNT) {
    Part merged;
    RowOut o = finalize_rows<T>(p, sm, U, G, base, r1, merged);
    const int r = base + threadIdx.x;
    if (r < r1) {
      const size_t at = (size_t)b * p.Lt + p.rows[r].y;
      if (p.conf) p.conf[at] = o.conf;
      if (p.cand) p.cand[at] = o.cand;
      if (p.entropy) p.entropy[at] = o.entropy;
      if (p.logp) p.logp[at] = o.logp;
      if (p.row_status) p.row_status[at] = o.status;
      p.final_rec[r] = make_float4(o.conf, o.logp, __int_as_float(o.cand), 0.f);
      any |= (o.conf > p.threshold) ? 1 : 0;                 /* U_t non-empty (Algorithm 2, line 6) */
    }
  }
  any = __syncthreads_or(any);
  const int fb = any ? 0 : 1;                                /* fallback step: max_k c <= lambda */
  int count = 0;
  for (int base = r0; base < r1; base += kNT) {
    const int r = base + threadIdx.x;
    if (r < r1) {
      const float4 f = p.final_rec[r];                       /* written by this same thread above */
      const bool commit = fb ? (r == r0) : (f.x > p.threshold);   /* leftmost(M_t), or the threshold set */
      if (commit) {
        const size_t at = (size_t)b * p.Lt + p.rows[r].y;
        p.tokens[at] = __float_as_int(f.z);
        p.mask[at] = 0;
        if (p.commit_step) p.commit_step[at] = p.step;
        if (p.commit_fallback) p.commit_fallback[at] = (uint8_t)fb;
        if (p.commit_logp) p.commit_logp[at] = f.y;
        ++count;
      }
    }
  }
  if (threadIdx.x == 0) sm.count = 0;
  __syncthreads();
  if (count) atomicAdd(&sm.count, count);
  __syncthreads();
  if (threadIdx.x == 0) {
    if (p.n_unmasked) p.n_unmasked[b] = sm.count;
    if (p.is_fallback) p.is_fallback[b] = (uint8_t)fb;
    if (p.fallback_pos) p.fallback_pos[b] = fb ? p.rows[r0].y : -1;
    if (p.nfe) p.nfe[b] += 1;
    if (p.n_fallback) p.n_fallback[b] += fb;
  }
  __syncthreads();
}

template <typename T>
__device__ void finalize_logprob_sequence(const ReduceParams& p, Smem& sm, long long U, int G, int b) {
  const int r0 = p.seq_off[b], r1 = p.seq_off[b + 1];
  float local = 0.f;
  for (int base = r0; base < r1; base += kNT) {
    Part merged;
    RowOut o = finalize_rows<T>(p, sm, U, G, base, r1, merged);
    const int r = base + threadIdx.x;
    if (r < r1) {
      const int k = p.rows[r].y;
      const size_t at = (size_t)b * p.Lt + k;
      const int tok = p.lp_tokens[at];
      uint32_t st = o.status;
      float lp;
      if (tok < 0 || tok >= p.src.V) { st |= FORK_ROW_BAD_TOKEN; lp = 0.f; }
      else if (o.status) lp = o.logp;                        /* NaN for a non-finite row */
      else lp = (to_f32(row_ptr<T>(p.src, b, k)[tok]) - merged.m) + o.logp;   /* x_tok - m - ln s */
      p.lp_out[at] = lp;
      if (p.row_status) p.row_status[at] = st;
      local += lp;
    }
  }
  const float total = block_sum_f32<kNT>(local, sm.fl);
  if (threadIdx.x == 0) {
    if (p.seq_sum) p.seq_sum[b] = total;
    if (p.seq_cnt) p.seq_cnt[b] = r1 - r0;
  }
  __syncthreads();
}

template <typename T, int MODE>
__global__ void __launch_bounds__(kNT, 4) reduce_select_kernel(ReduceParams p) {
  constexpr bool WITH_T = (MODE == kModeStep);
  __shared__ Smem sm;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int R = p.hdr->R;
  if (R <= 0) return;
  const int g = blockIdx.x, C = p.C;
  const long long U = (long long)R * C;
  const int G = fork_effective_grid(U, (int)gridDim.x);     /* CTAs beyond the number of units have no work */
  if (g >= G) return;
  long long u = fork_part_begin(U, G, g);
  const long long u1 = fork_part_begin(U, G, g + 1);

  while (u < u1) {
    const int r = (int)(u / C);
    const int c0 = (int)(u - (long long)r * C);
    long long uend = (long long)(r + 1) * C;
    if (uend > u1) uend = u1;
    const int c1 = (int)(uend - (long long)r * C);
    const int e0 = c0 * FORK_CHUNK;
    int e1 = c1 * FORK_CHUNK;
    if (e1 > p.src.V) e1 = p.src.V;
    const int2 bk = p.rows[r];
    const T* row = row_ptr<T>(p.src, bk.x, bk.y);

    Part part;
    if (p.fast) {
      Acc<WITH_T> acc;
      acc.init();
      stream_direct<T, WITH_T, kNT, kUnroll>(acc, row, e0, e1);
      part = part_block_reduce<kNT>(acc.part(), sm.parts);
    } else {
      bool bad;
      part = careful_segment<T, kNT>(row, e0, e1, sm.parts, sm.fl, bad);
    }
    if (threadIdx.x == 0) {
      p.parts[r + g] = make_float4(part.m, part.s, part.t, __int_as_float(part.idx));
      __threadfence();
      const int old = atomicAdd(p.ticket + bk.x, 1);
      sm.flag = (old + 1 == p.expected[bk.x]) ? 1 : 0;
    }
    __syncthreads();
    const int last = sm.flag;
    __syncthreads();
    if (last) {                                   /* every part of sequence b has been delivered */
      __threadfence();
      if (MODE == kModeStep) finalize_step_sequence<T>(p, sm, U, G, bk.x);
      else finalize_logprob_sequence<T>(p, sm, U, G, bk.x);
    }
    u = uend;
  }
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

struct DeviceInfo { int sms = 0; int occ[2][2] = {{0, 0}, {0, 0}}; };
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
    d.sms = sms;
  }
  *out = &d;
  return true;
}

static int grid_size(const DeviceInfo& d, int dtype, int mode) {
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

static cudaError_t launch_reduce_inner(const ReduceParams& rp, int dtype, int mode, int G, cudaStream_t st) {
  const bool pdl = g_tune[FORK_TUNE_PDL].load() != 0;
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

static fork_status step_impl(const fork_step_args* a, const int32_t* lo, const int32_t* hi, void* ws,
                             cudaStream_t st) {
  DeviceInfo* dev;
  if (!device_info(&dev)) return FORK_ERR_CUDA;
  WsView w = ws_view(ws, a->B, a->Lt);
  const int mode = kModeStep;
  const int G = grid_size(*dev, a->dtype, mode);
  const int C = (a->V + FORK_CHUNK - 1) / FORK_CHUNK;

  SetupParams sp;
  memset(&sp, 0, sizeof(sp));
  sp.flags = a->mask; sp.lo = lo; sp.hi = hi;
  sp.B = a->B; sp.Lt = a->Lt; sp.pos0 = a->pos0; sp.Ll = a->Ll; sp.C = C; sp.G = G;
  sp.hdr = w.hdr; sp.seq_off = w.seq_off; sp.expected = w.expected; sp.ticket = w.ticket; sp.rows = w.rows;
  sp.n_unmasked = a->n_unmasked; sp.is_fallback = a->is_fallback; sp.fallback_pos = a->fallback_pos;
  if (launch(active_set_kernel, dim3(1), dim3(kSetupNT), st, false, sp) != cudaSuccess) return FORK_ERR_CUDA;

  ReduceParams rp;
  memset(&rp, 0, sizeof(rp));
  rp.src = RowSource{a->logits, (long long)a->stride_b, (long long)a->stride_l, a->pos0, a->Ll, a->V};
  rp.B = a->B; rp.Lt = a->Lt; rp.C = C;
  rp.fast = source_is_vector_aligned(a->logits, a->stride_b, a->stride_l, a->dtype) ? 1 : 0;
  rp.hdr = w.hdr; rp.seq_off = w.seq_off; rp.expected = w.expected; rp.ticket = w.ticket;
  rp.rows = w.rows; rp.final_rec = w.final_rec; rp.parts = w.parts;
  rp.tokens = a->tokens; rp.mask = a->mask; rp.threshold = a->threshold; rp.step = a->step;
  rp.conf = a->conf; rp.cand = a->cand; rp.entropy = a->entropy; rp.logp = a->logp; rp.row_status = a->row_status;
  rp.commit_step = a->commit_step; rp.commit_fallback = a->commit_fallback; rp.commit_logp = a->commit_logp;
  rp.n_unmasked = a->n_unmasked; rp.is_fallback = a->is_fallback; rp.fallback_pos = a->fallback_pos;
  rp.nfe = a->nfe; rp.n_fallback = a->n_fallback;
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
  const int G = grid_size(*dev, a->dtype, mode);
  const int C = (a->V + FORK_CHUNK - 1) / FORK_CHUNK;
  if (cudaMemsetAsync(a->logp, 0, sizeof(float) * (size_t)a->B * a->Lt, st) != cudaSuccess) return FORK_ERR_CUDA;

  SetupParams sp;
  memset(&sp, 0, sizeof(sp));
  sp.flags = a->select; sp.lo = nullptr; sp.hi = nullptr;
  sp.B = a->B; sp.Lt = a->Lt; sp.pos0 = a->pos0; sp.Ll = a->Ll; sp.C = C; sp.G = G;
  sp.hdr = w.hdr; sp.seq_off = w.seq_off; sp.expected = w.expected; sp.ticket = w.ticket; sp.rows = w.rows;
  sp.seq_sum = a->seq_sum; sp.seq_cnt = a->seq_cnt;
  if (launch(active_set_kernel, dim3(1), dim3(kSetupNT), st, false, sp) != cudaSuccess) return FORK_ERR_CUDA;

  ReduceParams rp;
  memset(&rp, 0, sizeof(rp));
  rp.src = RowSource{a->logits, (long long)a->stride_b, (long long)a->stride_l, a->pos0, a->Ll, a->V};
  rp.B = a->B; rp.Lt = a->Lt; rp.C = C;
  rp.fast = source_is_vector_aligned(a->logits, a->stride_b, a->stride_l, a->dtype) ? 1 : 0;
  rp.hdr = w.hdr; rp.seq_off = w.seq_off; rp.expected = w.expected; rp.ticket = w.ticket;
  rp.rows = w.rows; rp.final_rec = w.final_rec; rp.parts = w.parts;
  rp.lp_tokens = a->tokens; rp.lp_out = a->logp; rp.seq_sum = a->seq_sum; rp.seq_cnt = a->seq_cnt;
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

/* ---- host-buffer entry point --------------------------------------------------------------- */
struct StagingView {
  char* logits; int32_t* tokens; uint8_t* mask; int32_t* lo; int32_t* hi;
  float* conf; int32_t* cand; float* entropy; float* logp; uint32_t* row_status;
  int32_t* commit_step; uint8_t* commit_fallback; float* commit_logp;
  int32_t* n_unmasked; uint8_t* is_fallback; int32_t* fallback_pos; int32_t* nfe; int32_t* n_fallback;
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

/* ---- host-side view of the partition, for tests ------------------------------------------- */
extern "C" int64_t fork_debug_part_begin(int64_t U, int32_t G, int32_t g) { return fork_part_begin(U, G, g); }
extern "C" int32_t fork_debug_part_owner(int64_t U, int32_t G, int64_t x) { return fork_part_owner(U, G, x); }
extern "C" int32_t fork_debug_row_parts(int64_t U, int32_t G, int32_t C, int64_t r) { return fork_row_parts(U, G, C, r); }
extern "C" int32_t fork_debug_chunk(void) { return FORK_CHUNK; }
extern "C" int32_t fork_debug_effective_grid(int64_t U, int32_t G) { return fork_effective_grid(U, G); }
