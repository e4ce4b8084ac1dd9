/*
 * The one-CTA set-up kernels: the active set of a step (Algorithm 2, line 3) and the block cursors of
 * the semi-autoregressive decode loop (Section 4.1 Setup).
 */
#pragma once
#include "fork_params.cuh"

namespace forkd {

/* ---- kernel 1: the active set -------------------------------------------------------------- */
/* One CTA.  live(b,k) = flags[b,k] != 0 and k inside the sequence's window (block bounds clipped
   to the sequence buffer and to the positions the logits buffer covers). */
struct SetupParams {
  const uint8_t* flags;              /* mask (step) or select (log-probability) */
  const int32_t* lo; const int32_t* hi;   /* NULL: the whole sequence */
  int B, Lt, pos0, Ll, C, G, min_units;
  WsHeader* hdr; int32_t* seq_off; int32_t* expected; int32_t* ticket; int2* rows;
  /* outputs for sequences without a live row */
  int32_t* n_unmasked; uint8_t* is_fallback; int32_t* fallback_pos;   /* step mode */
  float* seq_sum; int32_t* seq_cnt;                                   /* log-probability mode */
  LoopCtl* loop; int step;                                            /* a step of fork_decode_loop (else NULL) */
  const int32_t* pos0_seq;           /* NULL, or [B]: the position of row 0 of each sequence's window (instead of pos0) */
};

__device__ __forceinline__ void seq_window(const SetupParams& p, int b, int& lo, int& hi, bool& clipped) {
  int l0 = p.lo ? p.lo[b] : 0, h0 = p.hi ? p.hi[b] : p.Lt;
  lo = l0; hi = h0;
  if (lo < 0) lo = 0;
  if (hi > p.Lt) hi = p.Lt;
  const int pos0 = p.pos0_seq ? p.pos0_seq[b] : p.pos0;
  if (lo < pos0) lo = pos0;
  if (hi > pos0 + p.Ll) hi = pos0 + p.Ll;
  clipped = (h0 > l0) && (lo != l0 || hi != h0);
  if (hi < lo) hi = lo;
}

/* sequences whose counts fit in shared memory (more: counts go through global memory); small enough
   that this CTA fits on an SM beside a CTA of the bulk-copy kernel, so that with programmatic
   dependent launch it is already resident when the step before it ends */
constexpr int kSetupMaxB = 2048;

__global__ void __launch_bounds__(kSetupNT, 1) active_set_kernel(SetupParams p) {
  /* with programmatic dependent launch this grid may already be resident while the kernel before
     it in the stream (normally the previous step) is still running: nothing is read or written
     before that kernel has completed; the streaming kernel of this step may be made resident now */
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;");
  __shared__ int sh_cnt[kSetupMaxB + 1];          /* sh_cnt[b+1] = live rows of b, then their inclusive scan */
  __shared__ int sh_warp[kSetupNT / 32];
  __shared__ int sh_carry, sh_idle;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = kSetupNT / 32;
  if (tid == 0) sh_idle = 0;
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
  const PartitionCtx c = make_partition(R, p.C, p.G, p.min_units);
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
        if (p.loop) { loop_copy_idle_cursor(p.loop, p.step, p.lo, p.hi, b); atomicAdd(&sh_idle, 1); }
      }
    }
  }
  clipped_any = __syncthreads_or((int)clipped_any);
  if (tid == 0) {
    p.hdr->dev_status = clipped_any ? FORK_DEV_WINDOW_CLAMPED : 0u;
    if (p.loop && sh_idle > 0) { __threadfence(); loop_sequences_done(p.loop, p.step, p.B, sh_idle); }
  }
}

/* ---- decode-loop helpers ------------------------------------------------------------------- */
struct CursorParams {
  const uint8_t* mask; int B, Lt, gen_lo, gen_hi, block_len;
  int32_t* lo; int32_t* hi; LoopCtl* loop; int init;
};

/* Start of a decode loop.  One warp per sequence: the first block that holds a masked position;
   lo = hi = gen_hi when there is none.  Sets up the loop state and reports the number of
   unfinished sequences to the host under the ticket before the first step's. */
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
  if (tid == 0) {
    LoopCtl* L = p.loop;
    L->remaining = sh_remaining; L->seq_done = 0;
    const unsigned long long v = ((unsigned long long)(uint32_t)sh_remaining << 32) | (unsigned long long)(L->ticket0 - 1u);
    *reinterpret_cast<volatile unsigned long long*>(L->flags + (kLoopFlags - 1)) = v;
    __threadfence_system();
  }
}

}  // namespace forkd
