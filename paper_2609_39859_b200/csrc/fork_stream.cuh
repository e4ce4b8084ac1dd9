/*
 * The streaming kernels: direct 128-bit loads, and the bulk-copy (TMA) shared-memory ring with
 * warp-specialised producer, consumers and finaliser; the select kernel of the vocabulary-parallel step.
 */
#pragma once
#include "fork_finalize.cuh"

namespace forkd {

/* ---- kernel 2a: direct 128-bit loads (also the path for buffers that are not 16-byte aligned) -- */
struct Smem {
  Part parts[kNT / 32];
  float fl[kNT / 32];
  float bmax;
  int flag;
};

/* Candidates drawn at a temperature, guarded scalar path (buffers that are not 16-byte aligned, rows
   re-read after a non-finite result are flagged anyway): the tempered weights of segment [e0,e1) of
   `row` against M, thread t taking the vectors that belong to lane t of the draw's order. */
template <typename T>
__device__ __forceinline__ TauPart tempered_scalar(const T* row, int e0, int e1, int V, float M, float ct, int tid) {
  constexpr int VEC = 16 / (int)sizeof(T);
  const int Vf = (V / VEC) * VEC, end = min(e1, Vf);
  TauPart tp{0.f, 0.f};
  for (int vec = e0 / VEC + tid; (vec + 1) * VEC <= end; vec += kLanes)
    for (int j = 0; j < VEC; ++j) {
      const float x = to_f32(row[vec * VEC + j]);
      if (x > -INFINITY) tp.vec += exp2f((x - M) * ct);
    }
  if (tid == 0)
    for (int e = max(e0, Vf); e < e1; ++e) {
      const float x = to_f32(row[e]);
      if (x > -INFINITY) tp.tail += exp2f((x - M) * ct);
    }
  return tp;
}

template <typename T, int MODE>
__global__ void __launch_bounds__(kNT, 4) reduce_select_kernel(const __grid_constant__ ReduceParams p) {
  constexpr bool WITH_T = mode_is_step(MODE);
  constexpr bool SAMPLE = mode_is_sample(MODE);
  constexpr bool VP = mode_is_vp(MODE);
  static_assert(kNT == kLanes, "the lanes of the draw's order are the streaming threads of a CTA");
  __shared__ Smem sm;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;");
  const int R = p.hdr->R;
  if (R <= 0) return;
  const PartitionCtx c = make_partition(R, p.C, (int)gridDim.x, p.min_units);
  const int g = blockIdx.x;
  if (g >= c.G) return;                                     /* CTAs beyond the number of units have no work */
  const RowMap rm = row_map_lists(p);
  SegmentIter it;
  it.init(c, g, p.src.V);
  Segment sg;
  bool sticky = false;
  while (it.next(sg)) {
    const int2 bk = rm.bk(sg.r);
    const T* row = row_ptr<T>(p.src, bk.x, bk.y);
    Part part, mine = part_empty();
    TauPart tp{0.f, 0.f};
    bool bad = false;
    if (p.fast) {
      mine = stream_thread<T, WITH_T, kNT, kUnroll, SAMPLE>(row, sg.e0, sg.e1, threadIdx.x, threadIdx.x == 0, sticky, p.inv_tau,
                                                            p.raise_nats, &tp);
      part = part_block_reduce<kNT>(mine, sm.parts);
    } else {
      part = careful_segment<T, kNT>(row, sg.e0, sg.e1, sm.parts, sm.fl, bad);
    }
    if (SAMPLE) {
      /* every thread's tempered weights against the CTA's maximum: the part's lane sums, its trailing
         elements and its total, for whoever draws the row's candidate */
      if (threadIdx.x == 0) sm.bmax = part.m;
      __syncthreads();
      const float M = sm.bmax;
      float vec = 0.f, tl = 0.f;
      if (p.fast) {
        if (mine.m > kClamp && mine.m < INFINITY && M < INFINITY) {
          const float w = ex2_approx((mine.m - M) * p.noise_c);
          vec = tp.vec * w; tl = tp.tail * w;
        }
      } else if (!bad && M > kClamp && M < INFINITY) {
        const TauPart q = tempered_scalar<T>(row, sg.e0, sg.e1, p.src.V, M, p.noise_c, (int)threadIdx.x);
        vec = q.vec; tl = q.tail;
      }
      float* slot = p.sslots + (size_t)(sg.r + g) * kSlotStride;
      slot[threadIdx.x] = vec;
      const float total = block_sum_f32<kNT>(vec + tl, sm.fl);
      if (threadIdx.x == 0) { slot[kSlotTail] = tl; slot[kSlotTotal] = total; }
      if (threadIdx.x < 32) store_part(p, part, sg.r, g);      /* the row's maximum is taken from the parts' records */
      __threadfence();
      __syncthreads();
      if (threadIdx.x < 32) row_part_arrived<T>(p, c, sg.r, bk.x, bk.y);
    }
    if (threadIdx.x < 32) {
      const bool last = publish_part(p, part, sg.r, g, bk.x, p.expected[bk.x]);
      if (last) {                                           /* every part of sequence b has been delivered */
        const SeqHint h = load_seq_hint(p, rm, bk.x);
        if (MODE == kModeLogprob) finalize_logprob_sequence<T>(p, rm, c, bk.x, h);
        else if (VP) finalize_vp_local<T, SAMPLE>(p, rm, c, bk.x, h);
        else finalize_step_sequence<T, SAMPLE>(p, rm, c, bk.x, h);
      }
    }
  }
}

/* ---- kernel 2b: bulk-copy (TMA) shared-memory ring, warp-specialised --------------------------
 * One CTA per SM holds two such groups ("halves").  In each half warps 0..kCW-1 consume, warp kCW
 * produces, warp kCW+1 finalises.
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
constexpr int kHalves = 2;                                 /* independent producer/consumer groups per CTA */
constexpr int kHalfThreads = (kCW + 2) * 32;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr uint32_t kSpinLimitTest = 1u << 13;              /* the test-only instance gives up after a fraction of a millisecond */
__host__ __device__ constexpr int ring_stage_bytes() { return kCW * 32 * kUnroll * 16; }     /* 16 KB */

constexpr int kSegRing = 16;                               /* > stages: the producer is never that many segments ahead */
struct RingSmem {
  unsigned long long full[kMaxStages], empty[kMaxStages], mfull[kMail], mempty[kMail];
  Part mail[kMail][kMaxCW];
  float slot[kMail][kLanes];                               /* candidates at a temperature: every consumer thread's tempered weights ... */
  float tailw[kMail];                                      /* ... and those of the trailing elements, against the thread's warp's maximum */
  int2 seg_bk[kSegRing];                                   /* (sequence, position) of the producer's recent segments, for the consumers */
};
static_assert(kSegRing > kMaxStages, "segment ring shorter than the stage ring");

/* the snapshot of the active set a half takes for itself in a one-kernel step */
struct SnapSmem {
  int off[kFuseMaxB + 1];                                  /* first row of each sequence; off[B] = R */
  int lo[kFuseMaxB], hi[kFuseMaxB];                        /* the clipped block window, absolute positions */
  uint32_t bits[kFuseMaxWords];                            /* live positions, W words per sequence, bit 0 of word 0 = pos0 */
  int clipped;
};

/* shared memory of one half: its stages, its barriers and its snapshot, rounded to 1 KB */
__host__ __device__ constexpr size_t ring_half_bytes(int n_stages) {
  return ((size_t)n_stages * ring_stage_bytes() + sizeof(RingSmem) + sizeof(SnapSmem) + 1023) / 1024 * 1024;
}

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
template <uint32_t LIMIT = kSpinLimit>
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity, const ReduceParams& p) {
  for (uint32_t i = 0; i < LIMIT; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  atomicOr(&p.hdr->dev_status, FORK_DEV_TIMEOUT);
  return false;
}
__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, uint32_t bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               :: "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
/* The same copy with an L2 eviction-priority hint.  A row is read exactly once, so its lines are
   marked "evict first": what the step needs again -- the kernel's own code, mask and bounds, parts,
   tickets, the per-position outputs -- then survives in L2 while hundreds of MB of logits stream
   through it, instead of being fetched from HBM at the start and the end of every launch. */
__device__ __forceinline__ unsigned long long l2_policy_evict_first() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_copy_g2s_hint(void* dst, const void* src, uint32_t bytes, unsigned long long* bar,
                                                   unsigned long long pol) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
               :: "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(pol) : "memory");
}
/* barrier among the threads of one half (barrier 0 belongs to __syncthreads) */
__device__ __forceinline__ void half_sync(int half) {
  /* immediate barrier numbers: with a register operand the compiler reserves all sixteen */
  if (half == 0) asm volatile("bar.sync 1, %0;" :: "n"(kHalfThreads) : "memory");
  else asm volatile("bar.sync 2, %0;" :: "n"(kHalfThreads) : "memory");
}

__device__ __forceinline__ uint32_t low_bits(int n) { return n >= 32 ? 0xffffffffu : (n <= 0 ? 0u : ((1u << n) - 1u)); }

/* One-kernel step: this half's own snapshot of the active set (Algorithm 2, line 3) -- M_t restricted
   to each sequence's block window, as bitmaps, and the first row of each sequence.  Every thread of
   the half calls it; on return the snapshot is complete and visible to all of them.  The same clipping
   rules as the set-up kernel. */
struct SnapArgs { const uint8_t* mask; const int32_t* blk_lo; const int32_t* blk_hi; int B, W, Lt; RowSource src; };
__device__ __noinline__ void take_snapshot(const SnapArgs p, SnapSmem& sn, int half, int htid) {
  const int warp = htid >> 5, lane = htid & 31;
  /* This runs cold at the start of every launch (instructions are fetched at a fraction of the
     normal rate), and after a step has streamed its logits through L2 the small arrays it reads are
     usually back in HBM.  So: few instructions, and every load independent of every other -- one
     thread per (sequence, 32-position word), two 128-bit loads of mask bytes, the bytes squeezed
     to bits with SIMD compares; one trip to memory for the whole snapshot. */
  int l0 = 0, h0 = 0;
  if (htid < p.B) { l0 = p.blk_lo[htid]; h0 = p.blk_hi[htid]; }
  const int n_items = p.B * p.W;
  const int lim = min(p.Lt, p.src.pos0 + p.src.Ll);         /* positions at or past it do not exist */
  for (int it = htid; it < n_items; it += kHalfThreads) {
    const int b = it / p.W, first = p.src.pos0 + 32 * (it - b * p.W);
    const uint8_t* m = p.mask + (size_t)b * p.Lt + first;
    uint32_t word = 0u;
    if (first + 32 <= p.Lt && (reinterpret_cast<uintptr_t>(m) & 15u) == 0) {
      const uint4 a = *reinterpret_cast<const uint4*>(m), c = *reinterpret_cast<const uint4*>(m + 16);
      const uint32_t w8[8] = {a.x, a.y, a.z, a.w, c.x, c.y, c.z, c.w};
#pragma unroll
      for (int j = 0; j < 8; ++j)                            /* byte != 0 -> 0xff -> one bit each, four at a time */
        word |= (((__vcmpne4(w8[j], 0u) & 0x01010101u) * 0x01020408u) >> 24) << (4 * j);
    } else {
      for (int j = 0; j < 32; ++j)
        if (first + j < p.Lt && m[j] != 0) word |= 1u << j;
    }
    sn.bits[it] = word & low_bits(lim - first);
  }
  for (int b = htid; b < p.B; b += kHalfThreads) {          /* the same clipping rules as the set-up kernel */
    if (b != htid) { l0 = p.blk_lo[b]; h0 = p.blk_hi[b]; }
    int lo = l0, hi = h0;
    if (lo < 0) lo = 0;
    if (hi > p.Lt) hi = p.Lt;
    if (lo < p.src.pos0) lo = p.src.pos0;
    if (hi > p.src.pos0 + p.src.Ll) hi = p.src.pos0 + p.src.Ll;
    if (hi < lo) hi = lo;
    sn.lo[b] = lo; sn.hi[b] = hi;
    if ((h0 > l0) && (lo != l0 || hi != h0)) sn.clipped = 1;  /* zeroed before the CTA-wide barrier */
  }
  half_sync(half);
  if (warp == 0) {                                           /* cut each sequence's words to its window; rows and their running sum */
    int carry = 0;
    for (int b0 = 0; b0 < p.B; b0 += 32) {
      const int b = b0 + lane;
      int n = 0;
      if (b < p.B) {
        const int lo = sn.lo[b], hi = sn.hi[b];
        for (int i = 0; i < p.W; ++i) {
          const int first = p.src.pos0 + 32 * i;
          const uint32_t word = sn.bits[b * p.W + i] & low_bits(hi - first) & ~low_bits(lo - first);
          sn.bits[b * p.W + i] = word;
          n += __popc(word);
        }
      }
      int x = n;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, x, o); if (lane >= o) x += y; }
      if (b < p.B) sn.off[b + 1] = carry + x;
      carry += __shfl_sync(0xffffffffu, x, 31);
    }
    if (lane == 0) sn.off[0] = 0;
  }
  half_sync(half);
}

/* One-kernel step, finaliser warp of every half, once the snapshot is taken: count this half (its
   reads of `mask` are complete: the barrier that ended take_snapshot orders them before this); the
   half that counts itself last applies the mask updates that finalisers had to hand on; virtual
   CTA 0 reports what the set-up kernel would have.  Returns whether every virtual CTA of the launch
   has its snapshot. */
__device__ __noinline__ bool count_snapshot(const ReduceParams& p, const SnapSmem& sn, int g, int R, int G_eff) {
  const int lane = threadIdx.x & 31;
  unsigned long long old = 0ull;
  if (lane == 0)
    asm volatile("atom.acq_rel.gpu.global.add.u64 %0, [%1], 1;" : "=l"(old) : "l"(&p.ctl->started) : "memory");
  old = __shfl_sync(0xffffffffu, old, 0);
  const bool snap_done = (old + 1ull) % (unsigned long long)p.Gv == 0ull;
  if (snap_done) {
    asm volatile("fence.sc.gpu;" ::: "memory");
    for (int b = lane; b < p.B; b += 32) {
      uint32_t f;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(f) : "l"(p.ctl->deferred + b) : "memory");
      if (f) apply_deferred(p, b);
    }
  }
  if (g == 0) {
    if (lane == 0) {
      p.hdr->R = R; p.hdr->C = p.C; p.hdr->G = G_eff;
      p.hdr->dev_status = sn.clipped ? FORK_DEV_WINDOW_CLAMPED : 0u;
    }
    int idle = 0;
    for (int b = lane; b < p.B; b += 32)
      if (sn.off[b] == sn.off[b + 1]) {                       /* no live row: the sequence takes no part in the step */
        if (p.n_unmasked) p.n_unmasked[b] = 0;
        if (p.is_fallback) p.is_fallback[b] = 0;
        if (p.fallback_pos) p.fallback_pos[b] = -1;
        if (p.loop) { loop_copy_idle_cursor(p.loop, p.step, p.blk_lo, p.blk_hi, b); ++idle; }
      }
    if (p.loop) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) idle += __shfl_xor_sync(0xffffffffu, idle, o);
      if (lane == 0 && idle > 0) loop_sequences_done(p.loop, p.step, p.B, idle);
    }
  }
  return snap_done;
}

template <typename T, int MODE, bool LATE_HOOK = false>
__global__ void __launch_bounds__(kHalfThreads * kHalves, 1) reduce_select_ring_kernel(const __grid_constant__ ReduceParams p, int n_stages) {
  constexpr bool WITH_T = mode_is_step(MODE);
  constexpr bool SAMPLE = mode_is_sample(MODE);
  constexpr bool VP = mode_is_vp(MODE);
  constexpr int VEC = 16 / (int)sizeof(T);
  constexpr int kCT = kCW * 32;                              /* consumer threads */
  constexpr int kStageVecs = kCT * kUnroll;                  /* 128-bit vectors per stage */
  constexpr int kStageBytes = kStageVecs * 16;
  /* The test-only instance has two hooks (p.late_g): g + 1 > 0 makes virtual CTA g take its snapshot
     late; -(g + 1) < 0 makes the producer of virtual CTA g leave out the copy of its second stage, so
     that the bounded waits of that half run out -- with a limit short enough for a test -- and the
     give-up path can be checked: every thread of the half returns, FORK_DEV_TIMEOUT is reported,
     nothing is left in flight. */
  constexpr uint32_t kLimit = LATE_HOOK ? kSpinLimitTest : kSpinLimit;
  extern __shared__ __align__(1024) unsigned char dyn_smem_all[];
  /* One CTA per SM made of kHalves independent halves, each a complete producer / consumers /
     finaliser group with its own ring, barriers and share of the work ("virtual CTA" g).  As two
     separate CTAs on one SM the group launched first was favoured by the warp schedulers and finished
     some 15% ahead of its neighbour, which then ran the rest alone; warps of one CTA are treated
     alike. */
  const int half = (int)threadIdx.x / kHalfThreads;
  const int htid = (int)threadIdx.x % kHalfThreads;          /* thread within the half */
  unsigned char* dyn_smem = dyn_smem_all + (size_t)half * ring_half_bytes(n_stages);
  unsigned char* ring = dyn_smem;
  RingSmem& rs = *reinterpret_cast<RingSmem*>(dyn_smem + (size_t)n_stages * kStageBytes);
  SnapSmem& sn = *reinterpret_cast<SnapSmem*>(dyn_smem + (size_t)n_stages * kStageBytes + sizeof(RingSmem));
  const int warp = htid >> 5, lane = htid & 31;

  if (htid == 0) {
    sn.clipped = 0;
    for (int s = 0; s < n_stages; ++s) { mbar_init(&rs.full[s], 1); mbar_init(&rs.empty[s], kCW); }
    for (int d = 0; d < kMail; ++d) { mbar_init(&rs.mfull[d], kCW); mbar_init(&rs.mempty[d], 1); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  const int g = (int)blockIdx.x * kHalves + half;             /* the virtual CTA this half plays */
  const bool fused = p.ctl != nullptr;                        /* one-kernel step: no set-up kernel ran */
  RowMap rm = row_map_lists(p);
  if (fused) { rm.off = sn.off; rm.bits = sn.bits; rm.W = p.W; }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;");          /* the next kernel in the stream may take free SM slots */
  int R;
  if (fused) {
    if (LATE_HOOK && p.late_g == g + 1)                       /* test-only instance: this virtual CTA takes its snapshot late */
      for (int i = 0; i < 100; ++i) __nanosleep(1000);
    take_snapshot(SnapArgs{p.mask, p.blk_lo, p.blk_hi, p.B, p.W, p.Lt, p.src}, sn, half, htid);
    R = sn.off[p.B];
    if (!sn.clipped) { rm.win_lo = sn.lo; rm.win_hi = sn.hi; }
  } else {
    R = p.hdr->R;
  }
  const PartitionCtx c = make_partition(R, p.C, (int)gridDim.x * kHalves, p.min_units);
  SegmentIter it;
  Segment sg = Segment{0, 0, 0};
  bool have = false;                                          /* this half has a first segment */
  if (R > 0 && g < c.G) {
    it.init(c, g, p.src.V);
    have = it.next(sg);
  }
  bool snap_done = true;                                      /* every virtual CTA of the launch has its snapshot */
  if (fused && warp == kCW + 1) snap_done = count_snapshot(p, sn, g, R, c.G);
  if (!have) return;                                          /* no live row, or more virtual CTAs than units */

  if (warp == kCW) {
    /* ---------------- producer ---------------- */
    if (lane != 0) return;
    uint32_t n = 0, s = 0, ph = 0;                           /* stages issued, ring slot, its phase */
    bool ok = true;
    const bool hint = p.l2_evict_first != 0;
    const unsigned long long pol = l2_policy_evict_first();
    uint32_t pseg = 0, withheld = 0xffffffffu;
    for (; ok && have; have = it.next(sg), ++pseg) {
      const int2 bk = rm.bk(sg.r);
      rs.seg_bk[pseg % kSegRing] = bk;                       /* visible to the consumers through the stage's full barrier */
      const char* src = reinterpret_cast<const char*>(row_ptr<T>(p.src, bk.x, bk.y) + sg.e0);
      const uint32_t total = (uint32_t)((sg.e1 - sg.e0) / VEC) * 16u;
      for (uint32_t off = 0; off < total; off += kStageBytes, ++n) {
        const uint32_t bytes = (total - off < (uint32_t)kStageBytes) ? (total - off) : (uint32_t)kStageBytes;
        if (!mbar_wait<kLimit>(&rs.empty[s], ph ^ 1u, p)) { ok = false; break; }
        if (LATE_HOOK && p.late_g == -(g + 1) && n == 1) {
          withheld = n;                                      /* never armed, never copied: its consumers wait in vain */
        } else {
          mbar_arrive_expect_tx(&rs.full[s], bytes);
          if (hint) bulk_copy_g2s_hint(ring + (size_t)s * kStageBytes, src + off, bytes, &rs.full[s], pol);
          else bulk_copy_g2s(ring + (size_t)s * kStageBytes, src + off, bytes, &rs.full[s]);
        }
        if (++s == (uint32_t)n_stages) { s = 0; ph ^= 1u; }
      }
    }
    if (!ok) {                                               /* do not leave with copies still landing */
      const uint32_t first = n > (uint32_t)n_stages ? n - (uint32_t)n_stages : 0u;
      for (uint32_t q = first; q < n; ++q)                   /* (with the full limit: a copy that is in flight does land) */
        if (q != withheld) mbar_wait(&rs.full[q % (uint32_t)n_stages], (q / (uint32_t)n_stages) & 1u, p);
    }
    return;
  }

  if (warp < kCW) {
    /* ---------------- consumers ---------------- */
    const int ctid = htid;                                  /* 0 .. kCT-1 */
    uint32_t s = 0, ph = 0, nseg = 0;                       /* ring slot, its phase, segments done */
    bool sticky = false;                                    /* this thread has met a -inf logit before */
    for (; have; have = it.next(sg)) {
      Acc<T, WITH_T, false, SAMPLE> a;
      a.init();
      if (SAMPLE) a.set_temperature(p.inv_tau, p.raise_nats);
      const int nvec = (sg.e1 - sg.e0) / VEC;
      /* (sequence, position) of this segment: posted by the producer before the segment's first
         copy, so readable once a stage of the segment has landed; a segment shorter than one vector
         has no stage and looks its row up itself */
      for (int voff = 0; voff < nvec; voff += kStageVecs) {
        if (!mbar_wait<kLimit>(&rs.full[s], ph, p)) return;
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
        } else {
          /* the last, partly filled stage of a segment: same unrolled code, vectors past the end
             replaced by the clamp value (contributes 2^-huge = 0 to every sum and never wins the
             maximum against a finite logit; an all -inf row is re-read by the finaliser anyway) */
          uint4 v[kUnroll];
#pragma unroll
          for (int j = 0; j < kUnroll; ++j)
            v[j] = (ctid + j * kCT < nv) ? sp[ctid + j * kCT] : neutral_vector(T{});
          if (!sticky) a.template track<kUnroll>(v, sg.e0 + (voff + ctid) * VEC, kCT * VEC);
          __syncwarp();
          if (lane == 0) mbar_arrive(&rs.empty[s]);
          if (!sticky) a.template accumulate<kUnroll>(v);
        }
        if (++s == (uint32_t)n_stages) { s = 0; ph ^= 1u; }
      }
      const bool tail = (ctid == 0) && (sg.e0 + nvec * VEC < sg.e1);   /* fewer than VEC trailing elements */
      Part pt;
      TauPart tp{0.f, 0.f};
      if (tail && !sticky) {
        const int2 bk = nvec > 0 ? rs.seg_bk[nseg % kSegRing] : rm.bk(sg.r);
        const T* row = row_ptr<T>(p.src, bk.x, bk.y);
        for (int e = sg.e0 + nvec * VEC; e < sg.e1; ++e) a.one(to_f32(row[e]), e);
      }
      if (!sticky) {
        pt = a.part();
        if (SAMPLE) a.tempered(pt.m, tp.vec, tp.tail);
        if (!part_is_finite(pt)) sticky = true;
      }
      /* a thread that met -inf (now or earlier) takes its own vectors again from global memory, clamped */
      if (sticky) {
        const int2 bk = nvec > 0 ? rs.seg_bk[nseg % kSegRing] : rm.bk(sg.r);
        pt = stream_thread_clamped<T, WITH_T, kCT, SAMPLE>(row_ptr<T>(p.src, bk.x, bk.y), sg.e0, sg.e1, ctid, ctid == 0, p.inv_tau,
                                                           p.raise_nats, &tp);
      }
      __syncwarp();
      const float m_own = pt.m;
      pt = part_warp_reduce(pt);
      const uint32_t d = nseg % kMail, mph = (nseg / kMail) & 1u;
      if (SAMPLE) {
        /* this thread's tempered weights against its warp's maximum: the finaliser turns the 256 of
           them into the part's lane sums */
        float w = 0.f;
        if (m_own > kClamp && m_own < INFINITY && pt.m < INFINITY) w = ex2_approx((m_own - pt.m) * p.noise_c);
        int ok = 1;
        if (lane == 0) ok = mbar_wait<kLimit>(&rs.mempty[d], mph ^ 1u, p) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (ok) {
          rs.slot[d][ctid] = tp.vec * w;
          if (ctid == 0) rs.tailw[d] = tp.tail * w;
          __syncwarp();
          if (lane == 0) { rs.mail[d][warp] = pt; mbar_arrive(&rs.mfull[d]); }
        }
      } else if (lane == 0) {
        if (mbar_wait<kLimit>(&rs.mempty[d], mph ^ 1u, p)) {
          rs.mail[d][warp] = pt;
          mbar_arrive(&rs.mfull[d]);
        }
      }
      ++nseg;
    }
    return;
  }

  /* ---------------- finaliser ---------------- */
  uint32_t nseg = 0;
  int cur_b = -1, want = 0;
  SeqHint h = SeqHint{0, 0, -1, 0, 0, 0, 0};
  for (; have; have = it.next(sg)) {
    /* everything that does not depend on the parts is fetched while the consumers still stream */
    const int b = fused ? rm.seq_of(sg.r) : p.rows[sg.r].x;
    if (b != cur_b) {
      cur_b = b;
      h = load_seq_hint(p, rm, b);
      want = fused ? seq_expected_warp(c, h.r0, h.r1) : p.expected[b];
    }
    if (fused && !snap_done) snap_done = snapshots_complete(p);
    const uint32_t d = nseg % kMail, ph = (nseg / kMail) & 1u;
    if (!mbar_wait<kLimit>(&rs.mfull[d], ph, p)) return;
    Part pt = (lane < kCW) ? rs.mail[d][lane] : part_empty();
    const float m_warp = pt.m;                                /* lane i: the maximum of consumer warp i */
    float sv[kCW], tl = 0.f;
    if (SAMPLE) {
#pragma unroll
      for (int i = 0; i < kCW; ++i) sv[i] = rs.slot[d][i * 32 + lane];
      tl = rs.tailw[d];
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&rs.mempty[d]);
    pt = part_warp_reduce(pt);
    if (SAMPLE) {
      /* the part's lane sums of the tempered weights, against the part's maximum */
      float wq = 0.f;
      if (lane < kCW && m_warp > kClamp && m_warp < INFINITY && pt.m < INFINITY) wq = ex2_approx((m_warp - pt.m) * p.noise_c);
      float* slot = p.sslots + (size_t)(sg.r + g) * kSlotStride;
      float tot = 0.f;
#pragma unroll
      for (int i = 0; i < kCW; ++i) {
        const float v = sv[i] * __shfl_sync(0xffffffffu, wq, i);
        slot[i * 32 + lane] = v;
        tot += v;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
      const float tlv = tl * __shfl_sync(0xffffffffu, wq, 0);
      if (lane == 0) { slot[kSlotTail] = tlv; slot[kSlotTotal] = tot + tlv; }
      store_part(p, pt, sg.r, g);                             /* the row's maximum is taken from the parts' records */
      row_part_arrived<T>(p, c, sg.r, b, rm.k_of(b, sg.r));
    }
    if (publish_part(p, pt, sg.r, g, b, want)) {
      if (MODE == kModeLogprob) finalize_logprob_sequence<T>(p, rm, c, b, h);
      else if (VP) finalize_vp_local<T, SAMPLE>(p, rm, c, b, h);
      else finalize_step_sequence<T, SAMPLE>(p, rm, c, b, h, snap_done);
    }
    ++nseg;
  }
}

/* ---- vocabulary-parallel select phase: one warp per sequence on the gathered slices ---------- */
constexpr int kVpNT = 256;
template <bool SAMPLE>
__global__ void __launch_bounds__(kVpNT) vp_select_kernel(const __grid_constant__ ReduceParams p) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int b = (int)blockIdx.x * (kVpNT / 32) + (int)(threadIdx.x >> 5);
  if (b >= p.B) return;
  const RowMap rm = row_map_lists(p);
  const SeqHint h = load_seq_hint(p, rm, b);
  if (h.r1 <= h.r0) return;                                  /* no live row: the active-set kernel wrote its outputs */
  PartitionCtx c;
  c.U = 0; c.G = 1; c.C = 1; c.small = true;
  finalize_step_sequence<float, SAMPLE, true>(p, rm, c, b, h);
}

}  // namespace forkd
