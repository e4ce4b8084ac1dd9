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
constexpr int ring_stage_bytes() { return kCW * 32 * kUnroll * 16; }     /* 16 KB */

struct RingSmem {
  unsigned long long full[kMaxStages], empty[kMaxStages], mfull[kMail], mempty[kMail];
  Part mail[kMail][kMaxCW];
  KeyPart kmail[kMail][kMaxCW];
};

/* shared memory of one half: its stages and its barriers, rounded to 1 KB */
__host__ __device__ constexpr size_t ring_half_bytes(int n_stages) {
  return ((size_t)n_stages * ring_stage_bytes() + sizeof(RingSmem) + 1023) / 1024 * 1024;
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


template <typename T, int MODE>
__global__ void __launch_bounds__(kHalfThreads * kHalves, 1) reduce_select_ring_kernel(ReduceParams p, int n_stages) {
  constexpr bool WITH_T = mode_is_step(MODE);
  constexpr bool SAMPLE = (MODE == kModeSample);
  constexpr int VEC = 16 / (int)sizeof(T);
  constexpr int kCT = kCW * 32;                              /* consumer threads */
  constexpr int kStageVecs = kCT * kUnroll;                  /* 128-bit vectors per stage */
  constexpr int kStageBytes = kStageVecs * 16;
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
  const int warp = htid >> 5, lane = htid & 31;

  if (htid == 0) {
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
  const PartitionCtx c = make_partition(R, p.C, (int)gridDim.x * kHalves);
  const int g = (int)blockIdx.x * kHalves + half;             /* the virtual CTA this half plays */
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
    const int ctid = htid;                                  /* 0 .. kCT-1 */
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

}  // namespace forkd
