/*
 * What happens once every part of a sequence has arrived: merging the parts of a row, the unmask
 * rule (Algorithm 2, lines 6-9) with its fallback orders, scoring (Section 3.2), and the two phases of the
 * vocabulary-parallel step.
 */
#pragma once
#include "fork_params.cuh"

namespace forkd {

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
__device__ __forceinline__ MergedRow merge_rows_warp(const ReduceParams& p, const RowMap& rm, const PartitionCtx& c, int b,
                                                     int base, int r1, int k_hint) {
  const int lane = threadIdx.x & 31;
  const int r = base + lane;
  MergedRow m;
  m.valid = r < r1; m.bad = false; m.nonfinite = false;
  m.merged = part_empty();
  m.k = 0; m.g0 = 0; m.nparts = 0;
  bool redo = false;
  if (m.valid) { m.k = (k_hint >= 0) ? k_hint : rm.k_of(b, r); m.merged = merge_row_parts(p, c, r, m.g0, m.nparts); }
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
__device__ __forceinline__ RowOut finalize_rows_warp(const ReduceParams& p, const RowMap& rm, const PartitionCtx& c, int b,
                                                     int base, int r1, Part& merged, int& k, int k_hint) {
  const int lane = threadIdx.x & 31;
  const int r = base + lane;
  MergedRow m = merge_rows_warp<T>(p, rm, c, b, base, r1, k_hint);
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
struct SeqHint {
  int r0, r1, k;
  int cur_lo, cur_hi;        /* decode loop: the sequence's cursor if its block still holds a masked position after the step ... */
  int nxt_lo, nxt_hi;        /* ... and if it does not: the next block that holds one (gen_hi, gen_hi when there is none) */
};
__device__ __forceinline__ SeqHint load_seq_hint(const ReduceParams& p, const RowMap& rm, int b) {
  SeqHint h;
  rm.seq_range(b, h.r0, h.r1);
  const int lane = (int)(threadIdx.x & 31);
  const int r = h.r0 + lane;
  h.k = (r < h.r1) ? rm.k_of(b, r) : -1;
  h.cur_lo = h.cur_hi = h.nxt_lo = h.nxt_hi = 0;
  if (p.loop) {
    /* Section 4.1: blocks are decoded in order, and a block is left when it holds no masked position
       any more.  Which block comes next does not depend on this step (it touches the current block
       only), so it is looked up now, while the row's parts are still on their way. */
    const LoopCtl* L = p.loop;
    const int lo = rm.win_lo ? rm.win_lo[b] : p.blk_lo[b], hi = rm.win_hi ? rm.win_hi[b] : p.blk_hi[b];
    const int gen_hi = L->gen_hi, bl = L->block_len;
    h.cur_lo = lo; h.cur_hi = hi;
    /* a window that reaches outside the logits buffer keeps masked positions the steps cannot see:
       its cursor never moves on (the loop then ends at its step limit) */
    const bool whole = lo >= 0 && hi <= p.Lt && lo >= p.src.pos0 && hi <= p.src.pos0 + p.src.Ll;
    h.nxt_lo = h.nxt_hi = whole ? gen_hi : -1;
    if (whole) {
      for (int s = lo + bl; s < gen_hi; s += bl) {
        const int e = min(s + bl, gen_hi);
        unsigned any = 0u;
        for (int k0 = s; k0 < e; k0 += 32) {
          const int k = k0 + lane;
          any |= __ballot_sync(0xffffffffu, k < e && p.mask[(size_t)b * p.Lt + k] != 0);
        }
        if (any) { h.nxt_lo = s; h.nxt_hi = e; break; }
      }
    }
  }
  return h;
}

/* Decode loop, sequence b after its step committed `committed` of its `live` positions: the cursor
   for the next step goes into the other buffer, a finished sequence leaves the count of unfinished
   ones, and the sequence is counted as dealt with.  One thread. */
__device__ __forceinline__ void loop_advance_cursor(const ReduceParams& p, int b, const SeqHint& h, int live, int committed) {
  LoopCtl* L = p.loop;
  const bool leaves = committed == live && h.nxt_lo >= 0;
  const int nlo = leaves ? h.nxt_lo : h.cur_lo, nhi = leaves ? h.nxt_hi : h.cur_hi;
  const int nxt = ((p.step - L->step0) + 1) & 1;
  L->lo[nxt][b] = nlo; L->hi[nxt][b] = nhi;
  if (nlo >= nhi) atomicSub(&L->remaining, 1);
  loop_sequences_done(L, p.step, p.B, 1);
}

/* Parts sequence b will receive (rows r0 .. r1-1 under partition c), by the whole warp: what the
   set-up kernel stores in `expected` when there is one. */
__device__ __forceinline__ int seq_expected_warp(const PartitionCtx& c, int r0, int r1) {
  int parts = 0;
  for (int r = r0 + (int)(threadIdx.x & 31); r < r1; r += 32)
    parts += c.owner((long long)(r + 1) * c.C - 1) - c.owner((long long)r * c.C) + 1;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) parts += __shfl_xor_sync(0xffffffffu, parts, o);
  return parts;
}

/* ---- one-kernel step: when may `mask` be modified ------------------------------------------- */
__device__ unsigned long long g_mask_handovers;               /* mask updates handed on since the library was loaded (all workspaces) */
__device__ __forceinline__ bool snapshots_complete(const ReduceParams& p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(&p.ctl->started) : "memory");
  return v % (unsigned long long)p.Gv == 0ull;
}
/* One thread: clear the mask at the positions sequence b's finaliser recorded, then drop the flag. */
__device__ __forceinline__ void apply_deferred(const ReduceParams& p, int b) {
  for (int i = 0; i < p.W; ++i) {
    uint32_t x = __ldcg(p.commit_bits + (size_t)b * p.W + i);
    while (x) {
      const int bit = __ffs(x) - 1;
      x &= x - 1;
      p.mask[(size_t)b * p.Lt + p.src.pos0 + 32 * i + bit] = 0;
    }
  }
  atomicExch(p.ctl->deferred + b, 0u);
}

/* ---- vocabulary-parallel slices ------------------------------------------------------------- */
/* Local phase: what this slice contributes to every live row of sequence b, written per position
   for the exchange: (m, s, t2, global index of the lowest arg-max), s = NaN when the slice holds
   NaN or +inf, the neutral element (m = -inf, s = t2 = 0) when it holds nothing but -inf; with
   stochastic candidates also (largest perturbed key, global index of its entry, that logit). */
template <typename T, bool SAMPLE>
__device__ void finalize_vp_local(const ReduceParams& p, const RowMap& rm, const PartitionCtx& c, int b, const SeqHint& h) {
  const int lane = threadIdx.x & 31;
  const float qnan = __int_as_float(0x7fc00000);
  for (int base = h.r0; base < h.r1; base += 32) {
    const int r = base + lane;
    MergedRow m = merge_rows_warp<T>(p, rm, c, b, base, h.r1, base == h.r0 ? h.k : -1);
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
    if (p.vp_peers > 0) {
      /* the exchange itself: plain 16-byte stores into every rank's gather buffer, the remote ones
         over NVLink while the rest of the reduction goes on; nothing is ever loaded from a peer */
      const size_t slot = (size_t)p.vp_rank * ((size_t)p.B * p.Lt) + at;
      for (int j = 0; j < p.vp_peers; ++j) {
        p.vp_peer_tab->part[j][slot] = out;
        if (SAMPLE) p.vp_peer_tab->key[j][slot] = kout;
      }
    } else {
      p.vp_part[at] = out;
      if (SAMPLE) p.vp_key[at] = kout;
    }
  }
}

/* Select phase: the statistics of rows base .. base+31 of sequence b from the gathered slices,
   merged in rank order (ascending vocabulary offset; ties keep the lowest global index). */
template <bool SAMPLE>
__device__ __forceinline__ RowOut gathered_rows_warp(const ReduceParams& p, const RowMap& rm, int b, int base, int r1, int& k,
                                                     int k_hint) {
  const int lane = threadIdx.x & 31;
  const int r = base + lane;
  k = 0;
  if (r >= r1) return row_out_from(part_empty(), true);
  k = (k_hint >= 0) ? k_hint : rm.k_of(b, r);
  const size_t at = p.vp_row_stride > 0 ? (size_t)b * p.src.Ll + (size_t)(k - p.src.pos0) : (size_t)b * p.Lt + k;
  const size_t n = p.vp_row_stride > 0 ? (size_t)p.vp_row_stride : (size_t)p.B * p.Lt;
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
   comparison order picks; write tokens, mask and the per-token records.  `snapshots_done`: the
   caller already knows that `mask` may be modified (always so when a set-up kernel took the
   snapshot). */
template <typename T, bool SAMPLE, bool GATHERED = false>
__device__ void finalize_step_sequence(const ReduceParams& p, const RowMap& rm, const PartitionCtx& c, int b, const SeqHint& h,
                                       bool snapshots_done = true) {
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
    const RowOut o = GATHERED ? gathered_rows_warp<SAMPLE>(p, rm, b, base, r1, k, base == r0 ? h.k : -1)
                              : finalize_rows_warp<T, true, SAMPLE>(p, rm, c, b, base, r1, merged, k, base == r0 ? h.k : -1);
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
  /* one-kernel step: a virtual CTA that has not started yet must still find M_t in `mask` */
  const bool direct = !p.ctl || snapshots_done || snapshots_complete(p);
  if (!direct) {
    for (int i = lane; i < p.W; i += 32) p.commit_bits[(size_t)b * p.W + i] = 0u;
    __syncwarp();
  }
  int count = 0, pick_k = -1;
  for (int base = r0; base < r1; base += 32) {
    const int r = base + lane;
    bool commit = false;
    if (r < r1) {
      const float4 f = one_batch ? keep : p.final_rec[r];    /* written by this same lane above */
      commit = fb ? (r == pick) : (f.x > p.threshold);       /* the fallback position, or the threshold set */
      if (commit) {
        const int k = one_batch ? keep_k : rm.k_of(b, r);
        const size_t at = (size_t)b * p.Lt + k;
        if (fb) pick_k = k;
        p.tokens[at] = __float_as_int(f.z);
        if (direct) p.mask[at] = 0;
        else atomicOr(p.commit_bits + (size_t)b * p.W + ((k - p.src.pos0) >> 5), 1u << ((k - p.src.pos0) & 31));
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
  if (p.loop && lane == 0) loop_advance_cursor(p, b, h, r1 - r0, count);
  if (!direct) {
    /* hand the mask update on: record, raise the flag, look again.  The CTA that counts itself last
       raises its count, then reads the flags; with a sequentially consistent fence on both sides
       at least one of the two sees the other. */
    __syncwarp();
    if (lane == 0) {
      atomicAdd(&g_mask_handovers, 1ull);
      __threadfence();
      atomicExch(p.ctl->deferred + b, 1u);
      asm volatile("fence.sc.gpu;" ::: "memory");
      if (snapshots_complete(p)) apply_deferred(p, b);
    }
  }
}

/* Scoring for one sequence by one warp: log q(token) = x_tok - m - ln s at every selected position
   and their sum (Section 3.2 of the paper: the likelihood terms of the ForkGRPO ratio). */
template <typename T>
__device__ void finalize_logprob_sequence(const ReduceParams& p, const RowMap& rm, const PartitionCtx& c, int b, const SeqHint& h) {
  const int lane = threadIdx.x & 31;
  const int r0 = h.r0, r1 = h.r1;
  float local = 0.f;
  for (int base = r0; base < r1; base += 32) {
    Part merged; int k;
    const RowOut o = finalize_rows_warp<T, false, false>(p, rm, c, b, base, r1, merged, k, base == r0 ? h.k : -1);
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
    if (last) p.ticket[b] = 0;               /* nobody else touches it again in this launch: clean for the next one */
  }
  return __shfl_sync(0xffffffffu, last, 0) != 0;
}

/* The rows a CTA works on: its contiguous unit range cut at row boundaries. */
struct Segment { int r, e0, e1; };
struct SegmentIter {
  long long u, u1; int C, V;
  __device__ __forceinline__ void init(const PartitionCtx& c, int g, int V_) {
    if (c.small) {                                           /* g*U < 2^32: two 32-bit divisions instead of two 64-bit ones */
      u = (long long)((uint32_t)g * (uint32_t)c.U / (uint32_t)c.G);
      u1 = (long long)((uint32_t)(g + 1) * (uint32_t)c.U / (uint32_t)c.G);
    } else {
      u = fork_part_begin(c.U, c.G, g); u1 = fork_part_begin(c.U, c.G, g + 1);
    }
    C = c.C; V = V_;
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

}  // namespace forkd
