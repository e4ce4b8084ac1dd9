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

/* ---- candidates drawn at a temperature (Algorithm 2 line 4, tau > 0): the draw itself ----------
 * By ONE lane for its row.  The parts of the row carry the sums of the tempered weights per lane of
 * the draw's order (sslots); U2 times their total is located first among the 256 lanes (then the
 * trailing elements), then among the parts of that lane (they follow one another in index order),
 * and last among that lane's vectors inside the part, which are read again (a few dozen 16-byte
 * loads) and summed element by element.  Returns the token (an index into this buffer) and its logit;
 * `total` receives the sum of all tempered weights against M. */
template <typename T>
__device__ __forceinline__ float tempered_weight(T v, float M, float ct) {
  const float x = to_f32(v);
  return (x > -INFINITY) ? ex2_approx((x - M) * ct) : 0.f;
}

/* the slow way, for a row whose parts cannot be trusted (it was re-read by the guarded routine):
   both passes over the whole row in the draw's order */
template <typename T>
__device__ __noinline__ int draw_token_scalar(const T* row, int V, float M, float ct, float u, float& xs, float& total) {
  constexpr int VEC = 16 / (int)sizeof(T);
  const int nvec = V / VEC;
  float S = 0.f;
  for (int e = 0; e < V; ++e) S += tempered_weight(row[e], M, ct);
  total = S;
  const float target = u * S;
  float run = 0.f;
  int last = -1;
  for (int lane = 0; lane <= kLanes; ++lane) {
    const int v0 = lane < kLanes ? lane : nvec, dv = lane < kLanes ? kLanes : 1, v1 = lane < kLanes ? nvec : nvec + 1;
    for (int vec = v0; vec < v1; vec += dv)
      for (int e = vec * VEC; e < min(vec * VEC + VEC, V); ++e) {
        const float w = tempered_weight(row[e], M, ct);
        if (w > 0.f) { last = e; run += w; if (run >= target) { xs = to_f32(row[e]); return e; } }
      }
  }
  if (last < 0) last = 0;
  xs = to_f32(row[last]);
  return last;
}

/* The draw for row r (sequence b, position k), by a whole WARP, once every part of the row has stored
   its lane sums: every lane returns the token (-1: nothing in the row has weight), its logit in `xs`,
   the total of the tempered weights against the row's maximum in `total`.  Three short stretches of
   loads, each followed by a warp scan: all 256 lane sums of all parts (lane l of the warp holds lanes
   8l .. 8l+7 of the order, so a scan over the warp follows the order); the chosen lane's share of
   every part (they follow one another in index order); that lane's vectors inside the chosen part,
   at most two per lane of the warp, read again and summed element by element. */
__device__ __forceinline__ float warp_scan_incl(float v) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) { const float y = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += y; }
  return v;
}

/* Rounding left the running sum a hair short of the target: the last entry of the stretch that has
   weight stands (one lane, scalar loads; practically never reached). */
template <typename T>
__device__ __noinline__ int draw_last_with_weight(const T* row, bool fast, bool in_tail, int first, int nv, int t0, int t1, float M,
                                                  float ct, float& xs) {
  constexpr int VEC = 16 / (int)sizeof(T);
  int tok = -1;
  if (in_tail) {
    for (int e = t0; e < t1; ++e) if (tempered_weight(row[e], M, ct) > 0.f) { tok = e; xs = to_f32(row[e]); }
  } else {
    for (int i = 0; i < nv; ++i)
      for (int j = 0; j < VEC; ++j) {
        const int e = (first + i * kLanes) * VEC + j;
        if (tempered_weight(row[e], M, ct) > 0.f) { tok = e; xs = to_f32(row[e]); }
      }
  }
  return tok;
}

template <typename T>
__device__ __noinline__ int row_draw_warp(const ReduceParams& p, const PartitionCtx& c, int r, int b, int k, float& xs, float& total) {
  constexpr int VEC = 16 / (int)sizeof(T);
  const int lane = threadIdx.x & 31;
  const float ct = p.noise_c;
  const int g0 = c.owner((long long)r * c.C), n = c.owner((long long)(r + 1) * c.C - 1) - g0 + 1;
  const float4* pq = p.parts + (r + g0);
  const float* sq = p.sslots + (size_t)(r + g0) * kSlotStride;
  const T* row = row_ptr<T>(p.src, b, k);
  /* The parts' maxima (lane j holds part j's; the rare row with more than 32 parts reads them again
     as it goes) and, in the same trip to memory, stretch 1: lane sums 8*lane .. 8*lane+7 of the order
     from every part, and the trailing elements'.  The weights need the row's maximum, the loads do not. */
  const float m_lane = lane < n ? __ldcg(pq + lane).x : -INFINITY;
  float M = (m_lane == m_lane) ? m_lane : -INFINITY;
  for (int j = lane + 32; j < n; j += 32) { const float mj = __ldcg(pq + j).x; if (mj == mj) M = fmaxf(M, mj); }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  xs = M; total = 0.f;
  if (!(M > kClamp) || M == INFINITY) return -1;            /* nothing finite: the row is flagged elsewhere */
  const float w_lane = (m_lane > kClamp && m_lane < INFINITY) ? ex2_approx((m_lane - M) * ct) : 0.f;
  auto weight = [&](int j) -> float {                        /* weight of part j against the row's maximum */
    if (j < 32) return __shfl_sync(0xffffffffu, w_lane, j);
    const float mj = __ldcg(pq + j).x;
    return (mj > kClamp && mj < INFINITY) ? ex2_approx((mj - M) * ct) : 0.f;
  };
  float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  float tail = 0.f;
  for (int j0 = 0; j0 < n; j0 += 4) {                         /* four parts' loads in flight together: one trip for the usual row */
    float4 a0[4], a1[4];
    float tl[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int j = min(j0 + i, n - 1);
      const float4* q4 = reinterpret_cast<const float4*>(sq + (size_t)j * kSlotStride) + 2 * lane;
      a0[i] = __ldcg(q4); a1[i] = __ldcg(q4 + 1);
      tl[i] = __ldcg(sq + (size_t)j * kSlotStride + kSlotTail);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (j0 + i < n) {
        const float w = weight(j0 + i);
        v[0] = fmaf(w, a0[i].x, v[0]); v[1] = fmaf(w, a0[i].y, v[1]); v[2] = fmaf(w, a0[i].z, v[2]); v[3] = fmaf(w, a0[i].w, v[3]);
        v[4] = fmaf(w, a1[i].x, v[4]); v[5] = fmaf(w, a1[i].y, v[5]); v[6] = fmaf(w, a1[i].z, v[6]); v[7] = fmaf(w, a1[i].w, v[7]);
        tail = fmaf(w, tl[i], tail);
      }
    }
  }
  const float mine = ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
  const float incl = warp_scan_incl(mine);
  const float S = __shfl_sync(0xffffffffu, incl, 31) + tail;
  total = S;
  const float u = sample_uniform_token(sample_row_key(p.sample_seed, p.step, b, k));
  const float target = u * S;
  /* the first lane of the warp whose running sum reaches the target, then the lane of the order inside it */
  const unsigned hit = __ballot_sync(0xffffffffu, incl >= target);
  int slot = kLanes;                                         /* the trailing elements unless a lane takes it */
  float rest = target - __shfl_sync(0xffffffffu, incl, 31);  /* ... what is left to cover there */
  if (hit) {
    const int wl = __ffs(hit) - 1;
    float run = incl - mine;                                 /* sum of the lanes before this one's eight */
    int sl = 8 * lane + 7;                                   /* (the last of the eight if rounding leaves the sum short) */
    bool found = false;
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if (!found) { if (run + v[i] >= target || i == 7) { sl = 8 * lane + i; found = true; } else run += v[i]; }
    slot = __shfl_sync(0xffffffffu, sl, wl);
    rest = target - __shfl_sync(0xffffffffu, run, wl);
  }
  /* stretch 2: which part of the row (a lane's vectors of part j come before those of part j + 1) */
  int js = 0;
  if (n > 1) {
    js = n - 1;
    float before = 0.f;
    bool done = false;
    for (int j0 = 0; j0 < n && !done; j0 += 32) {
      const int j = j0 + lane;
      const float wj = (j0 == 0) ? w_lane : (j < n ? weight(j) : 0.f);   /* round one: lane j holds part j's weight; later rounds (j >= 32) read it again */
      const float pj = j < n ? wj * __ldcg(sq + (size_t)j * kSlotStride + slot) : 0.f;
      const float inc = warp_scan_incl(pj);
      const unsigned h2 = __ballot_sync(0xffffffffu, j < n && before + inc >= rest);
      if (h2) {
        const int wl = __ffs(h2) - 1;
        js = j0 + wl;
        rest -= before + __shfl_sync(0xffffffffu, inc - pj, wl);
        done = true;
      } else {
        before += __shfl_sync(0xffffffffu, inc, 31);
      }
    }
    if (!done) rest -= before - weight(n - 1) * __ldcg(sq + (size_t)(n - 1) * kSlotStride + slot);   /* rounding left the sum short: the last part */
  }
  /* stretch 3: the part's stretch of the row; the lane's vectors (or the trailing elements) inside it */
  const int g = g0 + js;
  int ub, ue;                                                /* the part's units, relative to the row's first */
  if (c.small) {
    ub = (int)((uint32_t)g * (uint32_t)c.U / (uint32_t)c.G) - r * c.C;
    ue = (int)((uint32_t)(g + 1) * (uint32_t)c.U / (uint32_t)c.G) - r * c.C;
  } else {
    ub = (int)(fork_part_begin(c.U, c.G, g) - (long long)r * c.C);
    ue = (int)(fork_part_begin(c.U, c.G, g + 1) - (long long)r * c.C);
  }
  ub = max(ub, 0); ue = min(ue, c.C);
  const int e0 = ub * FORK_CHUNK, e1 = min(ue * FORK_CHUNK, p.src.V);
  const int Vf = (p.src.V / VEC) * VEC;
  const bool in_tail = slot >= kLanes;
  /* entries are visited 64 vectors a round, two consecutive ones per lane of the warp, so that a scan
     over the warp follows the order; the trailing elements (fewer than a vector) are one "vector" of
     lane 0.  The running sum carries over from round to round. */
  const int first = in_tail ? 0 : e0 / VEC + slot;
  const int end_v = min(e1, Vf) / VEC;
  const int nv = in_tail ? 1 : (end_v > first ? (end_v - first + kLanes - 1) / kLanes : 0);
  float before = 0.f;
  int tok = -1;
  float x_tok = M;
  for (int base = 0; base < nv && tok < 0; base += 64) {
    float x[2 * VEC];
    float both = 0.f;
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const int i = base + 2 * lane + q;
#pragma unroll
      for (int j = 0; j < VEC; ++j) x[q * VEC + j] = -INFINITY;
      if (i < nv) {
        if (in_tail) {
          for (int j = 0; j < VEC; ++j) { const int e = max(e0, Vf) + j; if (e < e1) x[j] = to_f32(row[e]); }
        } else {
          const size_t at = (size_t)(first + i * kLanes) * VEC;
          T raw[VEC];
          if (p.fast) *reinterpret_cast<uint4*>(raw) = __ldg(reinterpret_cast<const uint4*>(row + at));
          else
            for (int j = 0; j < VEC; ++j) raw[j] = row[at + j];
#pragma unroll
          for (int j = 0; j < VEC; ++j) x[q * VEC + j] = to_f32(raw[j]);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 2 * VEC; ++j) both += (x[j] > -INFINITY) ? ex2_approx((x[j] - M) * ct) : 0.f;
    const float inc = warp_scan_incl(both);
    const unsigned hit3 = __ballot_sync(0xffffffffu, both > 0.f && before + inc >= rest);
    if (hit3) {
      const int wl = __ffs(hit3) - 1;
      int te = -1; float tx = M;
      if (lane == wl) {
        float acc = before + inc - both;
        bool got = false;
        for (int j = 0; j < 2 * VEC; ++j) {
          const float w = (x[j] > -INFINITY) ? ex2_approx((x[j] - M) * ct) : 0.f;
          if (w > 0.f && !got) {                             /* (the lane's last entry with weight stands if rounding leaves it short) */
            acc += w;
            const int q = j / VEC;
            te = in_tail ? max(e0, Vf) + j : (first + (base + 2 * lane + q) * kLanes) * VEC + (j - q * VEC);
            tx = x[j];
            got = acc >= rest;
          }
        }
      }
      tok = __shfl_sync(0xffffffffu, te, wl); x_tok = __shfl_sync(0xffffffffu, tx, wl);
    } else {
      before += __shfl_sync(0xffffffffu, inc, 31);
    }
  }
  if (tok < 0 && nv > 0) tok = draw_last_with_weight<T>(row, p.fast != 0, in_tail, first, nv, max(e0, Vf), e1, M, ct, x_tok);
  xs = x_tok;
  return tok;
}

/* After the calling warp has stored the lane sums of part (r, g): count the part in, and if it was
   the row's last, draw the row's candidate and leave it in row_draw[r] for whoever finalises the
   sequence.  Must run before the warp takes the sequence's ticket. */
template <typename T>
__device__ __forceinline__ void row_part_arrived(const ReduceParams& p, const PartitionCtx& c, int r, int b, int k) {
  const int lane = threadIdx.x & 31;
  const int n = c.owner((long long)(r + 1) * c.C - 1) - c.owner((long long)r * c.C) + 1;
  int last = 1;
  if (n > 1) {
    __threadfence();
    __syncwarp();
    if (lane == 0) {
      int old;
      asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(p.row_ticket + r) : "memory");
      last = (old + 1 == n) ? 1 : 0;
      if (last) p.row_ticket[r] = 0;                         /* zero again for the next launch */
    }
    last = __shfl_sync(0xffffffffu, last, 0);
  }
  if (last) {
    float xs, total;
    const int tok = row_draw_warp<T>(p, c, r, b, k, xs, total);
    if (lane == 0) p.row_draw[r] = make_float4(__int_as_float(tok), xs, total, 0.f);   /* released by this lane's ticket (publish_part) */
    __syncwarp();
  }
}

/* Final statistics of up to 32 rows (one per lane) of sequence b starting at row `base`.
   Rows whose streamed result is not finite are re-read by the whole warp with the guarded routine.
   With SAMPLE the candidate is the drawn token (the element holding the row's largest perturbed
   key) and confidence / log-probability are those of that token; flagged rows keep the arg-max. */
/* Rows base .. base+31 of sequence b, one per lane: the row's parts merged, rows whose streamed
   result is not finite re-read by the whole warp with the guarded routine. */
struct MergedRow {
  Part merged; int k, g0, nparts; bool valid, bad, nonfinite, reread;
};
template <typename T>
__device__ __forceinline__ MergedRow merge_rows_warp(const ReduceParams& p, const RowMap& rm, const PartitionCtx& c, int b,
                                                     int base, int r1, int k_hint) {
  const int lane = threadIdx.x & 31;
  const int r = base + lane;
  MergedRow m;
  m.valid = r < r1; m.bad = false; m.nonfinite = false; m.reread = false;
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
    if (lane == src) { m.merged = cp; m.bad = bd; m.nonfinite = nf; m.reread = true; }
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
      const T* row = row_ptr<T>(p.src, b, k);
      float total;
      int tok;
      if (m.reread) {
        const float u = sample_uniform_token(sample_row_key(p.sample_seed, p.step, b, k));
        tok = draw_token_scalar<T>(row, p.src.V, m.merged.m, p.noise_c, u, xs, total);
      } else {
        const float4 d = __ldcg(p.row_draw + r);             /* left there by the warp that delivered the row's last part */
        tok = __float_as_int(d.x); xs = d.y;
      }
      if (tok < 0) { tok = resolve_index<T>(row, m.merged.idx, p.src.V, m.merged.m); xs = m.merged.m; }   /* (rare) the arg-max stands in */
      m.merged.idx = tok;
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
    const int pos0 = p.vp_pos0_seq ? p.vp_pos0_seq[b] : p.src.pos0;
    const bool whole = lo >= 0 && hi <= p.Lt && lo >= pos0 && hi <= pos0 + p.src.Ll;
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
    float4 out, kout = make_float4(0.f, __int_as_float(kIdxNone), 0.f, 0.f);
    if (m.bad && !m.nonfinite) {
      out = make_float4(-INFINITY, 0.f, 0.f, __int_as_float(p.vocab_offset));
    } else if (m.bad) {
      out = make_float4(m.merged.m, qnan, qnan, __int_as_float(p.vocab_offset + m.merged.idx));
    } else {
      const int idx = resolve_index<T>(row, m.merged.idx, p.src.V, m.merged.m);
      out = make_float4(m.merged.m, m.merged.s, m.merged.t, __int_as_float(p.vocab_offset + idx));
      if (SAMPLE) {
        /* the slice's own draw (with U2), and the sum of its tempered weights against its maximum:
           the select phase picks the slice with U1 and takes that slice's token */
        float xs = m.merged.m, total = 0.f;
        int si;
        if (m.reread) {
          const float u = sample_uniform_token(sample_row_key(p.sample_seed, p.step, b, m.k));
          si = draw_token_scalar<T>(row, p.src.V, m.merged.m, p.noise_c, u, xs, total);
        } else {
          const float4 d = __ldcg(p.row_draw + r);
          si = __float_as_int(d.x); xs = d.y; total = d.z;
        }
        if (si < 0) { si = idx; xs = m.merged.m; }
        kout = make_float4(total, __int_as_float(p.vocab_offset + si), xs, 0.f);
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
  const size_t at = p.vp_row_stride > 0 ? (size_t)b * p.src.Ll + (size_t)(k - (p.vp_pos0_seq ? p.vp_pos0_seq[b] : p.src.pos0))
                                        : (size_t)b * p.Lt + k;
  const size_t n = p.vp_row_stride > 0 ? (size_t)p.vp_row_stride : (size_t)p.B * p.Lt;
  Part acc = part_empty();
  for (int j0 = 0; j0 < p.vp_ranks; j0 += 8) {               /* eight slices' records in flight together, merged in rank order */
    float4 q[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) q[i] = __ldg(p.vp_parts_in + (size_t)min(j0 + i, p.vp_ranks - 1) * n + at);
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if (j0 + i < p.vp_ranks) acc = part_merge(acc, part_from(q[i]));
  }
  const bool bad = !(isfinite(acc.s) && isfinite(acc.t)) || !(acc.m > -INFINITY) || acc.m == INFINITY;
  if (!SAMPLE || bad) return row_out_from(acc, bad);
  if (p.head_draw) {                                         /* fused LM-head step: the row's draw was made by head_draw_kernel */
    const float4 d = __ldg(p.head_draw + at);
    const int tok = __float_as_int(d.x);
    if (tok < 0) return row_out_from(acc, false);            /* nothing had weight: the arg-max stands in */
    acc.idx = tok;
    return row_out_sampled(acc, false, d.y);
  }
  /* the slice by inversion with U1 over the slices' tempered totals (each against its own maximum,
     re-weighted to the row's), in rank order; the token is that slice's own draw */
  const float u1 = sample_uniform_slice(sample_row_key(p.sample_seed, p.step, b, k));
  float grand = 0.f;
  for (int j = 0; j < p.vp_ranks; ++j) {
    const float mj = __ldg(p.vp_parts_in + j * n + at).x;
    if (mj > -INFINITY && mj < INFINITY) grand += __ldg(p.vp_keys_in + j * n + at).x * ex2_approx((mj - acc.m) * p.noise_c);
  }
  const float target = u1 * grand;
  float run = 0.f, xs = acc.m;
  int bidx = acc.idx;
  for (int j = 0; j < p.vp_ranks; ++j) {
    const float mj = __ldg(p.vp_parts_in + j * n + at).x;
    if (!(mj > -INFINITY && mj < INFINITY)) continue;
    const float4 q = __ldg(p.vp_keys_in + j * n + at);
    const float wj = q.x * ex2_approx((mj - acc.m) * p.noise_c);
    if (!(wj > 0.f)) continue;
    run += wj;
    bidx = __float_as_int(q.y); xs = q.z;                     /* (the last slice with weight stands if rounding leaves the sum short) */
    if (run >= target) break;
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
__device__ __forceinline__ void store_part(const ReduceParams& p, const Part& part, int r, int g) {
  if ((threadIdx.x & 31) == 0) p.parts[r + g] = make_float4(part.m, part.s, part.t, __int_as_float(part.idx));
}
__device__ __forceinline__ bool publish_part(const ReduceParams& p, const Part& part, int r, int g, int b, int want) {
  int last = 0;
  if ((threadIdx.x & 31) == 0) {
    p.parts[r + g] = make_float4(part.m, part.s, part.t, __int_as_float(part.idx));
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
