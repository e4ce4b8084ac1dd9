/*
 * Device-side building blocks of the vocabulary reduction.
 *
 * For one logits row the step needs (Section 2 of the paper: c = q(x_0 | x_t) with x_0 the
 * arg-max; token entropy of Section 3.1; log-probability of Section 3.2)
 *     m = max_v x_v,  a = lowest arg-max,  s = sum_v e^{x_v-m},  t = sum_v (x_v-m) e^{x_v-m}
 * from which  conf = 1/s,  H = ln s - t/s,  log p(a) = -ln s.
 *
 * Everything is kept in the base-2 domain: with L = log2(e), y = (x-m)*L, e = 2^y, the
 * accumulators are s = sum e and t2 = sum y*e (t = t2 * ln 2).  Two accumulators with different
 * reference maxima merge associatively:
 *     M = max(m1,m2), d_i = (m_i-M)*L, w_i = 2^{d_i}:  s = sum w_i s_i,  t2 = sum w_i (t2_i + d_i s_i).
 *
 * Non-finite inputs: a logit of -inf is clamped to FORK_CLAMP (about -1e38) by a NaN-propagating
 * max, so it contributes 2^(-huge) = 0 to both sums at no extra cost.  NaN and +inf end up as a
 * NaN in s or t2 (NaN*0 stays NaN in every rescale), which the caller detects once per row and
 * then re-reads that row with the guarded scalar routine.
 */
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <math.h>

namespace forkd {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kClamp = -9.9692e37f;              /* bf16 0xFE96 widened: the clamp value for -inf */
constexpr uint32_t kClampBf16x2 = 0xFE96FE96u;
constexpr int kIdxNone = 0x7fffffff;

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max_nan_f32(float a, float b) {
  float d;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}
__device__ __forceinline__ uint32_t max_nan_bf16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
/* streaming 128-bit load: read-only path, do not keep the line in L1 */
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

struct bf16_t { uint16_t bits; };                   /* storage type tag for bf16 logits */
__device__ __forceinline__ float to_f32(bf16_t v) { return __uint_as_float(((uint32_t)v.bits) << 16); }
__device__ __forceinline__ float to_f32(float v) { return v; }

/* ------------------------------------------------------------------------------------------ */
/* A reduced piece of a row: what a thread, a warp, a CTA or a row ends up with.               */
struct Part {
  float m;    /* reference max (-inf when nothing was accumulated) */
  float s;    /* sum 2^{(x-m)L} */
  float t;    /* sum (x-m)L * 2^{(x-m)L} */
  int idx;    /* lowest index attaining m (kIdxNone when empty) */
};

__device__ __forceinline__ Part part_empty() { return Part{-INFINITY, 0.f, 0.f, kIdxNone}; }

/* (s,t) of `a` re-expressed against the larger reference M */
__device__ __forceinline__ void part_rebase(const Part& a, float M, float& s, float& t) {
  if (a.m == M) { s = a.s; t = a.t; return; }
  if (a.m <= kClamp) { s = a.s * 0.f; t = a.t * 0.f; return; }   /* only -inf so far: weight 0, NaN kept */
  float d = (a.m - M) * kLog2e;
  float w = ex2_approx(d);
  s = w * a.s;
  t = w * fmaf(d, a.s, a.t);
}

__device__ __forceinline__ Part part_merge(const Part& a, const Part& b) {
  Part o;
  bool bwins = (b.m > a.m) || (b.m == a.m && b.idx < a.idx);
  o.idx = bwins ? b.idx : a.idx;
  o.m = fmaxf(a.m, b.m);
  float sa, ta, sb, tb;
  part_rebase(a, o.m, sa, ta);
  part_rebase(b, o.m, sb, tb);
  o.s = sa + sb;
  o.t = ta + tb;
  return o;
}

__device__ __forceinline__ Part part_shfl_down(const Part& p, int delta) {
  Part q;
  q.m = __shfl_down_sync(0xffffffffu, p.m, delta);
  q.s = __shfl_down_sync(0xffffffffu, p.s, delta);
  q.t = __shfl_down_sync(0xffffffffu, p.t, delta);
  q.idx = __shfl_down_sync(0xffffffffu, p.idx, delta);
  return q;
}

/* Fixed-shape tree over the CTA; the result is valid in thread 0 only.  `sh` holds NT/32 parts.
   Contains two __syncthreads(): call from uniform control flow. */
template <int NT>
__device__ __forceinline__ Part part_block_reduce(Part p, Part* sh) {
  constexpr int NW = NT / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) p = part_merge(p, part_shfl_down(p, o));
  __syncthreads();                         /* previous users of sh are done */
  if (lane == 0) sh[warp] = p;
  __syncthreads();
  if (warp == 0) {
    p = (lane < NW) ? sh[lane] : part_empty();
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) p = part_merge(p, part_shfl_down(p, o));
  }
  return p;
}

/* ------------------------------------------------------------------------------------------ */
/* Per-thread streaming accumulator with a lazily raised reference max and 4 independent lanes. */
template <bool WITH_T>
struct Acc {
  float m, nmL;          /* reference max and -m*L */
  int idx;
  float s[4], t[4];

  __device__ __forceinline__ void init() {
    m = -INFINITY; nmL = INFINITY; idx = kIdxNone;
#pragma unroll
    for (int j = 0; j < 4; ++j) { s[j] = 0.f; t[j] = 0.f; }
  }
  /* raise the reference to newm (> m): s *= w, t = w (t + d s) with d = (m-newm) L */
  __device__ __forceinline__ void raise(float newm) {
    if (m <= kClamp) {
#pragma unroll
      for (int j = 0; j < 4; ++j) { s[j] *= 0.f; if (WITH_T) t[j] *= 0.f; }
    } else {
      float d = (m - newm) * kLog2e;
      float w = ex2_approx(d);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (WITH_T) t[j] = w * fmaf(d, s[j], t[j]);
        s[j] *= w;
      }
    }
    m = newm;
    nmL = -newm * kLog2e;
  }
  __device__ __forceinline__ void add(int j, float x) {
    float y = fmaf(x, kLog2e, nmL);
    float e = ex2_approx(y);
    s[j] += e;
    if (WITH_T) t[j] = fmaf(y, e, t[j]);
  }
  /* one element (already clamped), at vocabulary index i; used for ragged tails */
  __device__ __forceinline__ void one(float x, int i) {
    if (x > m) { idx = i; raise(x); }
    add(0, x);
  }
  __device__ __forceinline__ Part part() const {
    Part p;
    p.m = m; p.idx = idx;
    p.s = (s[0] + s[1]) + (s[2] + s[3]);
    p.t = WITH_T ? (t[0] + t[1]) + (t[2] + t[3]) : 0.f;
    return p;
  }
};

/* 8 bf16 logits starting at vocabulary index base */
template <bool WITH_T>
__device__ __forceinline__ void acc_vec(Acc<WITH_T>& a, uint4 v, int base, bf16_t) {
  v.x = max_nan_bf16x2(v.x, kClampBf16x2);
  v.y = max_nan_bf16x2(v.y, kClampBf16x2);
  v.z = max_nan_bf16x2(v.z, kClampBf16x2);
  v.w = max_nan_bf16x2(v.w, kClampBf16x2);
  const float x0 = bf16_lo(v.x), x1 = bf16_hi(v.x), x2 = bf16_lo(v.y), x3 = bf16_hi(v.y);
  const float x4 = bf16_lo(v.z), x5 = bf16_hi(v.z), x6 = bf16_lo(v.w), x7 = bf16_hi(v.w);
  const float vmax = fmaxf(fmaxf(fmaxf(x0, x1), fmaxf(x2, x3)), fmaxf(fmaxf(x4, x5), fmaxf(x6, x7)));
  if (vmax > a.m) {                      /* rare after the first few vectors */
    int j = 7;
    if (x6 == vmax) j = 6;
    if (x5 == vmax) j = 5;
    if (x4 == vmax) j = 4;
    if (x3 == vmax) j = 3;
    if (x2 == vmax) j = 2;
    if (x1 == vmax) j = 1;
    if (x0 == vmax) j = 0;
    a.idx = base + j;
    a.raise(vmax);
  }
  a.add(0, x0); a.add(1, x1); a.add(2, x2); a.add(3, x3);
  a.add(0, x4); a.add(1, x5); a.add(2, x6); a.add(3, x7);
}

/* 4 fp32 logits starting at vocabulary index base */
template <bool WITH_T>
__device__ __forceinline__ void acc_vec(Acc<WITH_T>& a, uint4 v, int base, float) {
  const float x0 = max_nan_f32(__uint_as_float(v.x), kClamp), x1 = max_nan_f32(__uint_as_float(v.y), kClamp);
  const float x2 = max_nan_f32(__uint_as_float(v.z), kClamp), x3 = max_nan_f32(__uint_as_float(v.w), kClamp);
  const float vmax = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
  if (vmax > a.m) {
    int j = 3;
    if (x2 == vmax) j = 2;
    if (x1 == vmax) j = 1;
    if (x0 == vmax) j = 0;
    a.idx = base + j;
    a.raise(vmax);
  }
  a.add(0, x0); a.add(1, x1); a.add(2, x2); a.add(3, x3);
}

/* Stream elements [e0,e1) of one row with 128-bit loads; e0 is a multiple of the vector width and
   the row base is 16-byte aligned.  Threads take vectors tid, tid+NT, ... so each thread sees
   ascending indices (strict '>' then keeps the lowest arg-max). */
template <typename T, bool WITH_T, int NT, int UNROLL>
__device__ __forceinline__ void stream_direct(Acc<WITH_T>& a, const T* row, int e0, int e1) {
  constexpr int VEC = 16 / (int)sizeof(T);
  const uint4* p = reinterpret_cast<const uint4*>(row + e0);
  const int nvec = (e1 - e0) / VEC;
  int i = threadIdx.x;
  for (; i + (UNROLL - 1) * NT < nvec; i += UNROLL * NT) {
    uint4 v[UNROLL];
#pragma unroll
    for (int j = 0; j < UNROLL; ++j) v[j] = ld_stream(p + i + j * NT);
#pragma unroll
    for (int j = 0; j < UNROLL; ++j) acc_vec(a, v[j], e0 + (i + j * NT) * VEC, T{});
  }
  for (; i < nvec; i += NT) acc_vec(a, ld_stream(p + i), e0 + i * VEC, T{});
  if (threadIdx.x == 0) {                                  /* fewer than VEC trailing elements */
    for (int e = e0 + nvec * VEC; e < e1; ++e) a.one(max_nan_f32(to_f32(row[e]), kClamp), e);
  }
}

/* ------------------------------------------------------------------------------------------ */
/* small CTA-wide helpers (all contain __syncthreads: uniform control flow only)               */
template <int NT>
__device__ __forceinline__ float block_sum_f32(float v, float* sh /*[NT/32]*/) {
  constexpr int NW = NT / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  float r = 0.f;
  if (warp == 0) {
    r = (lane < NW) ? sh[lane] : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) r += __shfl_down_sync(0xffffffffu, r, o);
    if (lane == 0) sh[0] = r;
  }
  __syncthreads();
  r = sh[0];
  return r;                                                /* same value in every thread */
}

/* Guarded scalar reduction of elements [e0,e1) of one row by the whole CTA: two passes, every
   special value handled explicitly.  Works for any alignment.  Returns the same Part in every
   thread; `bad` is set when the segment holds NaN or +inf, or nothing but -inf (then s = NaN). */
template <typename T, int NT>
__device__ Part careful_segment(const T* row, int e0, int e1, Part* shp, float* shf, bool& bad) {
  float m = -INFINITY;
  int idx = -1, isbad = 0;
  for (int i = e0 + threadIdx.x; i < e1; i += NT) {
    float x = to_f32(row[i]);
    if (x != x) { isbad = 1; continue; }
    if (x == INFINITY) isbad = 1;
    if (idx < 0 || x > m) { m = x; idx = i; }
  }
  Part p{m, 0.f, 0.f, idx < 0 ? kIdxNone : idx};
  p = part_block_reduce<NT>(p, shp);               /* only (m, idx) matter here; s = t = 0 */
  if (threadIdx.x == 0) shp[0] = p;
  isbad = __syncthreads_or(isbad);
  p = shp[0];
  if (isbad || p.idx == kIdxNone || p.m == -INFINITY) {
    bad = true;
    Part r{p.m, __int_as_float(0x7fc00000), __int_as_float(0x7fc00000), p.idx == kIdxNone ? 0 : p.idx};
    __syncthreads();
    return r;
  }
  bad = false;
  float s = 0.f, t = 0.f;
  for (int i = e0 + threadIdx.x; i < e1; i += NT) {
    float x = to_f32(row[i]);
    if (x == -INFINITY) continue;
    float y = (x - p.m) * kLog2e;
    float e = exp2f(y);
    s += e;
    if (e > 0.f) t = fmaf(y, e, t);
  }
  Part r{p.m, 0.f, 0.f, p.idx};
  r.s = block_sum_f32<NT>(s, shf);
  r.t = block_sum_f32<NT>(t, shf);
  return r;
}

/* Final per-row quantities from a merged Part. */
struct RowOut {
  float conf, entropy, logp;
  int cand;
  uint32_t status;
};

__device__ __forceinline__ bool part_needs_careful(const Part& p) {
  return !(isfinite(p.s) && isfinite(p.t)) || !(p.m > kClamp) || p.m == INFINITY;
}

__device__ __forceinline__ RowOut row_out_from(const Part& p, bool bad) {
  RowOut o;
  o.cand = (p.idx == kIdxNone) ? 0 : p.idx;
  if (bad) {
    o.conf = 0.f; o.entropy = __int_as_float(0x7fc00000); o.logp = __int_as_float(0x7fc00000);
    o.status = 1u;
    return o;
  }
  const float lns = logf(p.s);
  o.conf = 1.0f / p.s;
  o.entropy = fmaxf(lns - (p.t * kLn2) / p.s, 0.f);
  o.logp = -lns;
  o.status = 0u;
  return o;
}

}  // namespace forkd
