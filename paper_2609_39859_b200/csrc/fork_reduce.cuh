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
/* a 128-bit vector of logits that changes nothing: every element is the clamp value (about -1e38) */
__device__ __forceinline__ uint4 neutral_vector(bf16_t) { return make_uint4(0xFE96FE96u, 0xFE96FE96u, 0xFE96FE96u, 0xFE96FE96u); }
__device__ __forceinline__ uint4 neutral_vector(float) { return make_uint4(0xFE960000u, 0xFE960000u, 0xFE960000u, 0xFE960000u); }
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

/* Reduce one Part per lane over the warp; every lane returns the result.  Cheaper than a tree of
   part_merge: one max-reduction, ONE rebase per lane, then plain sums (fixed shape, deterministic). */
__device__ __forceinline__ Part part_warp_reduce(const Part& p) {
  float M = p.m;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  float s, t;
  part_rebase(p, M, s, t);
  int idx = (p.m == M) ? p.idx : kIdxNone;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, o);
    t += __shfl_xor_sync(0xffffffffu, t, o);
    idx = min(idx, __shfl_xor_sync(0xffffffffu, idx, o));
  }
  return Part{M, s, t, idx};
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
  p = part_warp_reduce(p);
  __syncthreads();                         /* previous users of sh are done */
  if (lane == 0) sh[warp] = p;
  __syncthreads();
  if (warp == 0) p = part_warp_reduce((lane < NW) ? sh[lane] : part_empty());
  return p;
}

/* ------------------------------------------------------------------------------------------ */
/* Per-thread streaming accumulator.
 *
 * The exponentials are taken against a per-thread REFERENCE that is not the running maximum: any
 * reference within a few dozen nats of the true maximum gives the same relative precision in fp32,
 * so the reference is set from the thread's first group of vectors and raised again only if the
 * running maximum exceeds it by more than kRaiseNats (overflow guard) -- a branch that is uniform
 * at the start of a segment and practically never taken afterwards, so warps do not diverge.
 * The true maximum is tracked separately with packed NaN-propagating max instructions.  The index
 * of its first occurrence is tracked per 128-bit vector, not per element: for each half of the
 * packed maximum the accumulator remembers the vector in which it last rose (predicated selects,
 * no branch).  Vectors of different threads are disjoint and ordered, so "lowest vector start"
 * orders candidates exactly; the Part therefore carries the START of the winning vector in `idx`
 * and whoever finalises the row reads those few elements once to find the exact position.
 * `part()` re-expresses (s, t) against the thread's true maximum.                                  */
constexpr float kRaiseNats = 32.f;

/* lo/hi halves of a that are greater than b's select `code` into g_lo / g_hi */
__device__ __forceinline__ void track_rise_bf16x2(uint32_t a, uint32_t b, int code, int& g_lo, int& g_hi) {
  asm("{\n\t.reg .pred p, q;\n\tsetp.gt.bf16x2 p|q, %2, %3;\n\tselp.s32 %0, %4, %0, p;\n\tselp.s32 %1, %4, %1, q;\n\t}"
      : "+r"(g_lo), "+r"(g_hi) : "r"(a), "r"(b), "r"(code));
}
__device__ __forceinline__ bool any_gt_bf16x2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("{\n\t.reg .pred p, q;\n\tsetp.gt.bf16x2 p|q, %1, %2;\n\tor.pred p, p, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r) : "r"(a), "r"(b));
  return r != 0;
}

template <typename T, bool WITH_T, bool CLAMP, bool TEMP = false>
struct Acc;

/* Shared arithmetic: four accumulator lanes held as two f32x2 pairs, so that y = x*L - ref*L,
   s += e and t += y*e each take ONE packed instruction (fma.rn.f32x2 / add.rn.f32x2, sm_100)
   per pair of logits; the two exp2 of a pair stay scalar (MUFU has no packed form).
   TEMP (candidates drawn at a temperature): a third sum, the tempered weights 2^{y / tau}, costs
   one packed multiply, two more exp2 and one packed add per pair; `tail_st` collects the tempered
   weights of the fewer-than-a-vector trailing elements, which the draw visits last. */
template <bool WITH_T, bool TEMP>
struct AccCore {
  float ref;                   /* reference, -inf before the first group */
  float2 nrefL2;               /* (-ref*L, -ref*L) */
  float2 s2[2], t2[2];
  float2 st2[2];               /* TEMP: sum 2^{(x-ref) L / tau} */
  float inv_tau, tail_st;      /* TEMP */
  float raise_nats;            /* the reference is raised when the running maximum exceeds it by this much */

  __device__ __forceinline__ void init_core() {
    ref = -INFINITY; nrefL2 = make_float2(INFINITY, INFINITY);
    s2[0] = s2[1] = t2[0] = t2[1] = make_float2(0.f, 0.f);
    st2[0] = st2[1] = make_float2(0.f, 0.f);
    inv_tau = 1.f; tail_st = 0.f; raise_nats = 32.f;
  }
  __device__ __forceinline__ float raise_margin() const { return TEMP ? raise_nats : kRaiseNats; }
  /* temperature of the draw; exponents up to raise_nats * L / tau must stay below the range of exp2 */
  __device__ __forceinline__ void set_temperature(float inv_tau_, float raise_nats_) { inv_tau = inv_tau_; raise_nats = raise_nats_; }
  __device__ __forceinline__ void rescale(float newref) {
    if (ref <= kClamp) {                     /* nothing but -inf so far: weight 0 (NaN is kept) */
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        s2[j].x *= 0.f; s2[j].y *= 0.f;
        if (WITH_T) { t2[j].x *= 0.f; t2[j].y *= 0.f; }
        if (TEMP) { st2[j].x = 0.f; st2[j].y = 0.f; }
      }
      if (TEMP) tail_st = 0.f;
    } else {
      const float d = (ref - newref) * kLog2e;
      const float w = ex2_approx(d);
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        if (WITH_T) { t2[j].x = w * fmaf(d, s2[j].x, t2[j].x); t2[j].y = w * fmaf(d, s2[j].y, t2[j].y); }
        s2[j].x *= w; s2[j].y *= w;
      }
      if (TEMP) {
        const float wt = ex2_approx(d * inv_tau);
#pragma unroll
        for (int j = 0; j < 2; ++j) { st2[j].x *= wt; st2[j].y *= wt; }
        tail_st *= wt;
      }
    }
    ref = newref;
    const float n = -newref * kLog2e;
    nrefL2 = make_float2(n, n);
  }
  /* two logits into pair k */
  __device__ __forceinline__ void add2(int k, float xa, float xb) {
    const float2 y = __ffma2_rn(make_float2(xa, xb), make_float2(kLog2e, kLog2e), nrefL2);
    const float2 e = make_float2(ex2_approx(y.x), ex2_approx(y.y));
    s2[k] = __fadd2_rn(s2[k], e);
    if (WITH_T) t2[k] = __ffma2_rn(y, e, t2[k]);
    if (TEMP) {
      const float2 yt = __fmul2_rn(y, make_float2(inv_tau, inv_tau));
      st2[k] = __fadd2_rn(st2[k], make_float2(ex2_approx(yt.x), ex2_approx(yt.y)));
    }
  }
  /* one trailing element (after all of the thread's vectors) */
  __device__ __forceinline__ void add1(float x) {
    const float y = fmaf(x, kLog2e, nrefL2.x);
    const float e = ex2_approx(y);
    s2[0].x += e;
    if (WITH_T) t2[0].x = fmaf(y, e, t2[0].x);
    if (TEMP) tail_st += ex2_approx(y * inv_tau);
  }
  /* (s, t) re-expressed against the true maximum m >= ref */
  __device__ __forceinline__ void totals(float m, float& ss, float& tt) const {
    ss = (s2[0].x + s2[0].y) + (s2[1].x + s2[1].y);
    tt = WITH_T ? (t2[0].x + t2[0].y) + (t2[1].x + t2[1].y) : 0.f;
    if (ref != m && ref > kClamp) {
      const float d = (ref - m) * kLog2e;
      const float w = ex2_approx(d);
      tt = WITH_T ? w * fmaf(d, ss, tt) : 0.f;
      ss *= w;
    }
  }
  /* TEMP: the tempered weights of the thread's vectors, and of its trailing elements, against m >= ref */
  __device__ __forceinline__ void tempered(float m, float& vec_sum, float& tail_sum) const {
    vec_sum = (st2[0].x + st2[0].y) + (st2[1].x + st2[1].y);
    tail_sum = tail_st;
    if (!(ref > kClamp)) { vec_sum = 0.f; tail_sum = 0.f; return; }
    if (ref != m) {
      const float w = ex2_approx((ref - m) * kLog2e * inv_tau);
      vec_sum *= w; tail_sum *= w;
    }
  }
};

/* ---- bf16: 8 logits per 128-bit vector --------------------------------------------------------
 * CLAMP = false is the normal path: -inf logits are NOT clamped, so a thread that meets one ends
 * with a NaN in t (0 * -inf) and redoes its own vectors with CLAMP = true (see stream_thread). */
template <bool WITH_T, bool CLAMP, bool TEMP>
struct Acc<bf16_t, WITH_T, CLAMP, TEMP> : AccCore<WITH_T, TEMP> {
  static constexpr int VEC = 8;
  uint32_t thr2;               /* packed bf16x2 (ref + kRaiseNats): a running max above it raises the reference */
  uint32_t pm;                 /* running packed maximum of the logits */
  int g_lo, g_hi;              /* element index of the start of the vector where each half last rose */
  float tail_m; int tail_idx;  /* scalar tail elements */

  __device__ __forceinline__ void init() {
    this->init_core();
    thr2 = 0xFF80FF80u; pm = 0xFF80FF80u; g_lo = kIdxNone; g_hi = kIdxNone;
    tail_m = -INFINITY; tail_idx = kIdxNone;
  }
  __device__ __forceinline__ void raise(float newref) {
    this->rescale(newref);
    const uint32_t tb = __float_as_uint(newref + this->raise_margin()) >> 16;
    thr2 = tb | (tb << 16);
  }
  /* N vectors; vector j starts at vocabulary index base + j*stride.  track() touches every loaded
     word (so the loads have landed once it has issued) and updates the maximum; accumulate() does
     the exponentials. */
  template <int N>
  __device__ __forceinline__ void track(uint4 (&v)[N], int base, int stride) {
#pragma unroll
    for (int j = 0; j < N; ++j) {
      if (CLAMP) {
        v[j].x = max_nan_bf16x2(v[j].x, kClampBf16x2); v[j].y = max_nan_bf16x2(v[j].y, kClampBf16x2);
        v[j].z = max_nan_bf16x2(v[j].z, kClampBf16x2); v[j].w = max_nan_bf16x2(v[j].w, kClampBf16x2);
      }
      const uint32_t vm = max_nan_bf16x2(max_nan_bf16x2(v[j].x, v[j].y), max_nan_bf16x2(v[j].z, v[j].w));
      track_rise_bf16x2(vm, pm, base + j * stride, g_lo, g_hi);
      pm = max_nan_bf16x2(pm, vm);
    }
    if (any_gt_bf16x2(pm, thr2)) raise(fmaxf(bf16_lo(pm), bf16_hi(pm)));
  }
  template <int N>
  __device__ __forceinline__ void group(uint4 (&v)[N], int base, int stride) {
    track<N>(v, base, stride);
    accumulate<N>(v);
  }
  template <int N>
  __device__ __forceinline__ void accumulate(const uint4 (&v)[N]) {
#pragma unroll
    for (int j = 0; j < N; ++j) {
      this->add2(0, bf16_lo(v[j].x), bf16_hi(v[j].x));
      this->add2(1, bf16_lo(v[j].y), bf16_hi(v[j].y));
      this->add2(0, bf16_lo(v[j].z), bf16_hi(v[j].z));
      this->add2(1, bf16_lo(v[j].w), bf16_hi(v[j].w));
    }
  }
  /* one trailing element at vocabulary index idx (after all of the thread's vectors) */
  __device__ __forceinline__ void one(float x, int idx) {
    if (CLAMP) x = max_nan_f32(x, kClamp);
    if (x > tail_m) { tail_m = x; tail_idx = idx; }
    if (x > this->ref + this->raise_margin() || this->ref == -INFINITY) raise(fmaxf(x, this->ref));
    this->add1(x);
  }
  __device__ __forceinline__ Part part() const {
    Part r;
    const float ml = bf16_lo(pm), mh = bf16_hi(pm);
    float m = fmaxf(ml, mh);
    int idx = (ml == m && (mh != m || g_lo <= g_hi)) ? g_lo : g_hi;
    if (g_lo == kIdxNone && g_hi == kIdxNone) m = -INFINITY;      /* no vector seen */
    if (tail_m > m) { m = tail_m; idx = tail_idx; }
    r.m = m; r.idx = idx;
    this->totals(m, r.s, r.t);
    if (ml != ml || mh != mh) r.s = ml + mh;                  /* a NaN logit was seen: make the part non-finite */
    return r;
  }
};

/* ---- fp32: 4 logits per 128-bit vector -------------------------------------------------------- */
template <bool WITH_T, bool CLAMP, bool TEMP>
struct Acc<float, WITH_T, CLAMP, TEMP> : AccCore<WITH_T, TEMP> {
  static constexpr int VEC = 4;
  float thr;
  float fm;                    /* running maximum of the logits */
  int g;                       /* element index of the start of the vector where fm last rose */
  float tail_m; int tail_idx;

  __device__ __forceinline__ void init() {
    this->init_core();
    thr = -INFINITY; fm = -INFINITY; g = kIdxNone;
    tail_m = -INFINITY; tail_idx = kIdxNone;
  }
  __device__ __forceinline__ void raise(float newref) {
    this->rescale(newref);
    thr = newref + this->raise_margin();
  }
  template <int N>
  __device__ __forceinline__ void track(uint4 (&v)[N], int base, int stride) {
#pragma unroll
    for (int j = 0; j < N; ++j) {
      if (CLAMP) {
        v[j].x = __float_as_uint(max_nan_f32(__uint_as_float(v[j].x), kClamp));
        v[j].y = __float_as_uint(max_nan_f32(__uint_as_float(v[j].y), kClamp));
        v[j].z = __float_as_uint(max_nan_f32(__uint_as_float(v[j].z), kClamp));
        v[j].w = __float_as_uint(max_nan_f32(__uint_as_float(v[j].w), kClamp));
      }
      const float vm = fmaxf(fmaxf(__uint_as_float(v[j].x), __uint_as_float(v[j].y)),
                             fmaxf(__uint_as_float(v[j].z), __uint_as_float(v[j].w)));
      g = (vm > fm) ? (base + j * stride) : g;
      fm = fmaxf(fm, vm);
    }
    if (fm > thr) raise(fm);
  }
  template <int N>
  __device__ __forceinline__ void accumulate(const uint4 (&v)[N]) {
#pragma unroll
    for (int j = 0; j < N; ++j) {
      this->add2(0, __uint_as_float(v[j].x), __uint_as_float(v[j].y));
      this->add2(1, __uint_as_float(v[j].z), __uint_as_float(v[j].w));
    }
  }
  template <int N>
  __device__ __forceinline__ void group(uint4 (&v)[N], int base, int stride) {
    track<N>(v, base, stride);
    accumulate<N>(v);
  }
  __device__ __forceinline__ void one(float x, int idx) {
    if (CLAMP) x = max_nan_f32(x, kClamp);
    if (x > tail_m) { tail_m = x; tail_idx = idx; }
    if (x > this->ref + this->raise_margin() || this->ref == -INFINITY) raise(fmaxf(x, this->ref));
    this->add1(x);
  }
  __device__ __forceinline__ Part part() const {
    Part r;
    float m = (g == kIdxNone) ? -INFINITY : fm;
    int idx = g;
    if (tail_m > m) { m = tail_m; idx = tail_idx; }
    r.m = m; r.idx = idx;
    this->totals(m, r.s, r.t);
    return r;
  }
};

__device__ __forceinline__ bool part_is_finite(const Part& p) { return isfinite(p.s) && isfinite(p.t); }

/* ------------------------------------------------------------------------------------------ */
/* Stochastic candidates (Algorithm 2 line 4 with tau > 0): x_0 ~ softmax(x / tau), drawn by inversion.
 * The vocabulary (of a buffer: the whole of it, or one rank's slice) is laid out in a fixed order --
 * 128-bit vectors dealt round robin to 256 lanes, lane after lane, the fewer-than-a-vector trailing
 * elements last: the order in which a CTA's 256 streaming threads meet them -- the tempered weights
 * 2^{(x - m) L / tau} are summed along it, and the token is the first at which the running sum reaches
 * U2 times the total.  With the vocabulary in slices the slice is drawn first, with U1.  The two
 * uniforms come from disjoint bit fields of one 64-bit key per (seed, step, sequence, position). */
constexpr int kLanes = 256;                /* lanes of the draw's order = streaming threads of a CTA / consumer threads of a half */
/* floats per part in the lane-sum storage: 256 lane sums, the trailing elements, the total, 2 spare
   (a multiple of 4) */
constexpr int kSlotTail = kLanes, kSlotTotal = kLanes + 1;
constexpr int kSlotStride = kLanes + 4;

__device__ __forceinline__ uint64_t noise_mix64(uint64_t z) {
  z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull; z ^= z >> 27; z *= 0x94D049BB133111EBull; z ^= z >> 31;
  return z;
}
__device__ __forceinline__ uint64_t sample_row_key(uint64_t seed, int step, int b, int k) {
  uint64_t z = noise_mix64(seed + 0x9E3779B97F4A7C15ull * (uint64_t)((uint32_t)step + 1u));
  return noise_mix64(z ^ (((uint64_t)(uint32_t)b << 32) | (uint64_t)(uint32_t)k));
}
/* ((n + 1/2) 2^-23: exact in fp32) */
__device__ __forceinline__ float sample_uniform_token(uint64_t key) { return ((float)(uint32_t)(key >> 41) + 0.5f) * (1.0f / 8388608.0f); }
__device__ __forceinline__ float sample_uniform_slice(uint64_t key) { return ((float)(uint32_t)((key >> 18) & 0x7FFFFFu) + 0.5f) * (1.0f / 8388608.0f); }

/* what a thread hands on about its share of a row segment besides the Part: the tempered weights of
   its vectors and of the trailing elements, against its own maximum (the Part's m) */
struct TauPart { float vec, tail; };

/* The exact position of the row maximum M, given the start `idx` of the vector that holds its
   first occurrence (or the exact position): look at one vector's worth of elements.  All loads are
   issued before any comparison (one 128-bit load when the window is aligned), because this sits
   on the critical path at the end of a step. */
template <typename T>
__device__ __forceinline__ int resolve_index(const T* row, int idx, int V, float M) {
  constexpr int VEC = 16 / (int)sizeof(T);
  if (idx < 0 || idx >= V) return 0;
  float x[VEC];
  if (idx + VEC <= V && (reinterpret_cast<uintptr_t>(row + idx) & 15u) == 0) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(row + idx));
    if (sizeof(T) == 2) {
      x[0] = bf16_lo(v.x); x[1] = bf16_hi(v.x); x[2 % VEC] = bf16_lo(v.y); x[3 % VEC] = bf16_hi(v.y);
      x[4 % VEC] = bf16_lo(v.z); x[5 % VEC] = bf16_hi(v.z); x[6 % VEC] = bf16_lo(v.w); x[7 % VEC] = bf16_hi(v.w);
    } else {
      x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y); x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
  } else {
#pragma unroll
    for (int j = 0; j < VEC; ++j) x[j] = (idx + j < V) ? to_f32(row[idx + j]) : __int_as_float(0x7fc00000);
  }
  int best = idx;
#pragma unroll
  for (int j = VEC - 1; j >= 0; --j)
    if (max_nan_f32(x[j], kClamp) == M) best = idx + j;
  return best;
}

/* One thread's share of elements [e0,e1) of a row, read with 128-bit loads straight from global
   memory: vectors tid, tid+NT, tid+2NT, ... (ascending indices), in groups of UNROLL; the thread
   with `tail` also takes the fewer-than-a-vector trailing elements.  e0 is a multiple of the vector
   width and the row base is 16-byte aligned.  With SAMPLE the tempered weights of the same elements
   come back in `tp` (against the returned Part's maximum). */
template <typename T, bool WITH_T, bool CLAMP, int NT, int UNROLL, bool SAMPLE>
__device__ __forceinline__ Part stream_thread_once(const T* row, int e0, int e1, int tid, bool tail, float inv_tau, float raise_nats,
                                                   TauPart* tp) {
  Acc<T, WITH_T, CLAMP, SAMPLE> a;
  a.init();
  if (SAMPLE) a.set_temperature(inv_tau, raise_nats);
  constexpr int VEC = 16 / (int)sizeof(T);
  const uint4* p = reinterpret_cast<const uint4*>(row + e0);
  const int nvec = (e1 - e0) / VEC;
  int i = tid;
  for (; i + (UNROLL - 1) * NT < nvec; i += UNROLL * NT) {
    uint4 v[UNROLL];
#pragma unroll
    for (int j = 0; j < UNROLL; ++j) v[j] = ld_stream(p + i + j * NT);
    a.template group<UNROLL>(v, e0 + i * VEC, NT * VEC);
  }
  for (; i < nvec; i += NT) {
    uint4 v[1];
    v[0] = ld_stream(p + i);
    a.template group<1>(v, e0 + i * VEC, NT * VEC);
  }
  if (tail) {
    for (int e = e0 + nvec * VEC; e < e1; ++e) a.one(to_f32(row[e]), e);
  }
  const Part pt = a.part();
  if (SAMPLE) a.tempered(pt.m, tp->vec, tp->tail);
  return pt;
}

/* The same share again with -inf clamped, for a thread whose unclamped pass came out non-finite
   (it met a -inf logit, or the row really holds NaN / +inf and will be flagged by the finaliser). */
template <typename T, bool WITH_T, int NT, bool SAMPLE>
__device__ __noinline__ Part stream_thread_clamped(const T* row, int e0, int e1, int tid, bool tail, float inv_tau, float raise_nats,
                                                   TauPart* tp) {
  return stream_thread_once<T, WITH_T, true, NT, 1, SAMPLE>(row, e0, e1, tid, tail, inv_tau, raise_nats, tp);
}

/* `sticky` remembers that this thread has met a -inf before and starts clamped from then on. */
template <typename T, bool WITH_T, int NT, int UNROLL, bool SAMPLE>
__device__ __forceinline__ Part stream_thread(const T* row, int e0, int e1, int tid, bool tail, bool& sticky, float inv_tau,
                                              float raise_nats, TauPart* tp) {
  if (!sticky) {
    const Part pt = stream_thread_once<T, WITH_T, false, NT, UNROLL, SAMPLE>(row, e0, e1, tid, tail, inv_tau, raise_nats, tp);
    if (part_is_finite(pt)) return pt;
    sticky = true;
  }
  return stream_thread_clamped<T, WITH_T, NT, SAMPLE>(row, e0, e1, tid, tail, inv_tau, raise_nats, tp);
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

/* The final quantities use the special-function unit's reciprocal and logarithm (one instruction
   each, errors of about 1e-7 relative / 2e-7 absolute: two orders below the tolerance of the
   outputs) instead of the IEEE division and the library logarithm: this code runs once per row at
   the very end of a step, where every instruction is fetched cold. */
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float ln_approx(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y * kLn2;
}

__device__ __forceinline__ RowOut row_out_from(const Part& p, bool bad) {
  RowOut o;
  o.cand = (p.idx == kIdxNone) ? 0 : p.idx;
  if (bad) {
    o.conf = 0.f; o.entropy = __int_as_float(0x7fc00000); o.logp = __int_as_float(0x7fc00000);
    o.status = 1u;
    return o;
  }
  const float lns = ln_approx(p.s), rs = rcp_approx(p.s);
  o.conf = rs;
  o.entropy = fmaxf(lns - (p.t * kLn2) * rs, 0.f);
  o.logp = -lns;
  o.status = 0u;
  return o;
}

/* The same with a drawn candidate whose logit is xs: its probability under the untempered softmax
   is the confidence (Algorithm 2 line 5 has no temperature), p.idx is the drawn token. */
__device__ __forceinline__ RowOut row_out_sampled(const Part& p, bool bad, float xs) {
  if (bad) return row_out_from(p, true);
  RowOut o;
  o.cand = (p.idx == kIdxNone) ? 0 : p.idx;
  const float lns = ln_approx(p.s), rs = rcp_approx(p.s), d = xs - p.m;
  o.conf = ex2_approx(d * kLog2e) * rs;
  o.entropy = fmaxf(lns - (p.t * kLn2) * rs, 0.f);
  o.logp = d - lns;
  o.status = 0u;
  return o;
}

}  // namespace forkd
