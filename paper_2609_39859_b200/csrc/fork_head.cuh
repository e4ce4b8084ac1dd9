/*
 * The confidence pass fused into the LM-head GEMM: logits = hidden x weight^T are formed tile by
 * tile in tensor memory and reduced to (m, s, t2, lowest arg-max) per row right there; they never
 * reach HBM.  (The paper's model "predicts a distribution q_theta^k(.|x_t) for every k in M_t",
 * Section 2; the logits the other kernels read from memory come straight out of this product.)
 *
 * One CTA = one 128-row block of the hidden-state window x one contiguous range of vocabulary
 * columns, a whole number of 32-column groups dealt out evenly over the CTAs (so that every SM gets
 * the same share of the weight whatever V is), walked in tiles of 256 columns with a narrower last
 * tile.  Warp roles (192 threads):
 *   warp 0  producer : TMA tensor copies (cp.async.bulk.tensor.2d, every CTA fetching for itself) of a tile of hidden
 *                      states (64 columns x 128 rows; 32 or 64 rows when the window has no more, which
 *                      leaves room for more stages) and a 256 x 64 tile of the weight (the narrow last
 *                      tile in 32-row boxes) per k-block into a ring of shared-memory stages
 *                      (128-byte swizzle), full/empty mbarriers;
 *   warp 1  MMA      : one elected thread issues tcgen05.mma (kind::f16, bf16 x bf16 -> fp32,
 *                      M = 128, N = the tile's width, K = 16 per instruction) from shared-memory descriptors into
 *                      one of two 256-column accumulators in tensor memory, frees a stage with
 *                      tcgen05.commit, and hands a finished accumulator to the epilogue the same way;
 *   warps 2-5 epilogue: thread = row (a lane of tensor memory); tcgen05.ld 32 columns at a time,
 *                      online soft-max statistics in registers (exact running maximum with its
 *                      first index, s and t2 rescaled when the maximum rises), while the MMA warp
 *                      already fills the other accumulator.
 * At the end every row's Part goes to head_parts[split][row]; head_merge_kernel merges the splits of
 * a row (they are slices of the vocabulary, exactly like the ranks of a vocabulary-parallel step) and
 * the select kernel of that step applies the unmask rule.  With candidates drawn at a temperature
 * the epilogue also treats every 32-column chunk as a slice of its own (its tempered weight and its
 * own draw), and a draw kernel picks the chunk once the rows' maxima are known.
 * Every mbarrier wait is bounded; a wait that runs out sets FORK_DEV_TIMEOUT, all roles leave their
 * loops, in-flight copies are waited for, tensor memory is given back.
 */
#pragma once
#include <cuda.h>

#include "fork_params.cuh"

namespace forkd {

constexpr int kHeadM = 128;                 /* rows per CTA (tensor-memory lanes) */
constexpr int kHeadN = 256;                 /* vocabulary columns per tile (accumulator columns) */
constexpr int kHeadK = 64;                  /* bf16 elements per k-block: 128 bytes, one swizzle row */
constexpr int kHeadGroup = 32;              /* columns per group: the unit in which the vocabulary is dealt out, and the rows of a small weight box */
constexpr int kHeadMaxStages = 8;
constexpr int kHeadThreads = 192;
constexpr int kHeadBBytes = kHeadN * kHeadK * 2;            /* 32 KB */
constexpr uint32_t kHeadSpinLimit = 1u << 24;
constexpr size_t kHeadSmemLimit = 227 * 1024;
constexpr size_t kHeadSmemExtra = 1024 /* alignment */ + 256 /* barriers */;

/* Rows of the hidden-state box: the window's rows rounded up to 32, 64 or 128.  The MMA always reads
   128 rows (16 KB) from the stage; with a smaller box the rows behind it are whatever the stage holds
   there (the weight tile), which only reaches accumulator lanes nobody reads. */
__host__ __device__ constexpr int head_a_box_rows(int rows) { return rows <= 32 ? 32 : rows <= 64 ? 64 : kHeadM; }
__host__ __device__ constexpr int head_stage_bytes(int a_box_rows) { return a_box_rows * kHeadK * 2 + kHeadBBytes; }
__host__ __device__ constexpr int head_stages(int a_box_rows) {
  const int n = (int)((kHeadSmemLimit - kHeadSmemExtra) / (size_t)head_stage_bytes(a_box_rows));
  return n < kHeadMaxStages ? n : kHeadMaxStages;
}

struct HeadParams {
  int rows;                  /* B * Ll window rows */
  int V, d;
  int n_groups;              /* ceil(V / 32) column groups */
  int unit;                  /* groups per unit of distribution: 1 with a single row block (the CTAs share nothing and the
                                weight streams from HBM: equal bytes per SM), 8 = whole 256-column tiles otherwise (full-width
                                MMAs matter more there: measured) */
  int u_base, u_rem;         /* units per split: u_base, one more for the first u_rem splits */
  int n_splits;
  int m_blocks;
  int a_box_rows;            /* rows of the hidden-state box: 32, 64 or 128 */
  int stages;                /* ring depth that fits shared memory with that box */
  float4* parts;             /* [n_splits][m_blocks * kHeadM] */
  WsHeader* hdr;
  /* candidates drawn at a temperature (Algorithm 2 line 4): per row and 32-column chunk the log2 of the chunk's
     tempered weight, and the chunk's own draw (with the row's entry uniform, in index order) */
  float c_tau;               /* log2(e) / tau */
  unsigned long long seed; int step;
  int Ll, pos0; const int32_t* row_pos0;   /* row -> (sequence, position), for the row's uniforms */
  float* lw;                 /* [n_groups][m_blocks * kHeadM] */
  float* xt;                 /* [n_groups][m_blocks * kHeadM] the logit of the chunk's drawn entry */
  unsigned char* jt;         /* [n_groups][m_blocks * kHeadM] its index inside the chunk (255: the chunk has no weight) */
  float* lws;                /* [n_splits][m_blocks * kHeadM] log2 of the tempered weight of a CTA's whole column range */
  const float4* merged;      /* head_draw_kernel: [m_blocks * kHeadM] the rows' merged records */
  float4* draw;              /* head_draw_kernel: [m_blocks * kHeadM] out (token, its logit, total, 0) */
};

/* One tensor map of the weight per tile width (box rows = 32, 64, ..., 256): a narrow tile fetched as
   one box of its own width moves as fast as a full one; fetched as several 32-row boxes it does not
   (measured: 1.6 x the time when every tile is fetched that way).  Only the widths a launch uses are
   encoded. */
struct HeadMaps {
  CUtensorMap h;
  CUtensorMap w[kHeadN / kHeadGroup];
};

/* column groups of split ns: its units, clipped to the end of the vocabulary */
__host__ __device__ inline int head_split_groups(const HeadParams& p, int ns) {
  const int g0 = (ns * p.u_base + (ns < p.u_rem ? ns : p.u_rem)) * p.unit;
  const int g1 = g0 + (p.u_base + (ns < p.u_rem ? 1 : 0)) * p.unit;
  return (g1 < p.n_groups ? g1 : p.n_groups) - g0;
}

struct HeadBarriers {
  unsigned long long full[kHeadMaxStages], empty[kHeadMaxStages], acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int abort;
};

__device__ __forceinline__ uint32_t head_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void head_mbar_init(unsigned long long* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(head_smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void head_mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(head_smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void head_mbar_expect_tx(unsigned long long* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(head_smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool head_mbar_try(unsigned long long* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(head_smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
/* bounded wait; gives up (and tells everybody) when the phase never completes or another role gave up */
__device__ __forceinline__ bool head_wait(unsigned long long* bar, uint32_t parity, HeadBarriers& hb, const HeadParams& p) {
  for (uint32_t i = 0; i < kHeadSpinLimit; ++i) {
    if (head_mbar_try(bar, parity)) return true;
    if ((i & 1023u) == 1023u && *reinterpret_cast<volatile int*>(&hb.abort)) return false;
  }
  *reinterpret_cast<volatile int*>(&hb.abort) = 1;
  atomicOr(&p.hdr->dev_status, FORK_DEV_TIMEOUT);
  return false;
}

__device__ __forceinline__ void head_tma_load_2d(void* dst, const CUtensorMap* map, int c0, int c1, unsigned long long* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               :: "r"(head_smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(head_smem_u32(bar)), "r"(c0), "r"(c1)
               : "memory");
}

/* Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16) in the
   128-byte swizzle: 8-row groups 1024 bytes apart (stride byte offset), leading byte offset unused
   (1), descriptor version 1, layout type 2 = SWIZZLE_128B.  Addresses in units of 16 bytes. */
__device__ __forceinline__ uint64_t head_smem_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3fffu);
  d |= (uint64_t)1u << 16;
  d |= (uint64_t)(1024u >> 4) << 32;
  d |= (uint64_t)1u << 46;
  d |= (uint64_t)2u << 61;
  return d;
}
/* Instruction descriptor of tcgen05.mma kind::f16: fp32 accumulator (bits 4-5 = 1), A and B bf16
   (bits 7-9 and 10-12 = 1), both K-major (bits 15, 16 = 0), N / 8 in bits 17-22, M / 16 in bits 24-28. */
__host__ __device__ constexpr uint32_t head_instr_desc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kHeadM >> 4) << 24);
}
__device__ __forceinline__ void head_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               :: "r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void head_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(head_smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void head_tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
               "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
               "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                 "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                 "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                 "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
               : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

template <bool TEMP>
__global__ void __launch_bounds__(kHeadThreads, 1)
head_gemm_reduce_kernel(const __grid_constant__ HeadMaps maps, const HeadParams p) {
  extern __shared__ unsigned char head_smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(head_smem_raw) + 1023) & ~(uintptr_t)1023);
  const int n_stages = p.stages;
  const int a_bytes = p.a_box_rows * kHeadK * 2, stage_bytes = a_bytes + kHeadBBytes;
  HeadBarriers& hb = *reinterpret_cast<HeadBarriers*>(smem + (size_t)n_stages * stage_bytes);
  const int warp = (int)threadIdx.x >> 5, lane = (int)threadIdx.x & 31;
  const int mb = (int)blockIdx.x % p.m_blocks, ns = (int)blockIdx.x / p.m_blocks;
  const int g_cta = head_split_groups(p, ns);                                           /* >= 1 by construction of the grid */
  const int c_begin = (ns * p.u_base + min(ns, p.u_rem)) * p.unit * kHeadGroup;
  /* tiles of at most 256 columns, all of (nearly) the same width so that every stage of the ring
     carries about the same number of bytes: tile t has g_base (+1 for the first g_rem) groups */
  const int n_my = (g_cta + kHeadN / kHeadGroup - 1) / (kHeadN / kHeadGroup);
  const int g_base = g_cta / n_my, g_rem = g_cta % n_my;
  auto tile_col0 = [&](int t) { return c_begin + (t * g_base + min(t, g_rem)) * kHeadGroup; };
  auto tile_width = [&](int t) { return (g_base + (t < g_rem ? 1 : 0)) * kHeadGroup; };
  const int kblocks = p.d / kHeadK;

  /* Nothing here reads what the kernel before it in the stream (the active-set kernel) writes, so
     under a dependent launch this kernel runs beside it and only waits for it at its very end:
     whoever comes after this kernel then finds both complete.  Its own dependents may take their
     places early (they wait at their top). */
  asm volatile("griddepcontrol.launch_dependents;");

  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) { head_mbar_init(&hb.full[s], 1); head_mbar_init(&hb.empty[s], 1); }
    for (int a = 0; a < 2; ++a) { head_mbar_init(&hb.acc_full[a], 1); head_mbar_init(&hb.acc_empty[a], 4); }
    hb.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {                                          /* the MMA warp owns tensor memory: all 512 columns, two accumulators */
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(head_smem_u32(&hb.tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&hb.tmem_base);

  if (warp == 0) {
    /* ---------------- producer ---------------- */
    if (lane == 0) {
      uint32_t n = 0, s = 0, ph = 0;                        /* stages issued; ring slot and its phase */
      bool ok = true;
      for (int t = 0; t < n_my && ok; ++t) {
        const int col0 = tile_col0(t), width = tile_width(t);   /* a multiple of 32 */
        for (int kb = 0; kb < kblocks; ++kb, ++n) {
          if (!head_wait(&hb.empty[s], ph ^ 1u, hb, p)) { ok = false; break; }
          unsigned char* a = smem + (size_t)s * stage_bytes;
          head_mbar_expect_tx(&hb.full[s], (uint32_t)(a_bytes + width * kHeadK * 2));
          head_tma_load_2d(a, &maps.h, kb * kHeadK, mb * kHeadM, &hb.full[s]);
          head_tma_load_2d(a + a_bytes, &maps.w[width / kHeadGroup - 1], kb * kHeadK, col0, &hb.full[s]);
          if (++s == (uint32_t)n_stages) { s = 0; ph ^= 1u; }
        }
      }
      if (!ok) {                                            /* do not leave with copies still landing */
        const uint32_t first = n > (uint32_t)n_stages ? n - (uint32_t)n_stages : 0u;
        for (uint32_t q = first; q < n; ++q) {
          unsigned long long* bar = &hb.full[q % (uint32_t)n_stages];
          const uint32_t par = (q / (uint32_t)n_stages) & 1u;
          for (uint32_t i = 0; i < kHeadSpinLimit && !head_mbar_try(bar, par); ++i) {}
        }
      }
    }
  } else if (warp == 1) {
    /* ---------------- MMA issuer ---------------- */
    if (lane == 0) {
      uint32_t s = 0, ph = 0;
      bool ok = true;
      for (int t = 0; t < n_my && ok; ++t) {
        const uint32_t acc = (uint32_t)t & 1u, use = (uint32_t)t >> 1;
        const uint32_t idesc = head_instr_desc(tile_width(t));
        if (!head_wait(&hb.acc_empty[acc], (use & 1u) ^ 1u, hb, p)) { ok = false; break; }   /* the epilogue has drained this accumulator */
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t tmem_d = tmem_base + acc * (uint32_t)kHeadN;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!head_wait(&hb.full[s], ph, hb, p)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = head_smem_u32(smem + (size_t)s * stage_bytes);
          const uint64_t adesc = head_smem_desc(a_addr), bdesc = head_smem_desc(a_addr + (uint32_t)a_bytes);
#pragma unroll
          for (int kk = 0; kk < kHeadK / 16; ++kk)          /* 16 bf16 = 32 bytes = 2 descriptor units further along the row */
            head_mma(tmem_d, adesc + (uint64_t)(2 * kk), bdesc + (uint64_t)(2 * kk), idesc, (kb > 0 || kk > 0) ? 1u : 0u);
          head_commit(&hb.empty[s]);                        /* the stage is free once these MMAs have read it */
          if (++s == (uint32_t)n_stages) { s = 0; ph ^= 1u; }
        }
        if (ok) head_commit(&hb.acc_full[acc]);             /* the accumulator is complete once they have all finished */
      }
    }
  } else {
    /* ---------------- epilogue: thread = row ---------------- */
    const int quad = warp & 3;                              /* the 32 tensor-memory lanes this warp may read */
    const int row = mb * kHeadM + quad * 32 + lane;
    const bool has_rows = mb * kHeadM + quad * 32 < p.rows;  /* a warp whose 32 rows lie beyond the window only hands the accumulator back */
    float u_tok = 0.5f;                                      /* TEMP: the uniform that draws inside a chunk, the same for every chunk of the row */
    if (TEMP && row < p.rows) {
      const int b = row / p.Ll, k = (p.row_pos0 ? p.row_pos0[b] : p.pos0) + (row - b * p.Ll);
      u_tok = sample_uniform_token(sample_row_key(p.seed, p.step, b, k));
    }
    const size_t rows_pad = (size_t)p.m_blocks * kHeadM;
    float st_run = 0.f;                                      /* TEMP: tempered weight of the columns so far, against the running maximum */
    float m = -INFINITY, s = 0.f, t2 = 0.f;
    int idx = kIdxNone;
    bool ok = true;
    for (int t = 0; t < n_my && ok; ++t) {
      const uint32_t acc = (uint32_t)t & 1u, use = (uint32_t)t >> 1;
      if (!head_wait(&hb.acc_full[acc], use & 1u, hb, p)) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int col0 = tile_col0(t);
      const int width = has_rows ? tile_width(t) : 0;
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * (uint32_t)kHeadN;
#pragma unroll 1
      for (int c = 0; c < width; c += 32) {
        uint32_t v[32];
        head_tmem_ld32(taddr + (uint32_t)c, v);
        const int cbase = col0 + c;
        if (cbase + 32 > p.V) {                             /* the ragged end of the vocabulary: columns that do not exist */
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (cbase + j >= p.V) v[j] = __float_as_uint(-1.0e30f);
        }
        float cmax = -INFINITY, cs = 0.f;                    /* TEMP: the chunk's maximum and its tempered weight against it */
        if (TEMP) {
          /* the chunk as a slice of the vocabulary: its tempered weight (as a log2, against nothing: the
             rows' maxima are not known yet) and its own draw by inversion in index order */
#pragma unroll
          for (int j = 0; j < 32; ++j) cmax = fmaxf(cmax, __uint_as_float(v[j]));
          const float nref = -cmax * p.c_tau;
          float wj[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            wj[j] = ex2_approx(fmaf(__uint_as_float(v[j]), p.c_tau, nref));   /* -inf and the columns that do not exist: 0 */
            cs += wj[j];
          }
          const float target = u_tok * cs;
          float run = 0.f;
          int jt = 255;
          bool found = false;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            if (!found && wj[j] > 0.f) { run += wj[j]; jt = j; found = run >= target; }   /* (the last entry with weight stands if rounding leaves the sum short) */
          }
          float xsel = cmax;
#pragma unroll
          for (int j = 0; j < 32; ++j) xsel = (j == jt) ? __uint_as_float(v[j]) : xsel;
          float lg;
          asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(lg) : "f"(cs));
          const size_t at = (size_t)(cbase >> 5) * rows_pad + (size_t)row;
          if (row < (int)rows_pad) {
            p.lw[at] = (cs > 0.f && cmax > -1.0e29f) ? lg + cmax * p.c_tau : -INFINITY;
            p.xt[at] = xsel;
            p.jt[at] = (unsigned char)jt;
          }
        }
        /* the exact running maximum and its first index (columns ascend: strict > keeps the lowest) */
        const float m_old = m;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float x = __uint_as_float(v[j]);
          if (x > m) { m = x; idx = cbase + j; }
        }
        /* (s, t2) re-expressed against the new maximum, then this chunk's terms */
        if (TEMP) {                                          /* the range's weight so far, re-expressed against the new maximum */
          const float keep = (m_old > -INFINITY) ? ex2_approx((m_old - m) * p.c_tau) : 0.f;
          const float add = (cs > 0.f && cmax > -1.0e29f) ? cs * ex2_approx((cmax - m) * p.c_tau) : 0.f;
          st_run = fmaf(st_run, keep, add);
        }
        const float dd = (m_old > -INFINITY) ? (m_old - m) * kLog2e : 0.f;
        const float w = (m_old > -INFINITY) ? ex2_approx(dd) : 0.f;
        t2 = w * fmaf(dd, s, t2);
        s *= w;
        const float nref = -m * kLog2e;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float y = fmaf(__uint_as_float(v[j]), kLog2e, nref);
          const float e = ex2_approx(y);
          s += e;
          t2 = fmaf(y, e, t2);
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) head_mbar_arrive(&hb.acc_empty[acc]);
    }
    if (ok && row < p.m_blocks * kHeadM) {
      p.parts[(size_t)ns * ((size_t)p.m_blocks * kHeadM) + row] = make_float4(m, s, t2, __int_as_float(idx));
      if (TEMP) {
        float lg;
        asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(lg) : "f"(st_run));
        p.lws[(size_t)ns * rows_pad + row] = (st_run > 0.f && m > -1.0e29f) ? lg + m * p.c_tau : -INFINITY;
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"(512u) : "memory");
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

/* The splits of a row merged into one Part: one warp per row, lanes over the splits (independent
   loads, then one warp reduction), so that the select kernel reads one record per row however many
   CTAs shared the vocabulary.  Ties keep the lowest column index, as everywhere. */
constexpr int kHeadMergeNT = 256;
__global__ void __launch_bounds__(kHeadMergeNT) head_merge_kernel(const HeadParams p, float4* __restrict__ merged) {
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int row = (int)blockIdx.x * (kHeadMergeNT / 32) + (int)(threadIdx.x >> 5), lane = (int)threadIdx.x & 31;
  if (row >= p.rows) return;
  const size_t n = (size_t)p.m_blocks * kHeadM;
  Part acc = part_empty();
  for (int j = lane; j < p.n_splits; j += 32) acc = part_merge(acc, part_from(__ldg(p.parts + (size_t)j * n + row)));
  acc = part_warp_reduce(acc);
  if (lane == 0) merged[row] = make_float4(acc.m, acc.s, acc.t, __int_as_float(acc.idx));
}

/* Drawn candidates, second stage: the chunk of every window row by inversion with the row's slice uniform
   over the chunks' tempered weights (now against the row's maximum), in ascending order; the token is
   that chunk's own draw.  One CTA per 32 rows, lane = row, the chunks dealt to the warps in consecutive
   ranges (reads of 32 consecutive rows are one line). */
constexpr int kHeadDrawNT = 1024;
constexpr int kHeadDrawBatch = 16;          /* loads in flight per thread: the loop is a chain of trips to L2 otherwise */
__global__ void __launch_bounds__(kHeadDrawNT) head_draw_kernel(const HeadParams p) {
  __shared__ float part[kHeadDrawNT / 32][32];
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int lane = (int)threadIdx.x & 31, warp = (int)threadIdx.x >> 5, nw = kHeadDrawNT / 32;
  const int row = (int)blockIdx.x * 32 + lane;
  const size_t rows_pad = (size_t)p.m_blocks * kHeadM;
  const bool valid = row < p.rows;
  const float M = valid ? p.merged[row].x : 0.f;
  const float nM = -M * p.c_tau;
  const int per = (p.n_groups + nw - 1) / nw, c0 = warp * per, c1 = min(c0 + per, p.n_groups);
  float sum = 0.f;
  if (valid)
    for (int c = c0; c < c1; c += kHeadDrawBatch) {
      float l[kHeadDrawBatch];
#pragma unroll
      for (int i = 0; i < kHeadDrawBatch; ++i) l[i] = (c + i < c1) ? __ldg(p.lw + (size_t)(c + i) * rows_pad + row) : -INFINITY;
#pragma unroll
      for (int i = 0; i < kHeadDrawBatch; ++i) sum += ex2_approx(l[i] + nM);   /* in ascending order, as the second look below */
    }
  part[warp][lane] = sum;
  __syncthreads();
  float total = 0.f;
#pragma unroll
  for (int w = 0; w < nw; ++w) total += part[w][lane];
  float u_slice = 0.5f;
  if (valid) {
    const int b = row / p.Ll, k = (p.row_pos0 ? p.row_pos0[b] : p.pos0) + (row - b * p.Ll);
    u_slice = sample_uniform_slice(sample_row_key(p.seed, p.step, b, k));
  }
  const float target = u_slice * total;
  int ws = -1;                                               /* the range that holds the target (the last one with weight if rounding leaves the sum short) */
  float before = 0.f, run = 0.f;
  bool found = false;
#pragma unroll
  for (int w = 0; w < nw; ++w) {
    const float pw = part[w][lane];
    if (!found && pw > 0.f) { before = run; run += pw; ws = w; found = run >= target; }
  }
  if (valid && ws == warp) {
    const float rest = target - before;
    float acc = 0.f;
    int pick = -1;
    bool got = false;
    for (int c = c0; c < c1 && !got; c += kHeadDrawBatch) {
      float l[kHeadDrawBatch];
#pragma unroll
      for (int i = 0; i < kHeadDrawBatch; ++i) l[i] = (c + i < c1) ? __ldg(p.lw + (size_t)(c + i) * rows_pad + row) : -INFINITY;
#pragma unroll
      for (int i = 0; i < kHeadDrawBatch; ++i) {
        const float w = ex2_approx(l[i] + nM);
        if (!got && w > 0.f) { acc += w; pick = c + i; got = acc >= rest; }
      }
    }
    int tok = -1;
    float xs = M;
    if (pick >= 0) {
      const size_t at = (size_t)pick * rows_pad + row;
      const int j = (int)p.jt[at];
      if (j < 32) { tok = pick * 32 + j; xs = p.xt[at]; }
    }
    p.draw[row] = make_float4(__int_as_float(tok), xs, total, 0.f);
  } else if (valid && ws < 0 && warp == 0) {
    p.draw[row] = make_float4(__int_as_float(-1), M, total, 0.f);   /* nothing with weight: the arg-max stands in */
  }
}

/* The same when a CTA's column range is short (few window rows, many CTAs along the vocabulary): first the CTA
   range by its weight (one value per range and row, written by the GEMM's epilogue), then the chunk inside
   that range only -- two short looks instead of two passes over all of a row's chunks. */
constexpr int kHeadDrawMaxRangeChunks = 32;     /* measured: with 54 chunks per range (256 window rows) the two passes over everything are faster */
__global__ void __launch_bounds__(kHeadDrawNT) head_draw_ranges_kernel(const HeadParams p) {
  __shared__ float part[kHeadDrawNT / 32][32];
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int lane = (int)threadIdx.x & 31, warp = (int)threadIdx.x >> 5, nw = kHeadDrawNT / 32;
  const int row = (int)blockIdx.x * 32 + lane;
  const size_t rows_pad = (size_t)p.m_blocks * kHeadM;
  const bool valid = row < p.rows;
  const float M = valid ? p.merged[row].x : 0.f;
  const float nM = -M * p.c_tau;
  constexpr int kPer = 8;                                    /* ranges per warp: 32 warps x 8 covers every grid this kernel is used for */
  const int s0 = warp * kPer;
  float wr[kPer];
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const float l = (valid && s0 + i < p.n_splits) ? __ldg(p.lws + (size_t)(s0 + i) * rows_pad + row) : -INFINITY;
    wr[i] = ex2_approx(l + nM);
    sum += wr[i];
  }
  part[warp][lane] = sum;
  __syncthreads();
  float total = 0.f;
#pragma unroll
  for (int w = 0; w < nw; ++w) total += part[w][lane];
  float u_slice = 0.5f;
  if (valid) {
    const int b = row / p.Ll, k = (p.row_pos0 ? p.row_pos0[b] : p.pos0) + (row - b * p.Ll);
    u_slice = sample_uniform_slice(sample_row_key(p.seed, p.step, b, k));
  }
  const float target = u_slice * total;
  int ws = -1;
  float before = 0.f, run = 0.f;
  bool found = false;
#pragma unroll
  for (int w = 0; w < nw; ++w) {
    const float pw = part[w][lane];
    if (!found && pw > 0.f) { before = run; run += pw; ws = w; found = run >= target; }
  }
  if (valid && ws == warp) {
    /* the range among this warp's eight, then the chunk among the range's */
    int ns = -1;
    float acc = before, acc_before = before;
    bool got = false;
#pragma unroll
    for (int i = 0; i < kPer; ++i)
      if (!got && wr[i] > 0.f) { acc_before = acc; acc += wr[i]; ns = s0 + i; got = acc >= target; }
    const float rest = target - acc_before;
    const int c0 = (ns * p.u_base + min(ns, p.u_rem)) * p.unit, c1 = c0 + head_split_groups(p, ns);
    float a2 = 0.f;
    int pick = -1;
    bool got2 = false;
    for (int c = c0; c < c1 && !got2; c += kHeadDrawBatch) {
      float l[kHeadDrawBatch];
#pragma unroll
      for (int i = 0; i < kHeadDrawBatch; ++i) l[i] = (c + i < c1) ? __ldg(p.lw + (size_t)(c + i) * rows_pad + row) : -INFINITY;
#pragma unroll
      for (int i = 0; i < kHeadDrawBatch; ++i) {
        const float w = ex2_approx(l[i] + nM);
        if (!got2 && w > 0.f) { a2 += w; pick = c + i; got2 = a2 >= rest; }
      }
    }
    int tok = -1;
    float xs = M;
    if (pick >= 0) {
      const size_t at = (size_t)pick * rows_pad + row;
      const int j = (int)p.jt[at];
      if (j < 32) { tok = pick * 32 + j; xs = p.xt[at]; }
    }
    p.draw[row] = make_float4(__int_as_float(tok), xs, total, 0.f);
  } else if (valid && ws < 0 && warp == 0) {
    p.draw[row] = make_float4(__int_as_float(-1), M, total, 0.f);
  }
}

}  // namespace forkd
