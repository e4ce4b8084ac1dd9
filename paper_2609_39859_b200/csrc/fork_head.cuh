/*
 * The confidence pass fused into the LM-head GEMM: logits = hidden x weight^T are formed tile by
 * tile in tensor memory and reduced to (m, s, t2, lowest arg-max) per row right there; they never
 * reach HBM.  (The paper's model "predicts a distribution q_theta^k(.|x_t) for every k in M_t",
 * Section 2; the logits the other kernels read from memory come straight out of this product.)
 *
 * One CTA = one 128-row block of the hidden-state window x one contiguous range of 256-column
 * vocabulary tiles.  Warp roles (192 threads):
 *   warp 0  producer : TMA tensor copies (cp.async.bulk.tensor.2d, no multicast) of a 128 x 64 tile of
 *                      hidden states and a 256 x 64 tile of the weight per k-block into a ring of
 *                      shared-memory stages (128-byte swizzle), full/empty mbarriers;
 *   warp 1  MMA      : one elected thread issues tcgen05.mma (kind::f16, bf16 x bf16 -> fp32,
 *                      M = 128, N = 256, K = 16 per instruction) from shared-memory descriptors into
 *                      one of two 256-column accumulators in tensor memory, frees a stage with
 *                      tcgen05.commit, and hands a finished accumulator to the epilogue the same way;
 *   warps 2-5 epilogue: thread = row (a lane of tensor memory); tcgen05.ld 32 columns at a time,
 *                      online soft-max statistics in registers (exact running maximum with its
 *                      first index, s and t2 rescaled when the maximum rises), while the MMA warp
 *                      already fills the other accumulator.
 * At the end every row's Part goes to head_parts[split][row]; the select kernel of the
 * vocabulary-parallel step merges the splits of a row (they are slices of the vocabulary, exactly
 * like ranks) and applies the unmask rule.
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
constexpr int kHeadStages = 4;
constexpr int kHeadThreads = 192;
constexpr int kHeadABytes = kHeadM * kHeadK * 2;            /* 16 KB */
constexpr int kHeadBBytes = kHeadN * kHeadK * 2;            /* 32 KB */
constexpr int kHeadStageBytes = kHeadABytes + kHeadBBytes;
constexpr uint32_t kHeadSpinLimit = 1u << 24;
constexpr size_t kHeadSmemBytes = (size_t)kHeadStages * kHeadStageBytes + 1024 /* alignment */ + 256 /* barriers */;

struct HeadParams {
  int rows;                  /* B * Ll window rows */
  int V, d;
  int n_tiles;               /* ceil(V / kHeadN) */
  int tiles_per_split;       /* vocabulary tiles per CTA */
  int n_splits;
  int m_blocks;
  float4* parts;             /* [n_splits][m_blocks * kHeadM] */
  WsHeader* hdr;
};

struct HeadBarriers {
  unsigned long long full[kHeadStages], empty[kHeadStages], acc_full[2], acc_empty[2];
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
__host__ __device__ constexpr uint32_t head_instr_desc() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kHeadN >> 3) << 17) | ((uint32_t)(kHeadM >> 4) << 24);
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

__global__ void __launch_bounds__(kHeadThreads, 1)
head_gemm_reduce_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w, const HeadParams p) {
  extern __shared__ unsigned char head_smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(head_smem_raw) + 1023) & ~(uintptr_t)1023);
  HeadBarriers& hb = *reinterpret_cast<HeadBarriers*>(smem + (size_t)kHeadStages * kHeadStageBytes);
  const int warp = (int)threadIdx.x >> 5, lane = (int)threadIdx.x & 31;
  const int mb = (int)blockIdx.x % p.m_blocks, ns = (int)blockIdx.x / p.m_blocks;
  const int tile0 = ns * p.tiles_per_split;
  const int tile1 = min(tile0 + p.tiles_per_split, p.n_tiles);
  const int n_my = tile1 - tile0;                           /* >= 1 by construction of the grid */
  const int kblocks = p.d / kHeadK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kHeadStages; ++s) { head_mbar_init(&hb.full[s], 1); head_mbar_init(&hb.empty[s], 1); }
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
      uint32_t n = 0;                                       /* stages issued */
      bool ok = true;
      for (int t = 0; t < n_my && ok; ++t) {
        const int col0 = (tile0 + t) * kHeadN;
        for (int kb = 0; kb < kblocks; ++kb, ++n) {
          const uint32_t s = n % kHeadStages, ph = (n / kHeadStages) & 1u;
          if (!head_wait(&hb.empty[s], ph ^ 1u, hb, p)) { ok = false; break; }
          unsigned char* a = smem + (size_t)s * kHeadStageBytes;
          head_mbar_expect_tx(&hb.full[s], (uint32_t)kHeadStageBytes);
          head_tma_load_2d(a, &map_h, kb * kHeadK, mb * kHeadM, &hb.full[s]);
          head_tma_load_2d(a + kHeadABytes, &map_w, kb * kHeadK, col0, &hb.full[s]);
        }
      }
      if (!ok) {                                            /* do not leave with copies still landing */
        const uint32_t first = n > (uint32_t)kHeadStages ? n - (uint32_t)kHeadStages : 0u;
        for (uint32_t q = first; q < n; ++q) {
          unsigned long long* bar = &hb.full[q % kHeadStages];
          const uint32_t par = (q / kHeadStages) & 1u;
          for (uint32_t i = 0; i < kHeadSpinLimit && !head_mbar_try(bar, par); ++i) {}
        }
      }
    }
  } else if (warp == 1) {
    /* ---------------- MMA issuer ---------------- */
    if (lane == 0) {
      const uint32_t idesc = head_instr_desc();
      uint32_t n = 0;
      bool ok = true;
      for (int t = 0; t < n_my && ok; ++t) {
        const uint32_t acc = (uint32_t)t & 1u, use = (uint32_t)t >> 1;
        if (!head_wait(&hb.acc_empty[acc], (use & 1u) ^ 1u, hb, p)) { ok = false; break; }   /* the epilogue has drained this accumulator */
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t tmem_d = tmem_base + acc * (uint32_t)kHeadN;
        for (int kb = 0; kb < kblocks; ++kb, ++n) {
          const uint32_t s = n % kHeadStages, ph = (n / kHeadStages) & 1u;
          if (!head_wait(&hb.full[s], ph, hb, p)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = head_smem_u32(smem + (size_t)s * kHeadStageBytes);
          const uint64_t adesc = head_smem_desc(a_addr), bdesc = head_smem_desc(a_addr + kHeadABytes);
#pragma unroll
          for (int kk = 0; kk < kHeadK / 16; ++kk)          /* 16 bf16 = 32 bytes = 2 descriptor units further along the row */
            head_mma(tmem_d, adesc + (uint64_t)(2 * kk), bdesc + (uint64_t)(2 * kk), idesc, (kb > 0 || kk > 0) ? 1u : 0u);
          head_commit(&hb.empty[s]);                        /* the stage is free once these MMAs have read it */
        }
        if (ok) head_commit(&hb.acc_full[acc]);             /* the accumulator is complete once they have all finished */
      }
    }
  } else {
    /* ---------------- epilogue: thread = row ---------------- */
    const int quad = warp & 3;                              /* the 32 tensor-memory lanes this warp may read */
    const int row = mb * kHeadM + quad * 32 + lane;
    float m = -INFINITY, s = 0.f, t2 = 0.f;
    int idx = kIdxNone;
    bool ok = true;
    for (int t = 0; t < n_my && ok; ++t) {
      const uint32_t acc = (uint32_t)t & 1u, use = (uint32_t)t >> 1;
      if (!head_wait(&hb.acc_full[acc], use & 1u, hb, p)) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int col0 = (tile0 + t) * kHeadN;
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * (uint32_t)kHeadN;
#pragma unroll 1
      for (int c = 0; c < kHeadN; c += 32) {
        uint32_t v[32];
        head_tmem_ld32(taddr + (uint32_t)c, v);
        const int cbase = col0 + c;
        if (cbase + 32 > p.V) {                             /* the ragged end of the vocabulary: columns that do not exist */
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (cbase + j >= p.V) v[j] = __float_as_uint(-1.0e30f);
        }
        /* the exact running maximum and its first index (columns ascend: strict > keeps the lowest) */
        const float m_old = m;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float x = __uint_as_float(v[j]);
          if (x > m) { m = x; idx = cbase + j; }
        }
        /* (s, t2) re-expressed against the new maximum, then this chunk's terms */
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
    if (ok && row < p.m_blocks * kHeadM)
      p.parts[(size_t)ns * ((size_t)p.m_blocks * kHeadM) + row] = make_float4(m, s, t2, __int_as_float(idx));
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"(512u) : "memory");
  }
}

}  // namespace forkd
