/*
 * Kernels and C ABI of the Fork-dLLM confidence pass (see include/fork_dllm.h for the contract).
 *
 * A step is one or two launches on the caller's stream:
 *   1. active_set_kernel (one CTA): M_t restricted to each sequence's block (Algorithm 2, line 3)
 *      compacted into a row list, per-sequence row offsets, and the number of partial results each
 *      sequence will receive.  The row list is the step's snapshot of the mask: the second kernel
 *      never reads `mask` (which it modifies).
 *   2. reduce_select_kernel (persistent grid): streams every live row once (lines 4-5: arg-max
 *      candidate and its softmax probability, plus entropy), and the CTA that delivers the last
 *      partial result of a sequence applies the unmask rule for it (lines 6-9: threshold set, or
 *      the leftmost masked position when that set is empty) and writes tokens, mask and records.
 *   Small batches on the bulk-copy kernel skip launch 1: every CTA takes the snapshot for itself
 *   (bitmaps of the block windows in shared memory), and no sequence's mask is modified before
 *   every CTA of the launch has done so (FusedCtl in fork_params.cuh).
 * Cross-CTA hand-over uses "last one to arrive" ticket counters (fence + atomic): nothing in
 * here ever waits for another CTA.
 *
 * The same two kernels serve the log-likelihood scoring (Section 3.2), the step with candidates
 * drawn at a temperature (a third instance of the streaming kernels that also tracks the largest
 * Gumbel-perturbed key) and the local phase of the vocabulary-parallel step (the finaliser writes
 * per-position parts instead of applying the rule).  Small kernels of their own: block cursors of the
 * decode loop, the select phase on gathered parts, top-entropy position selection, the ForkGRPO
 * objective (Eq. 2) and the log-softmax backward at the scored rows.
 *
 * Files: fork_reduce.cuh (per-thread accumulators, parts, noise stream), fork_partition.h (work
 * partition), fork_params.cuh (workspace and kernel parameters), fork_setup.cuh (active set, block
 * cursors), fork_finalize.cuh (merging parts, the unmask rule, scoring, vocabulary-parallel phases),
 * fork_stream.cuh (the two streaming kernels), this file (host side, the C ABI, the small kernels).
 */
#include <cuda_runtime.h>

#include <atomic>
#include <mutex>
#include <unordered_map>
#include <cstdint>
#include <cstdio>
#include <cstring>

#include "../../include/fork_dllm.h"
#include "fork_partition.h"
#include "fork_reduce.cuh"
#include "fork_params.cuh"
#include "fork_setup.cuh"
#include "fork_finalize.cuh"
#include "fork_stream.cuh"
#include "fork_head.cuh"

/* =============================================================================================
 *  Host side: argument checks, launch configuration, the C ABI
 * ============================================================================================= */
using namespace forkd;

static std::atomic<long long> g_launches{0};
static std::atomic<int> g_tune[FORK_TUNE_COUNT_];

static size_t ring_smem_bytes(int n_stages) { return kHalves * ring_half_bytes(n_stages); }

/* The bulk-copy kernel runs one CTA per SM made of two independent halves (8 consumer warps and 6
   stages of 16 KB each per half); the work partition counts halves ("virtual CTAs").  Two separate
   CTAs per SM, three with registers capped at 64, or 12 consumer warps per group measured worse. */
constexpr int kRingPerSM = kHalves;                        /* virtual CTAs per SM */
static void ring_config(int* n_stages) {
  int st = g_tune[FORK_TUNE_STAGES].load();
  const int max_st = (int)((220 * 1024 / kHalves - sizeof(RingSmem) - sizeof(SnapSmem) - 1024) / ring_stage_bytes());
  if (st <= 0 || st > max_st) st = max_st;
  if (st > kMaxStages) st = kMaxStages;
  if (st < 2) st = 2;
  *n_stages = st;
}

struct DeviceInfo { int sms = 0; int occ[2][kModeCount] = {}; bool ring_ready = false; };
static DeviceInfo g_dev[64];
static std::once_flag g_dev_once[64];                      /* first call on a device: one thread fills its entry, the others wait */

template <typename T, int MODE>
static int occupancy_of() {
  int n = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, reduce_select_kernel<T, MODE>, kNT, 0) != cudaSuccess) n = 0;
  return n;
}

static void device_info_init(int dev) {
  DeviceInfo& d = g_dev[dev];
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return;
  d.occ[0][0] = occupancy_of<bf16_t, kModeStep>();
  d.occ[0][1] = occupancy_of<bf16_t, kModeLogprob>();
  d.occ[1][0] = occupancy_of<float, kModeStep>();
  d.occ[1][1] = occupancy_of<float, kModeLogprob>();
  d.occ[0][2] = occupancy_of<bf16_t, kModeSample>();
  d.occ[1][2] = occupancy_of<float, kModeSample>();
  d.occ[0][3] = occupancy_of<bf16_t, kModeVp>();
  d.occ[1][3] = occupancy_of<float, kModeVp>();
  d.occ[0][4] = occupancy_of<bf16_t, kModeVpSample>();
  d.occ[1][4] = occupancy_of<float, kModeVpSample>();
  const int max_dyn = 220 * 1024;
  auto allow = [&](const void* fn) { return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, max_dyn) == cudaSuccess; };
  d.ring_ready =
      allow((const void*)reduce_select_ring_kernel<bf16_t, kModeStep>) &&
      allow((const void*)reduce_select_ring_kernel<bf16_t, kModeLogprob>) &&
      allow((const void*)reduce_select_ring_kernel<bf16_t, kModeSample>) &&
      allow((const void*)reduce_select_ring_kernel<float, kModeStep>) &&
      allow((const void*)reduce_select_ring_kernel<float, kModeLogprob>) &&
      allow((const void*)reduce_select_ring_kernel<float, kModeSample>) &&
      allow((const void*)reduce_select_ring_kernel<bf16_t, kModeVp>) &&
      allow((const void*)reduce_select_ring_kernel<bf16_t, kModeVpSample>) &&
      allow((const void*)reduce_select_ring_kernel<float, kModeVp>) &&
      allow((const void*)reduce_select_ring_kernel<float, kModeVpSample>) &&
      allow((const void*)reduce_select_ring_kernel<bf16_t, kModeStep, true>) &&
      allow((const void*)reduce_select_ring_kernel<float, kModeStep, true>);
  if (d.ring_ready) d.sms = sms;                           /* written last: sms != 0 means the entry is complete */
}

static bool device_info(DeviceInfo** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
  std::call_once(g_dev_once[dev], device_info_init, dev);
  if (g_dev[dev].sms == 0) return false;
  *out = &g_dev[dev];
  return true;
}

static int grid_size(const DeviceInfo& d, int dtype, int mode, bool fast) {
  const int variant = g_tune[FORK_TUNE_VARIANT].load();
  if (fast && (variant == 0 || variant == 2)) {
    return d.sms * kRingPerSM;
  }
  int per_sm = g_tune[FORK_TUNE_CTAS_PER_SM].load();
  int occ = d.occ[dtype][mode];
  if (occ <= 0) occ = 1;
  if (per_sm <= 0 || per_sm > occ) per_sm = occ;
  long long G = (long long)d.sms * per_sm;
  if (G > FORK_MAX_GRID) G = FORK_MAX_GRID;
  return (int)G;
}

/* units (of FORK_CHUNK logits) a participating CTA gets at least, on average, in a small step */
constexpr int kDefaultMinUnits = 8;
static int min_units_setting() {
  const int v = g_tune[FORK_TUNE_MIN_UNITS].load();
  return v > 0 ? v : kDefaultMinUnits;
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

/* G counts virtual CTAs: the launch has G / kHalves CTAs of kHalves * kHalfThreads threads */
template <typename T, int MODE>
static cudaError_t launch_ring(const ReduceParams& rp, int G, int n_stages, bool pdl, cudaStream_t st) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(G / kHalves); cfg.blockDim = dim3(kHalfThreads * kHalves); cfg.dynamicSmemBytes = ring_smem_bytes(n_stages);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  if (pdl) {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
  }
  cudaError_t e;
  if (MODE == kModeStep && rp.late_g != 0) e = cudaLaunchKernelEx(&cfg, reduce_select_ring_kernel<T, kModeStep, true>, rp, n_stages);
  else e = cudaLaunchKernelEx(&cfg, reduce_select_ring_kernel<T, MODE>, rp, n_stages);
  if (e == cudaSuccess) g_launches.fetch_add(1);
  return e;
}

template <typename T>
static cudaError_t launch_ring_mode(const ReduceParams& rp, int mode, int G, int n_stages, bool pdl, cudaStream_t st) {
  if (mode == kModeSample) return launch_ring<T, kModeSample>(rp, G, n_stages, pdl, st);
  if (mode == kModeStep) return launch_ring<T, kModeStep>(rp, G, n_stages, pdl, st);
  if (mode == kModeVp) return launch_ring<T, kModeVp>(rp, G, n_stages, pdl, st);
  if (mode == kModeVpSample) return launch_ring<T, kModeVpSample>(rp, G, n_stages, pdl, st);
  return launch_ring<T, kModeLogprob>(rp, G, n_stages, pdl, st);
}

/* variant 2 (bulk-copy ring) needs 16-byte aligned rows; everything else takes variant 1 */
static bool use_ring(const ReduceParams& rp) {
  const int v = g_tune[FORK_TUNE_VARIANT].load();
  return rp.fast && (v == 0 || v == 2);
}

template <typename T>
static cudaError_t launch_direct(const ReduceParams& rp, int mode, int G, bool pdl, cudaStream_t st) {
  if (mode == kModeSample) return launch(reduce_select_kernel<T, kModeSample>, dim3(G), dim3(kNT), st, pdl, rp);
  if (mode == kModeStep) return launch(reduce_select_kernel<T, kModeStep>, dim3(G), dim3(kNT), st, pdl, rp);
  if (mode == kModeVp) return launch(reduce_select_kernel<T, kModeVp>, dim3(G), dim3(kNT), st, pdl, rp);
  if (mode == kModeVpSample) return launch(reduce_select_kernel<T, kModeVpSample>, dim3(G), dim3(kNT), st, pdl, rp);
  return launch(reduce_select_kernel<T, kModeLogprob>, dim3(G), dim3(kNT), st, pdl, rp);
}
static cudaError_t launch_direct_dtype(const ReduceParams& rp, int dtype, int mode, int G, bool pdl, cudaStream_t st) {
  if (dtype == FORK_BF16) return launch_direct<bf16_t>(rp, mode, G, pdl, st);
  return launch_direct<float>(rp, mode, G, pdl, st);
}

static cudaError_t launch_reduce_inner(const ReduceParams& rp, int dtype, int mode, int G, cudaStream_t st) {
  const bool pdl = g_tune[FORK_TUNE_PDL].load() >= 0;
  if (use_ring(rp)) {
    int n_stages;
    ring_config(&n_stages);
    if (dtype == FORK_BF16) return launch_ring_mode<bf16_t>(rp, mode, G, n_stages, pdl, st);
    return launch_ring_mode<float>(rp, mode, G, n_stages, pdl, st);
  }
  return launch_direct_dtype(rp, dtype, mode, G, pdl, st);
}

extern "C" size_t fork_sample_scratch_bytes(int32_t B, int32_t Lt) {
  if (B < 0 || Lt <= 0) return 0;
  const size_t rows = (size_t)(B > 0 ? B : 1) * (size_t)Lt;
  return align_up(rows * sizeof(int32_t), 256) + align_up(rows * sizeof(float4), 256) +
         (rows + FORK_MAX_GRID) * kSlotStride * sizeof(float);
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

extern "C" int64_t fork_mask_handovers(void) {
  unsigned long long n = 0;
  if (cudaMemcpyFromSymbol(&n, g_mask_handovers, sizeof(n)) != cudaSuccess) return -1;
  return (int64_t)n;
}

extern "C" void fork_set_timing_events(void* start, void* stop) {
  t_ev_start = (cudaEvent_t)start;
  t_ev_stop = (cudaEvent_t)stop;
}

static fork_status check_workspace(void* ws, size_t bytes, int32_t B, int32_t Lt) {
  if (!ws || ((uintptr_t)ws % 256) != 0) return FORK_ERR_WORKSPACE;
  if (bytes < fork_workspace_bytes(B, Lt)) return FORK_ERR_WORKSPACE;
  return FORK_OK;
}

struct VpLocal {
  int32_t vocab_offset; float4* part; float4* key;
  int32_t rank = 0, peers = 0; void* const* peer_parts = nullptr; void* const* peer_keys = nullptr;
};

/* ---- one-kernel steps: the control blocks ---------------------------------------------------
 * Part of the library's device image (zero when loaded), one per workspace address seen on a
 * device, handed out on first sight and kept for the life of the process; every launch leaves its
 * block clean, so it does not matter what the caller does with the workspace memory in between,
 * or whether the address later belongs to a new allocation.  A block goes back to the pool only
 * when the caller says the workspace is done with (fork_workspace_release: nothing in here can tell
 * whether a launch or a CUDA graph still refers to it); when all are taken, further workspace
 * addresses run the two-kernel step. */
constexpr int kFusedSlots = 1024;
static __device__ FusedCtl g_fused_ctl[kFusedSlots + 1];   /* the last one belongs to the library's own static scratch */
struct FusedTable {
  FusedCtl* base = nullptr;
  std::unordered_map<const void*, int> slot_of;
  int Gv[kFusedSlots + 1] = {};
  int n_used = 0;                     /* blocks handed out at least once */
  int free_list[kFusedSlots] = {};    /* ... and given back */
  int n_free = 0;
};
static FusedTable g_fused[64];
static std::mutex g_fused_mu;

/* The control block of workspace `ws` for launches of Gv virtual CTAs; NULL if none is left.
   `started` is only meaningful modulo the launch size: when that changes it is put back to zero,
   in stream order. */
static FusedCtl* fused_ctl_for(const void* ws, int Gv, cudaStream_t st, bool* cuda_ok, bool own_scratch) {
  *cuda_ok = true;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { *cuda_ok = false; return nullptr; }
  std::lock_guard<std::mutex> lock(g_fused_mu);
  FusedTable& t = g_fused[dev];
  if (!t.base) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_fused_ctl) != cudaSuccess || !p) { *cuda_ok = false; return nullptr; }
    t.base = (FusedCtl*)p;
  }
  int i;
  auto it = own_scratch ? t.slot_of.end() : t.slot_of.find(ws);
  if (own_scratch) {
    i = kFusedSlots;                  /* no table entry, no host allocation: fork_step_static promises none */
    if (t.Gv[i] == 0) t.Gv[i] = Gv;
  } else if (it != t.slot_of.end()) {
    i = it->second;
  } else {
    if (t.n_free > 0) i = t.free_list[--t.n_free];
    else if (t.n_used < kFusedSlots) { i = t.n_used++; t.Gv[i] = Gv; }
    else return nullptr;
    t.slot_of.emplace(ws, i);
  }
  if (t.Gv[i] != Gv) {
    if (cudaMemsetAsync(&t.base[i].started, 0, sizeof(unsigned long long), st) != cudaSuccess) { *cuda_ok = false; return nullptr; }
    t.Gv[i] = Gv;
  }
  return t.base + i;
}

static fork_status step_impl(const fork_step_args* a, const int32_t* lo, const int32_t* hi, void* ws,
                             cudaStream_t st, const VpLocal* vp = nullptr, bool own_scratch = false,
                             LoopCtl* loop = nullptr) {
  DeviceInfo* dev;
  if (!device_info(&dev)) return FORK_ERR_CUDA;
  WsView w = ws_view(ws, a->B, a->Lt);
  const bool drawn = a->temperature > 0.f;
  const int mode = vp ? (drawn ? kModeVpSample : kModeVp) : (drawn ? kModeSample : kModeStep);
  const bool fast = source_is_vector_aligned(a->logits, a->stride_b, a->stride_l, a->dtype);
  const int G = grid_size(*dev, a->dtype, mode, fast);
  const int C = (a->V + FORK_CHUNK - 1) / FORK_CHUNK;

  /* a small batch on the bulk-copy kernel runs as one kernel: each virtual CTA takes its own
     snapshot of the active set, there is no set-up kernel */
  const int W = (a->Ll + 31) / 32;
  FusedCtl* ctl = nullptr;
  const int v = g_tune[FORK_TUNE_VARIANT].load();
  if (lo && hi && fast && (v == 0 || v == 2) && g_tune[FORK_TUNE_ONE_KERNEL].load() >= 0 &&
      a->B <= kFuseMaxB && W <= kFuseMaxSeqWords && (long long)a->B * W <= kFuseMaxWords) {
    bool cuda_ok;
    ctl = fused_ctl_for(ws, G, st, &cuda_ok, own_scratch);
    if (!cuda_ok) return FORK_ERR_CUDA;
  }

  if (!ctl) {
    SetupParams sp;
    memset(&sp, 0, sizeof(sp));
    sp.flags = a->mask; sp.lo = lo; sp.hi = hi;
    sp.B = a->B; sp.Lt = a->Lt; sp.pos0 = a->pos0; sp.Ll = a->Ll; sp.C = C; sp.G = G; sp.min_units = min_units_setting();
    sp.hdr = w.hdr; sp.seq_off = w.seq_off; sp.expected = w.expected; sp.ticket = w.ticket; sp.rows = w.rows;
    if (!vp) { sp.n_unmasked = a->n_unmasked; sp.is_fallback = a->is_fallback; sp.fallback_pos = a->fallback_pos; }
    sp.loop = loop; sp.step = a->step;
    if (launch(active_set_kernel, dim3(1), dim3(kSetupNT), st, g_tune[FORK_TUNE_PDL].load() >= 0, sp) != cudaSuccess) return FORK_ERR_CUDA;
  }

  ReduceParams rp;
  memset(&rp, 0, sizeof(rp));
  rp.src = RowSource{a->logits, (long long)a->stride_b, (long long)a->stride_l, a->pos0, a->Ll, a->V};
  rp.B = a->B; rp.Lt = a->Lt; rp.C = C;
  rp.fast = fast ? 1 : 0;
  rp.l2_evict_first = g_tune[FORK_TUNE_L2_EVICT_FIRST].load() >= 0 ? 1 : 0;
  rp.min_units = min_units_setting();
  rp.hdr = w.hdr; rp.seq_off = w.seq_off; rp.expected = w.expected; rp.ticket = w.ticket;
  rp.rows = w.rows; rp.final_rec = w.final_rec; rp.parts = w.parts;
  if (drawn) {
    /* lane sums of the tempered weights of every part go to the caller's sample scratch */
    if (!a->sample_scratch || ((uintptr_t)a->sample_scratch % 256) != 0 ||
        a->sample_scratch_bytes < fork_sample_scratch_bytes(a->B, a->Lt)) return FORK_ERR_WORKSPACE;
    {                                                          /* tickets, draws, lane sums: in that order */
      const size_t rows = (size_t)a->B * (size_t)a->Lt;
      char* base = (char*)a->sample_scratch;
      rp.row_ticket = (int32_t*)base;
      rp.row_draw = (float4*)(base + align_up(rows * sizeof(int32_t), 256));
      rp.sslots = (float*)(base + align_up(rows * sizeof(int32_t), 256) + align_up(rows * sizeof(float4), 256));
    }
    rp.noise_c = (float)(1.4426950408889634 / (double)a->temperature);
    rp.inv_tau = 1.0f / a->temperature;
    rp.raise_nats = fminf(32.f, 60.f * a->temperature);      /* tempered exponents stay below 60 * log2(e) < 127 */
  }
  rp.sample_seed = a->sample_seed;
  rp.tokens = a->tokens; rp.mask = a->mask; rp.threshold = a->threshold; rp.step = a->step;
  rp.conf = a->conf; rp.cand = a->cand; rp.entropy = a->entropy; rp.logp = a->logp; rp.row_status = a->row_status;
  rp.commit_step = a->commit_step; rp.commit_fallback = a->commit_fallback; rp.commit_logp = a->commit_logp;
  if (!vp) { rp.n_unmasked = a->n_unmasked; rp.is_fallback = a->is_fallback; rp.fallback_pos = a->fallback_pos; }   /* (the local phase of a vocabulary-parallel step decides nothing) */
  rp.nfe = a->nfe; rp.n_fallback = a->n_fallback;
  rp.fallback_mode = a->fallback_mode; rp.fallback_rand = a->fallback_rand;
  if (vp) {
    rp.vocab_offset = vp->vocab_offset; rp.vp_part = vp->part; rp.vp_key = vp->key;
    rp.vp_rank = vp->rank; rp.vp_peers = vp->peers;
    if (vp->peers > 0) {                                     /* the addresses go through the workspace (copied from a host
                                                                temporary: staged by the runtime before the call returns) */
      VpPeerTable tab;
      memset(&tab, 0, sizeof(tab));
      for (int j = 0; j < vp->peers; ++j) {
        tab.part[j] = (float4*)vp->peer_parts[j];
        tab.key[j] = vp->peer_keys ? (float4*)vp->peer_keys[j] : nullptr;
      }
      if (cudaMemcpyAsync(w.vp_peer_tab, &tab, sizeof(tab), cudaMemcpyHostToDevice, st) != cudaSuccess) return FORK_ERR_CUDA;
      rp.vp_peer_tab = w.vp_peer_tab;
    }
  }
  rp.loop = loop; rp.blk_lo = lo; rp.blk_hi = hi;
  if (ctl) {
    rp.ctl = ctl; rp.ticket = ctl->ticket; rp.commit_bits = w.commit_bits;
    rp.W = W; rp.Gv = G; rp.late_g = g_tune[FORK_TUNE_LATE_CTA].load();
  }
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
  if (a->fallback_mode < FORK_FALLBACK_LEFTMOST || a->fallback_mode > FORK_FALLBACK_RANDOM) return FORK_ERR_INVALID_ARG;
  if (a->fallback_mode == FORK_FALLBACK_RANDOM && !a->fallback_rand) return FORK_ERR_INVALID_ARG;
  if (!(a->temperature >= 0.f) || a->temperature > 3.0e38f) return FORK_ERR_INVALID_ARG;
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
  const bool fast = source_is_vector_aligned(a->logits, a->stride_b, a->stride_l, a->dtype);
  const int G = grid_size(*dev, a->dtype, mode, fast);
  const int C = (a->V + FORK_CHUNK - 1) / FORK_CHUNK;
  if (cudaMemsetAsync(a->logp, 0, sizeof(float) * (size_t)a->B * a->Lt, st) != cudaSuccess) return FORK_ERR_CUDA;

  SetupParams sp;
  memset(&sp, 0, sizeof(sp));
  sp.flags = a->select; sp.lo = nullptr; sp.hi = nullptr;
  sp.B = a->B; sp.Lt = a->Lt; sp.pos0 = a->pos0; sp.Ll = a->Ll; sp.C = C; sp.G = G; sp.min_units = min_units_setting();
  sp.hdr = w.hdr; sp.seq_off = w.seq_off; sp.expected = w.expected; sp.ticket = w.ticket; sp.rows = w.rows;
  sp.seq_sum = a->seq_sum; sp.seq_cnt = a->seq_cnt;
  if (launch(active_set_kernel, dim3(1), dim3(kSetupNT), st, g_tune[FORK_TUNE_PDL].load() >= 0, sp) != cudaSuccess) return FORK_ERR_CUDA;

  ReduceParams rp;
  memset(&rp, 0, sizeof(rp));
  rp.src = RowSource{a->logits, (long long)a->stride_b, (long long)a->stride_l, a->pos0, a->Ll, a->V};
  rp.B = a->B; rp.Lt = a->Lt; rp.C = C;
  rp.fast = fast ? 1 : 0;
  rp.l2_evict_first = g_tune[FORK_TUNE_L2_EVICT_FIRST].load() >= 0 ? 1 : 0;
  rp.min_units = min_units_setting();
  rp.hdr = w.hdr; rp.seq_off = w.seq_off; rp.expected = w.expected; rp.ticket = w.ticket;
  rp.rows = w.rows; rp.final_rec = w.final_rec; rp.parts = w.parts;
  rp.lp_tokens = a->tokens; rp.lp_out = a->logp; rp.seq_sum = a->seq_sum; rp.seq_cnt = a->seq_cnt;
  rp.lse_out = a->lse;
  rp.row_status = a->row_status;
  if (launch_reduce(rp, a->dtype, mode, G, st) != cudaSuccess) return FORK_ERR_CUDA;
  return FORK_OK;
}

/* ---- the decode loop ------------------------------------------------------------------------
 * The host's part is to call the provider and enqueue the step; whether anything is still masked
 * it learns from eight bytes of pinned host memory that the last finaliser of every step writes
 * (ticket, remaining), not from a stream synchronisation.  A call takes a ring of kLoopFlags such
 * words from a small pool that is allocated once per process. */
constexpr int kLoopCalls = 32;                              /* loops that may run at the same time in one process */
static unsigned long long* g_loop_flags = nullptr;          /* pinned, mapped: [kLoopCalls][kLoopFlags] */
static bool g_loop_used[kLoopCalls];
static std::mutex g_loop_mu;
static std::atomic<uint32_t> g_loop_ticket{1};

static int loop_ring_acquire() {
  std::lock_guard<std::mutex> lock(g_loop_mu);
  if (!g_loop_flags) {
    void* p = nullptr;
    if (cudaHostAlloc(&p, sizeof(unsigned long long) * kLoopCalls * kLoopFlags, cudaHostAllocPortable | cudaHostAllocMapped) != cudaSuccess)
      return -1;
    memset(p, 0, sizeof(unsigned long long) * kLoopCalls * kLoopFlags);
    g_loop_flags = (unsigned long long*)p;
  }
  for (int i = 0; i < kLoopCalls; ++i)
    if (!g_loop_used[i]) { g_loop_used[i] = true; return i; }
  return -1;
}
static void loop_ring_release(int i) {
  std::lock_guard<std::mutex> lock(g_loop_mu);
  g_loop_used[i] = false;
}

/* Waits until the word carries `ticket`; returns the count that came with it, or -1 if the stream
   ran dry (or failed) without the word arriving.  The wait is a host-side poll; every few thousand
   polls it asks the stream whether it still has work, so a failed launch cannot hold it for ever. */
static int loop_wait_flag(const volatile unsigned long long* word, uint32_t ticket, cudaStream_t st) {
  for (unsigned long long it = 0;; ++it) {
    const unsigned long long v = *word;
    if ((uint32_t)v == ticket) return (int)(uint32_t)(v >> 32);
    if ((it & 4095ull) == 4095ull) {
      const cudaError_t q = cudaStreamQuery(st);
      if (q == cudaSuccess) {                               /* everything enqueued has run: the word is there now or never */
        const unsigned long long v2 = *word;
        return ((uint32_t)v2 == ticket) ? (int)(uint32_t)(v2 >> 32) : -1;
      }
      if (q != cudaErrorNotReady) return -1;
    }
  }
}

/* The loop itself; `buffer` is what the provider fills (logits, or hidden states), `enqueue` puts one
   step on the stream for the cursors it is given. */
template <typename StepFn>
static fork_status decode_loop_impl(const fork_step_args* proto, void* buffer, int32_t block_len, int32_t gen_lo, int32_t gen_hi,
                                    fork_logits_fn provider, void* ctx, int32_t max_steps, int32_t* steps_taken,
                                    void* ws, void* stream, StepFn enqueue) {
  cudaStream_t st = (cudaStream_t)stream;
  WsView w = ws_view(ws, proto->B, proto->Lt);
  int ahead = g_tune[FORK_TUNE_LOOP_AHEAD].load();
  if (ahead < 0) ahead = 0;
  if (ahead > kLoopFlags - 2) ahead = kLoopFlags - 2;

  const int ring = loop_ring_acquire();
  if (ring < 0) return FORK_ERR_CUDA;
  unsigned long long* flags = g_loop_flags + (size_t)ring * kLoopFlags;
  void* flags_dev = nullptr;
  if (cudaHostGetDevicePointer(&flags_dev, flags, 0) != cudaSuccess) { loop_ring_release(ring); return FORK_ERR_CUDA; }
  const uint32_t ticket0 = g_loop_ticket.fetch_add((uint32_t)max_steps + 2u) + 1u;

  LoopCtl lc;
  memset(&lc, 0, sizeof(lc));
  lc.gen_lo = gen_lo; lc.gen_hi = gen_hi; lc.block_len = block_len; lc.step0 = proto->step;
  lc.ticket0 = ticket0; lc.flags = (unsigned long long*)flags_dev;
  for (int i = 0; i < 2; ++i) { lc.lo[i] = w.loop_lo[i]; lc.hi[i] = w.loop_hi[i]; }
  fork_status rc = FORK_OK;
  int32_t issued = 0, confirmed = 0, done_at = -1;         /* steps enqueued; steps whose report has been read; the step after which nothing was masked */
  int remaining = -1;
  /* (the struct is copied from this host temporary: staged by the runtime before the call returns) */
  CursorParams cp{proto->mask, proto->B, proto->Lt, gen_lo, gen_hi, block_len, w.loop_lo[0], w.loop_hi[0], w.loop, 1};
  if (cudaMemcpyAsync(w.loop, &lc, sizeof(lc), cudaMemcpyHostToDevice, st) != cudaSuccess ||
      launch(block_cursor_kernel, dim3(1), dim3(kSetupNT), st, false, cp) != cudaSuccess) rc = FORK_ERR_CUDA;
  if (rc == FORK_OK) {
    remaining = loop_wait_flag(flags + (kLoopFlags - 1), ticket0 - 1u, st);
    if (remaining < 0) rc = FORK_ERR_CUDA;
    else if (remaining == 0) done_at = 0;
  }
  while (rc == FORK_OK && done_at < 0) {
    /* read the reports that are due: all that have arrived, and those without which the loop would
       run more than `ahead` steps past what it knows */
    while (confirmed < issued && done_at < 0) {
      const volatile unsigned long long* word = flags + (confirmed % kLoopFlags);
      const uint32_t ticket = ticket0 + (uint32_t)confirmed;
      const bool must = issued - confirmed > ahead || issued >= max_steps;
      if (!must && (uint32_t)*word != ticket) break;
      remaining = loop_wait_flag(word, ticket, st);
      if (remaining < 0) { rc = FORK_ERR_CUDA; break; }
      ++confirmed;
      if (remaining == 0) done_at = confirmed;
    }
    if (rc != FORK_OK || done_at >= 0) break;
    if (issued >= max_steps) { rc = FORK_ERR_MAX_STEPS; break; }      /* every report is in: something is still masked */
    const int32_t* lo = w.loop_lo[issued & 1];
    const int32_t* hi = w.loop_hi[issued & 1];
    if (provider(ctx, proto->step + issued, proto->tokens, proto->mask, lo, hi, buffer, stream) != 0) {
      rc = FORK_ERR_PROVIDER;
      break;
    }
    fork_step_args a = *proto;
    a.step = proto->step + issued;
    rc = enqueue(a, lo, hi, w.loop);
    if (rc != FORK_OK) break;
    ++issued;
  }
  /* steps still in flight (enqueued ahead of the reports) find nothing to do once the batch is
     complete; their reports are taken in before the ring of words goes back to the pool */
  while (confirmed < issued) {
    const int r = loop_wait_flag(flags + (confirmed % kLoopFlags), ticket0 + (uint32_t)confirmed, st);
    if (r < 0) { if (rc == FORK_OK) rc = FORK_ERR_CUDA; break; }
    ++confirmed;
    if (r == 0 && done_at < 0) done_at = confirmed;
  }
  if (rc == FORK_ERR_PROVIDER && done_at >= 0) rc = FORK_OK;      /* the failed call was one made ahead, for a step that had nothing left to do */
  loop_ring_release(ring);
  if (steps_taken) *steps_taken = done_at >= 0 ? done_at : issued;
  return rc;
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
  return decode_loop_impl(proto, const_cast<void*>(proto->logits), block_len, gen_lo, gen_hi, provider, ctx, max_steps, steps_taken,
                          ws, stream, [&](const fork_step_args& a, const int32_t* lo, const int32_t* hi, LoopCtl* loop) {
                            return step_impl(&a, lo, hi, ws, st, nullptr, false, loop);
                          });
}

extern "C" fork_status fork_workspace_release(const void* ws) {
  if (!ws) return FORK_ERR_INVALID_ARG;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FORK_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_fused_mu);
  FusedTable& t = g_fused[dev];
  auto it = t.slot_of.find(ws);
  if (it != t.slot_of.end()) {
    t.free_list[t.n_free++] = it->second;
    t.slot_of.erase(it);
  }
  return FORK_OK;
}

static fork_status static_scratch(void** out);

extern "C" fork_status fork_device_status(const void* ws, uint32_t* host_out, void* stream) {
  if (!host_out) return FORK_ERR_INVALID_ARG;
  const bool own = ws == nullptr;              /* NULL: the scratch inside the library that fork_step_static runs on */
  if (own) {
    void* p = nullptr;
    const fork_status s = static_scratch(&p);
    if (s != FORK_OK) return s;
    ws = p;
  }
  const WsHeader* h = (const WsHeader*)ws;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(host_out, &h->dev_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) return FORK_ERR_CUDA;
  if (*host_out & FORK_DEV_TIMEOUT) {
    /* a launch that gave up may have left the workspace's control block with tickets or its
       snapshot count in the middle of a step: put it back to its initial state */
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FORK_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_fused_mu);
    FusedTable& t = g_fused[dev];
    int slot = -1;
    if (own) slot = kFusedSlots;
    else { auto it = t.slot_of.find(ws); if (it != t.slot_of.end()) slot = it->second; }
    if (slot >= 0 && t.base) {
      if (cudaMemsetAsync(t.base + slot, 0, sizeof(FusedCtl), st) != cudaSuccess ||
          cudaStreamSynchronize(st) != cudaSuccess) return FORK_ERR_CUDA;
    }
  }
  return FORK_OK;
}

/* ---- fork_step on the library's own scratch ------------------------------------------------- */
/* The scratch that fork_step normally receives from its caller, held instead in a fixed array that
   is part of this library's device image: every GPU that loads the library carries these bytes
   until the process exits.  In host code the NAME of a __device__ array is only a host-side
   stand-in, not a device address, so the address the kernels get is looked up once per device with
   cudaGetSymbolAddress and cached. */
static __device__ __align__(256) unsigned char g_static_scratch[FORK_STATIC_SCRATCH_BYTES];
static void* g_static_scratch_ptr[64];
static std::once_flag g_static_scratch_once[64];

static void static_scratch_init(int dev) {
  void* ptr = nullptr;                         /* set-up, once per device, with that device current */
  if (cudaGetSymbolAddress(&ptr, g_static_scratch) == cudaSuccess) g_static_scratch_ptr[dev] = ptr;
}

static fork_status static_scratch(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FORK_ERR_CUDA;
  std::call_once(g_static_scratch_once[dev], static_scratch_init, dev);
  if (g_static_scratch_ptr[dev] == nullptr) return FORK_ERR_CUDA;
  *out = g_static_scratch_ptr[dev];
  return FORK_OK;
}

extern "C" fork_status fork_step_static(const fork_step_args* a, void* stream) {
  fork_status s = check_step_args(a, true);
  if (s != FORK_OK) return s;
  if (fork_workspace_bytes(a->B, a->Lt) > (size_t)FORK_STATIC_SCRATCH_BYTES) return FORK_ERR_WORKSPACE;
  if (a->B == 0) return FORK_OK;
  void* ws = nullptr;
  s = static_scratch(&ws);
  if (s != FORK_OK) return s;
  /* nothing in the scratch has to survive from call to call: what a step reads there it has
     written itself; the one-kernel step's control block is a reserved one of the library's */
  return step_impl(a, a->blk_lo, a->blk_hi, ws, (cudaStream_t)stream, nullptr, true);
}

/* ---- top-entropy position selection (JustGRPO-Fast; Section 3.2, last paragraph) ------------ */
/* One CTA per rollout.  Keys sit in shared memory: the entropy of an eligible position (-inf when it
   is NaN, so that it ranks last), NaN for a position that is not eligible.  Position i is selected
   when fewer than `want` eligible positions rank before it (higher entropy, or equal entropy and a
   lower position). */
constexpr int kSelectNT = 256;
constexpr int kSelectMaxLt = 32768;

__global__ void __launch_bounds__(kSelectNT) select_top_entropy_kernel(const float* __restrict__ entropy,
                                                                      const uint8_t* __restrict__ eligible, int Lt,
                                                                      float ratio, uint8_t* __restrict__ select,
                                                                      int32_t* __restrict__ n_selected) {
  extern __shared__ float sel_key[];
  __shared__ int sh_n;
  const int b = blockIdx.x, tid = threadIdx.x;
  if (tid == 0) sh_n = 0;
  __syncthreads();
  int mine = 0;
  for (int k = tid; k < Lt; k += kSelectNT) {
    const size_t at = (size_t)b * Lt + k;
    float key = __int_as_float(0x7fc00000);
    if (eligible[at]) { const float h = entropy[at]; key = (h != h) ? -INFINITY : h; ++mine; }
    sel_key[k] = key;
  }
  if (mine) atomicAdd(&sh_n, mine);
  __syncthreads();
  const int n = sh_n;
  int want = (int)floor((double)ratio * (double)n);
  if (want < 1 && n > 0 && ratio > 0.f) want = 1;
  for (int i = tid; i < Lt; i += kSelectNT) {
    const float ki = sel_key[i];
    uint8_t out = 0;
    if (ki == ki && want > 0) {
      int before = 0;
      for (int j = 0; j < Lt; ++j) {
        const float kj = sel_key[j];                          /* a comparison with NaN is false: not eligible */
        before += (kj > ki || (kj == ki && j < i)) ? 1 : 0;
      }
      out = before < want ? 1 : 0;
    }
    select[(size_t)b * Lt + i] = out;
  }
  if (tid == 0 && n_selected) n_selected[b] = want;
}

extern "C" fork_status fork_select_top_entropy(const float* entropy, const uint8_t* eligible, int32_t B, int32_t Lt,
                                               float ratio, uint8_t* select, int32_t* n_selected, void* stream) {
  if (!entropy || !eligible || !select || B < 0 || Lt <= 0 || Lt > kSelectMaxLt) return FORK_ERR_INVALID_ARG;
  if (!(ratio >= 0.f) || ratio > 1.f) return FORK_ERR_INVALID_ARG;
  if (B == 0) return FORK_OK;
  const size_t smem = (size_t)Lt * sizeof(float);
  static std::atomic<int> raised[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return FORK_ERR_CUDA;
  if (smem > 48 * 1024 && (dev >= 64 || !raised[dev].load())) {
    if (cudaFuncSetAttribute(select_top_entropy_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kSelectMaxLt * (int)sizeof(float)) != cudaSuccess) return FORK_ERR_CUDA;
    if (dev < 64) raised[dev].store(1);
  }
  select_top_entropy_kernel<<<B, kSelectNT, smem, (cudaStream_t)stream>>>(entropy, eligible, Lt, ratio, select, n_selected);
  if (cudaGetLastError() != cudaSuccess) return FORK_ERR_CUDA;
  g_launches.fetch_add(1);
  return FORK_OK;
}

/* ---- ForkGRPO objective (Eq. 2) ------------------------------------------------------------- */
/* One CTA per prompt group.  Group statistics in fp64 (a handful of values), the per-position terms
   in fp32; one warp per rollout walks its positions twice (count of fallback steps, then the
   terms).  A second one-CTA kernel sums the per-rollout objectives in a fixed order. */
constexpr int kGrpoNT = 256;

/* mean and population standard deviation of the rewards of prompt group p (one thread, fp64, in index order) */
__device__ __forceinline__ void grpo_group_stats(const float* reward, int p, int G, double& mean, double& sd) {
  double m = 0.0, var = 0.0;
  for (int j = 0; j < G; ++j) m += (double)reward[p * G + j];
  m /= G;
  for (int j = 0; j < G; ++j) { const double d = (double)reward[p * G + j] - m; var += d * d; }
  mean = m; sd = sqrt(var / G);
}
/* number of fallback steps of rollout i (selected positions of its row of `select`), by one warp */
__device__ __forceinline__ int grpo_count_selected(const uint8_t* select, int i, int Lt) {
  const int lane = threadIdx.x & 31;
  int nf = 0;
  for (int k0 = 0; k0 < Lt; k0 += 32) {
    const int k = k0 + lane;
    nf += __popc(__ballot_sync(0xffffffffu, k < Lt && select[(size_t)i * Lt + k] != 0));
  }
  return nf;
}
/* One token of Eq. 2: the ratio, the clipped minimum, and dJ/dlogp_new (rho A / (B |F_i|) where the
   unclipped term is the minimum, else 0; nothing for a skipped group). */
__device__ __forceinline__ void grpo_token(float logp_new, float logp_old, float A, bool skip, float scale, float eps_lo,
                                           float eps_hi, float& rho, float& term, float& d) {
  rho = expf(logp_new - logp_old);
  const float clipped = fminf(fmaxf(rho, 1.f - eps_lo), 1.f + eps_hi);
  const float u = rho * A, c = clipped * A;
  term = (u <= c) ? u : c;                                   /* the clipped minimum of Eq. 2 */
  d = (!skip && u <= c) ? rho * A * scale : 0.f;             /* the unclipped term is active */
}

__global__ void __launch_bounds__(kGrpoNT) grpo_group_kernel(fork_grpo_args a) {
  __shared__ double sh_mean, sh_sd;
  const int p = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = kGrpoNT / 32;
  const int G = a.group, B = a.B, Lt = a.Lt;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (tid == 0) {
    double mean, sd;
    grpo_group_stats(a.reward, p, G, mean, sd);
    sh_mean = mean; sh_sd = sd;
    if (a.skipped) a.skipped[p] = (uint8_t)(!(sh_sd > 0.0));
  }
  __syncthreads();
  const bool skip = !(sh_sd > 0.0);
  for (int j = warp; j < G; j += nwarp) {
    const int i = p * G + j;
    const float A = skip ? 0.f : (float)(((double)a.reward[i] - sh_mean) / sh_sd);
    const int nf = grpo_count_selected(a.select, i, Lt);
    const float scale = nf > 0 ? 1.f / ((float)B * (float)nf) : 0.f;
    float acc = 0.f;
    for (int k = lane; k < Lt; k += 32) {
      const size_t at = (size_t)i * Lt + k;
      float rho = 0.f, d = 0.f;
      if (a.select[at]) {
        float term;
        grpo_token(a.logp_new[at], a.logp_old[at], A, skip, scale, a.eps_lo, a.eps_hi, rho, term, d);
        acc += term;
      }
      if (a.ratio) a.ratio[at] = rho;
      if (a.dlogp) a.dlogp[at] = d;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) {
      if (a.adv) a.adv[i] = A;
      a.seq_obj[i] = nf > 0 ? acc / (float)nf : 0.f;
    }
  }
}

__global__ void __launch_bounds__(kGrpoNT) grpo_sum_kernel(const float* seq_obj, int B, float* objective) {
  __shared__ double sh[kGrpoNT];
  double acc = 0.0;
  for (int i = threadIdx.x; i < B; i += kGrpoNT) acc += (double)seq_obj[i];
  sh[threadIdx.x] = acc;
  __syncthreads();
  for (int o = kGrpoNT / 2; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *objective = B > 0 ? (float)(sh[0] / B) : 0.f;
}

extern "C" fork_status fork_grpo_loss(const fork_grpo_args* a, void* stream) {
  if (!a || a->B < 0 || a->Lt <= 0 || a->group <= 0 || a->B % a->group != 0) return FORK_ERR_INVALID_ARG;
  if (!a->logp_new || !a->logp_old || !a->select || !a->reward || !a->seq_obj) return FORK_ERR_INVALID_ARG;
  if (!(a->eps_lo >= 0.f) || !(a->eps_hi >= 0.f)) return FORK_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (a->B > 0) {
    grpo_group_kernel<<<a->B / a->group, kGrpoNT, 0, st>>>(*a);
    if (cudaGetLastError() != cudaSuccess) return FORK_ERR_CUDA;
    g_launches.fetch_add(1);
  }
  if (a->objective) {
    grpo_sum_kernel<<<1, kGrpoNT, 0, st>>>(a->seq_obj, a->B, a->objective);
    if (cudaGetLastError() != cudaSuccess) return FORK_ERR_CUDA;
    g_launches.fetch_add(1);
  }
  return FORK_OK;
}

/* ---- derivative of the scored log-likelihoods with respect to the logits -------------------- */
/* d/dx_v [w (x_tok - lse)] = w (1[v = tok] - p_v), p_v = exp(x_v - lse): one read of the row, one
   write of the same size.  Work is cut into units of kBwdNT * kBwdVecs * kBwdIters 128-bit vectors of one row;
   the rows are those of the row list the active-set kernel built from `select`. */
constexpr int kBwdNT = 256;
constexpr int kBwdVecs = 2;
constexpr int kBwdIters = 8;          /* a unit = kBwdIters inner iterations of one row (64 KB): per-row values are fetched once per unit */

struct BwdParams {
  RowSource src; void* grad; long long gstride_b, gstride_l;
  const WsHeader* hdr; const int2* rows;
  const int32_t* tokens; const float* lse; const float* dlogp; int Lt, vector_ok;
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ void store_grad(bf16_t* p, float g) {
  p->bits = (uint16_t)(pack_bf16x2(g, 0.f) & 0xffffu);
}
__device__ __forceinline__ void store_grad(float* p, float g) { *p = g; }

template <typename T>
__global__ void __launch_bounds__(kBwdNT) logprob_backward_kernel(BwdParams p) {
  constexpr int VEC = 16 / (int)sizeof(T);
  constexpr int kStepElems = kBwdNT * kBwdVecs * VEC;          /* elements per inner iteration */
  constexpr int kUnitElems = kStepElems * kBwdIters;           /* elements of one row per unit */
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int R = p.hdr->R;
  const int V = p.src.V;
  const int units_per_row = (V + kUnitElems - 1) / kUnitElems;
  const long long U = (long long)R * units_per_row;
  for (long long u = blockIdx.x; u < U; u += gridDim.x) {
    const int r = (int)(u / units_per_row);
    const int u0 = (int)(u - (long long)r * units_per_row) * kUnitElems;
    const int u1 = min(u0 + kUnitElems, V);
    const int2 bk = p.rows[r];
    const size_t at = (size_t)bk.x * p.Lt + bk.y;
    const int tok = p.tokens[at];
    if (tok < 0 || tok >= V) continue;                       /* scored as FORK_ROW_BAD_TOKEN: no gradient */
    const float w = p.dlogp[at];
    const float nl = -p.lse[at] * kLog2e;
    const T* row = row_ptr<T>(p.src, bk.x, bk.y);
    T* grow = reinterpret_cast<T*>(p.grad) + ((long long)bk.x * p.gstride_b + (long long)(bk.y - p.src.pos0) * p.gstride_l);
    if (!p.vector_ok) {
      for (int q = u0 + (int)threadIdx.x; q < u1; q += kBwdNT) {
        const float pr = exp2f(fmaf(to_f32(row[q]), kLog2e, nl));
        store_grad(grow + q, w * ((q == tok ? 1.f : 0.f) - pr));
      }
      continue;
    }
    for (int e0 = u0; e0 < u1; e0 += kStepElems) {
      uint4 v[kBwdVecs];
      int e[kBwdVecs];
#pragma unroll
      for (int j = 0; j < kBwdVecs; ++j) {
        e[j] = e0 + ((int)threadIdx.x + j * kBwdNT) * VEC;
        if (e[j] + VEC <= V) v[j] = ld_stream(reinterpret_cast<const uint4*>(row + e[j]));
      }
#pragma unroll
      for (int j = 0; j < kBwdVecs; ++j) {
        if (e[j] + VEC <= V) {
          float x[VEC];
          if (sizeof(T) == 2) {
            x[0] = bf16_lo(v[j].x); x[1] = bf16_hi(v[j].x); x[2 % VEC] = bf16_lo(v[j].y); x[3 % VEC] = bf16_hi(v[j].y);
            x[4 % VEC] = bf16_lo(v[j].z); x[5 % VEC] = bf16_hi(v[j].z); x[6 % VEC] = bf16_lo(v[j].w); x[7 % VEC] = bf16_hi(v[j].w);
          } else {
            x[0] = __uint_as_float(v[j].x); x[1] = __uint_as_float(v[j].y); x[2] = __uint_as_float(v[j].z); x[3] = __uint_as_float(v[j].w);
          }
          float gr[VEC];
#pragma unroll
          for (int q = 0; q < VEC; ++q) {
            const float pr = ex2_approx(fmaf(x[q], kLog2e, nl));
            gr[q] = w * ((e[j] + q == tok ? 1.f : 0.f) - pr);
          }
          uint4 o;
          if (sizeof(T) == 2) {
            o.x = pack_bf16x2(gr[0], gr[1]); o.y = pack_bf16x2(gr[2 % VEC], gr[3 % VEC]);
            o.z = pack_bf16x2(gr[4 % VEC], gr[5 % VEC]); o.w = pack_bf16x2(gr[6 % VEC], gr[7 % VEC]);
          } else {
            o.x = __float_as_uint(gr[0]); o.y = __float_as_uint(gr[1]); o.z = __float_as_uint(gr[2]); o.w = __float_as_uint(gr[3]);
          }
          __stcs(reinterpret_cast<uint4*>(grow + e[j]), o);
        } else {
          for (int q = e[j]; q < V && q < e[j] + VEC; ++q) {  /* the ragged end of the row */
            const float pr = exp2f(fmaf(to_f32(row[q]), kLog2e, nl));
            store_grad(grow + q, w * ((q == tok ? 1.f : 0.f) - pr));
          }
        }
      }
    }
  }
}

extern "C" fork_status fork_logprob_backward(const fork_logprob_bwd_args* a, void* ws, size_t ws_bytes, void* stream) {
  if (!a) return FORK_ERR_INVALID_ARG;
  if (bad_source(a->logits, a->stride_b, a->stride_l, a->pos0, a->B, a->Lt, a->Ll, a->V, a->dtype))
    return FORK_ERR_INVALID_ARG;
  if (!a->tokens || !a->select || !a->lse || !a->dlogp || !a->grad) return FORK_ERR_INVALID_ARG;
  if (a->grad_stride_l < a->V || a->grad_stride_b < 0) return FORK_ERR_INVALID_ARG;
  fork_status s = check_workspace(ws, ws_bytes, a->B, a->Lt);
  if (s != FORK_OK) return s;
  if (a->B == 0) return FORK_OK;
  cudaStream_t st = (cudaStream_t)stream;
  DeviceInfo* dev;
  if (!device_info(&dev)) return FORK_ERR_CUDA;
  WsView w = ws_view(ws, a->B, a->Lt);
  SetupParams sp;
  memset(&sp, 0, sizeof(sp));
  sp.flags = a->select; sp.lo = nullptr; sp.hi = nullptr;
  sp.B = a->B; sp.Lt = a->Lt; sp.pos0 = a->pos0; sp.Ll = a->Ll; sp.C = 1; sp.G = 1; sp.min_units = 1;
  sp.hdr = w.hdr; sp.seq_off = w.seq_off; sp.expected = w.expected; sp.ticket = w.ticket; sp.rows = w.rows;
  const bool pdl = g_tune[FORK_TUNE_PDL].load() >= 0;
  if (launch(active_set_kernel, dim3(1), dim3(kSetupNT), st, pdl, sp) != cudaSuccess) return FORK_ERR_CUDA;
  BwdParams bp;
  memset(&bp, 0, sizeof(bp));
  bp.src = RowSource{a->logits, (long long)a->stride_b, (long long)a->stride_l, a->pos0, a->Ll, a->V};
  bp.grad = a->grad; bp.gstride_b = a->grad_stride_b; bp.gstride_l = a->grad_stride_l;
  bp.hdr = w.hdr; bp.rows = w.rows; bp.tokens = a->tokens; bp.lse = a->lse; bp.dlogp = a->dlogp; bp.Lt = a->Lt;
  bp.vector_ok = (source_is_vector_aligned(a->logits, a->stride_b, a->stride_l, a->dtype) &&
                  source_is_vector_aligned(a->grad, a->grad_stride_b, a->grad_stride_l, a->dtype)) ? 1 : 0;
  const int grid = dev->sms * 8;
  cudaError_t e = a->dtype == FORK_BF16 ? launch(logprob_backward_kernel<bf16_t>, dim3(grid), dim3(kBwdNT), st, pdl, bp)
                                        : launch(logprob_backward_kernel<float>, dim3(grid), dim3(kBwdNT), st, pdl, bp);
  return e == cudaSuccess ? FORK_OK : FORK_ERR_CUDA;
}

/* ---- ForkGRPO's training pass over the logits in one kernel ---------------------------------
 * fork_logprob, the derivative of Eq. 2 and fork_logprob_backward per selected row by ONE CTA: the
 * row is streamed once for (max, sum exp), the CTA's first thread turns that into log q(token), the
 * ratio and dJ/dlogp, and the row is streamed a second time for the gradient while most of it is
 * still in L2 (one row per SM in flight: 148 x 0.5 MB; measured: three quarters of the second pass
 * hit), so HBM sees about 1.25 reads and one write of every row instead of two reads and one write.
 * Advantage and 1 / (B |F_i|) per rollout come from a small kernel before it.  Eviction-priority
 * hints on the two passes changed nothing, a larger persisting-L2 set-aside made everything slower,
 * fewer CTAs (a smaller footprint in L2) were slower in proportion: a CTA's time per row is set by
 * the bytes it can keep in flight from registers (96 KB), not by HBM. */
constexpr int kFusedNT = 512;
/* 128-bit loads in flight per thread (as many as the register file holds without spilling): 96 KB per SM for
   fp32 rows, 64 KB for bf16 */
template <typename T> struct FusedLoads { static constexpr int n = sizeof(T) == 4 ? 12 : 8; };

struct GrpoFusedParams {
  RowSource src; void* grad; long long gstride_b, gstride_l;
  const WsHeader* hdr; const int2* rows;
  const int32_t* tokens; const float* logp_old;
  const float* adv; const float* scale;                       /* [B] each, from grpo_rollout_kernel; scale < 0 marks a skipped group */
  float* logp; float* lse; uint32_t* row_status; float* dlogp; float* ratio;
  int Lt, vector_ok; float eps_lo, eps_hi;
};

/* per rollout: A_i and 1 / (B |F_i|) (0 when F_i is empty, -1 for a group whose rewards are all equal) */
__global__ void __launch_bounds__(kGrpoNT) grpo_rollout_kernel(const float* reward, const uint8_t* select, int B, int Lt, int G,
                                                              float* adv, float* scale) {
  __shared__ double sh_mean, sh_sd;
  const int p = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nwarp = kGrpoNT / 32;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;");
  if (tid == 0) { double mean, sd; grpo_group_stats(reward, p, G, mean, sd); sh_mean = mean; sh_sd = sd; }
  __syncthreads();
  const bool skip = !(sh_sd > 0.0);
  for (int j = warp; j < G; j += nwarp) {
    const int i = p * G + j;
    const int nf = grpo_count_selected(select, i, Lt);
    if (lane == 0) {
      adv[i] = skip ? 0.f : (float)(((double)reward[i] - sh_mean) / sh_sd);
      scale[i] = skip ? -1.f : (nf > 0 ? 1.f / ((float)B * (float)nf) : 0.f);
    }
  }
}

template <typename T> __device__ __forceinline__ uint4 minus_inf_vector();
template <> __device__ __forceinline__ uint4 minus_inf_vector<bf16_t>() { return make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u); }
template <> __device__ __forceinline__ uint4 minus_inf_vector<float>() { return make_uint4(0xFF800000u, 0xFF800000u, 0xFF800000u, 0xFF800000u); }

template <typename T>
__device__ __forceinline__ void unpack_vector(const uint4& v, float (&x)[16 / sizeof(T)]) {
  constexpr int VEC = 16 / (int)sizeof(T);
  if (sizeof(T) == 2) {
    x[0] = bf16_lo(v.x); x[1] = bf16_hi(v.x); x[2 % VEC] = bf16_lo(v.y); x[3 % VEC] = bf16_hi(v.y);
    x[4 % VEC] = bf16_lo(v.z); x[5 % VEC] = bf16_hi(v.z); x[6 % VEC] = bf16_lo(v.w); x[7 % VEC] = bf16_hi(v.w);
  } else {
    x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y); x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
  }
}

/* running (reference, max, sum 2^((x - reference) L)) of one thread; the reference is the first finite
   maximum the thread meets and is raised only when a later value exceeds it by kRaiseNats */
struct LseAcc {
  float ref, m, s; bool have;
  __device__ __forceinline__ void init() { ref = 0.f; m = -INFINITY; s = 0.f; have = false; }
  __device__ __forceinline__ void meet(float vm) {           /* vm: maximum of the values about to be added (NaNs ignored) */
    if (!have) { if (vm > -INFINITY && vm < INFINITY) { ref = vm; have = true; } }
    else if (vm > ref + kRaiseNats && vm < INFINITY) { s *= ex2_approx((ref - vm) * kLog2e); ref = vm; }
    m = fmaxf(m, vm);
  }
  __device__ __forceinline__ void add(float x) { s += ex2_approx(fmaf(x, kLog2e, -ref * kLog2e)); }
  __device__ __forceinline__ Part part() const {
    if (!have) return Part{m, s, 0.f, kIdxNone};             /* nothing finite: (-inf, 0), or +inf / NaN in s */
    return Part{m, (m == ref) ? s : s * ex2_approx((ref - m) * kLog2e), 0.f, kIdxNone};
  }
};

template <typename T>
__global__ void __launch_bounds__(kFusedNT, 1) grpo_fused_kernel(const GrpoFusedParams p) {
  constexpr int VEC = 16 / (int)sizeof(T);
  constexpr int kFusedLoads = FusedLoads<T>::n;
  __shared__ Part sh_part[32];
  __shared__ float sh_w, sh_nl;
  __shared__ int sh_go;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int R = p.hdr->R, V = p.src.V;
  const int tid = (int)threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int r = (int)blockIdx.x; r < R; r += (int)gridDim.x) {
    const int2 bk = p.rows[r];
    const size_t at = (size_t)bk.x * p.Lt + bk.y;
    const int tok = p.tokens[at];
    const bool tok_ok = tok >= 0 && tok < V;
    const T* row = row_ptr<T>(p.src, bk.x, bk.y);
    T* grow = reinterpret_cast<T*>(p.grad) + ((long long)bk.x * p.gstride_b + (long long)(bk.y - p.src.pos0) * p.gstride_l);
    /* what the first thread needs once the sums are in: fetched now, used after the first pass */
    float x_tok = 0.f, lp_old = 0.f, adv = 0.f, sc = 0.f;
    if (tid == 0) {
      if (tok_ok) x_tok = to_f32(row[tok]);
      lp_old = p.logp_old[at]; adv = p.adv[bk.x]; sc = p.scale[bk.x];
    }
    /* ---- first pass: max and sum exp ---- */
    LseAcc acc;
    acc.init();
    const int nvec = p.vector_ok ? V / VEC : 0;
    const uint4* rv = reinterpret_cast<const uint4*>(row);
    for (int v0 = tid; v0 < nvec; v0 += kFusedNT * kFusedLoads) {
      uint4 q[kFusedLoads];
#pragma unroll
      for (int j = 0; j < kFusedLoads; ++j) {
        const int i = v0 + j * kFusedNT;
        q[j] = (i < nvec) ? ld_stream(rv + i) : minus_inf_vector<T>();
      }
      float vm = -INFINITY;
#pragma unroll
      for (int j = 0; j < kFusedLoads; ++j) {
        float x[VEC];
        unpack_vector<T>(q[j], x);
#pragma unroll
        for (int e = 0; e < VEC; ++e) vm = fmaxf(vm, x[e]);
      }
      acc.meet(vm);
#pragma unroll
      for (int j = 0; j < kFusedLoads; ++j) {
        float x[VEC];
        unpack_vector<T>(q[j], x);
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc.add(x[e]);
      }
    }
    for (int e = nvec * VEC + tid; e < V; e += kFusedNT) {   /* the ragged end of the row, or all of an unaligned one */
      const float x = to_f32(row[e]);
      acc.meet(x);
      acc.add(x);
    }
    Part part = part_warp_reduce(acc.part());
    __syncthreads();                                         /* the previous row's readers of the shared values are done */
    if (lane == 0) sh_part[warp] = part;
    __syncthreads();
    if (warp == 0) {
      part = part_warp_reduce(lane < kFusedNT / 32 ? sh_part[lane] : part_empty());
      if (lane == 0) {
        const bool bad = !isfinite(part.s) || !(part.m > -INFINITY) || part.m == INFINITY;
        const float lns = ln_approx(part.s);
        uint32_t st = bad ? (uint32_t)FORK_ROW_NONFINITE : 0u;
        const float qnan = __int_as_float(0x7fc00000);
        float lp;
        if (!tok_ok) { st |= FORK_ROW_BAD_TOKEN; lp = 0.f; }
        else if (bad) lp = qnan;
        else lp = (x_tok - part.m) - lns;                     /* x_tok - m - ln s */
        const float lse = bad ? qnan : part.m + lns;
        float rho, term, d;
        grpo_token(lp, lp_old, adv, sc < 0.f, sc < 0.f ? 0.f : sc, p.eps_lo, p.eps_hi, rho, term, d);
        p.logp[at] = lp;
        if (p.lse) p.lse[at] = lse;
        if (p.row_status) p.row_status[at] = st;
        if (p.dlogp) p.dlogp[at] = d;
        if (p.ratio) p.ratio[at] = rho;
        sh_w = d; sh_nl = -lse * kLog2e; sh_go = tok_ok ? 1 : 0;
      }
    }
    __syncthreads();
    if (!sh_go) continue;                                    /* scored as FORK_ROW_BAD_TOKEN: no gradient (uniform over the CTA) */
    /* ---- second pass: grad = dlogp * (1[v = token] - exp(x - lse)), the row coming from L2 ---- */
    const float w = sh_w, nl = sh_nl;
    uint4* gv = reinterpret_cast<uint4*>(grow);
    for (int v0 = tid; v0 < nvec; v0 += kFusedNT * kFusedLoads) {
      uint4 q[kFusedLoads];
#pragma unroll
      for (int j = 0; j < kFusedLoads; ++j) {
        const int i = v0 + j * kFusedNT;
        if (i < nvec) q[j] = ld_stream(rv + i);
      }
#pragma unroll
      for (int j = 0; j < kFusedLoads; ++j) {
        const int i = v0 + j * kFusedNT;
        if (i < nvec) {
          float x[VEC], gr[VEC];
          unpack_vector<T>(q[j], x);
#pragma unroll
          for (int e = 0; e < VEC; ++e) gr[e] = w * ((i * VEC + e == tok ? 1.f : 0.f) - ex2_approx(fmaf(x[e], kLog2e, nl)));
          uint4 o;
          if (sizeof(T) == 2) {
            o.x = pack_bf16x2(gr[0], gr[1]); o.y = pack_bf16x2(gr[2 % VEC], gr[3 % VEC]);
            o.z = pack_bf16x2(gr[4 % VEC], gr[5 % VEC]); o.w = pack_bf16x2(gr[6 % VEC], gr[7 % VEC]);
          } else {
            o.x = __float_as_uint(gr[0]); o.y = __float_as_uint(gr[1]); o.z = __float_as_uint(gr[2]); o.w = __float_as_uint(gr[3]);
          }
          __stcs(gv + i, o);
        }
      }
    }
    for (int e = nvec * VEC + tid; e < V; e += kFusedNT) {
      const float pr = exp2f(fmaf(to_f32(row[e]), kLog2e, nl));
      store_grad(grow + e, w * ((e == tok ? 1.f : 0.f) - pr));
    }
  }
}

/* The same pass for 16-byte aligned rows, fed by bulk copies instead of register loads, by a pair
   of CTAs (a cluster of two) per row, each on one half of it.  A producer lane copies the half row
   in 16 KB pieces into a ring in shared memory -- first for the sums, then, straight behind, once
   more for the gradient, then the next row -- and sixteen consumer warps work through the stages in
   that order.  What is in flight is the ring (192 KB), not what the register file holds; the second
   pass's pieces arrive while the first pass is still being summed, and the next row's first pass
   streams in under the gradient stores.  The two CTAs exchange their (max, sum) through each
   other's shared memory (a 16-byte remote store and a remote mbarrier arrival each way; nothing
   spins on global memory) and both work out the row's values from the two halves in the same order.
   Why pairs: with one CTA per row the second pass found only half of the row still in L2 (148 rows of
   0.5 MB in flight, and the gradient stores pass through L2 too); with half the rows in flight it
   finds nearly all of it.  Every wait is bounded; the cluster-wide barriers at the two ends of the
   kernel are reached by every CTA on every path. */
constexpr int kFrStageBytes = 16384;
constexpr int kFrStages = 12;
constexpr int kFrWarps = 16;
constexpr int kFrPerSm = 1;
constexpr int kFrConsumers = kFrWarps * 32;
constexpr int kFrThreads = kFrConsumers + 32;
constexpr uint32_t kFrSpinLimit = 1u << 24;

constexpr int kFrCluster = 2;
struct FrSmem {
  unsigned long long full[kFrStages], empty[kFrStages];
  unsigned long long red, go;                              /* the warps' sums are in / the row's values are out */
  unsigned long long xbar;                                 /* both halves' sums are in xpart (one arrival per CTA of the pair) */
  float4 xpart[2][kFrCluster];                             /* [row parity][rank]: (m, s, -, -) of each half */
  Part part[kFrWarps];
  float w, nl;
  int abort;
};
constexpr size_t kFrSmemBytes = (size_t)kFrStages * kFrStageBytes + sizeof(FrSmem) + 128;

__device__ __forceinline__ uint32_t fr_peer_addr(const void* local, uint32_t rank) {
  uint32_t ra;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(smem_u32(local)), "r"(rank));
  return ra;
}
__device__ __forceinline__ bool fr_try_wait_cluster(unsigned long long* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
template <bool CLUSTER_SCOPE = false>
__device__ __forceinline__ bool fr_wait(unsigned long long* bar, uint32_t parity, FrSmem& sm, const WsHeader* hdr) {
  for (uint32_t i = 0; i < kFrSpinLimit; ++i) {
    if (CLUSTER_SCOPE ? fr_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u && *reinterpret_cast<volatile int*>(&sm.abort)) return false;
  }
  *reinterpret_cast<volatile int*>(&sm.abort) = 1;
  atomicOr(const_cast<uint32_t*>(&hdr->dev_status), (uint32_t)FORK_DEV_TIMEOUT);
  return false;
}

template <typename T>
__global__ void __launch_bounds__(kFrThreads, kFrPerSm) grpo_fused_ring_kernel(const GrpoFusedParams p) {
  constexpr int VEC = 16 / (int)sizeof(T);
  constexpr int kStageVecs = kFrStageBytes / 16;
  extern __shared__ unsigned char fr_raw[];
  unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(fr_raw) + 127) & ~(uintptr_t)127);
  FrSmem& sm = *reinterpret_cast<FrSmem*>(ring + (size_t)kFrStages * kFrStageBytes);
  const int tid = (int)threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (int s = 0; s < kFrStages; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], kFrWarps); }
    mbar_init(&sm.red, kFrWarps); mbar_init(&sm.go, 1); mbar_init(&sm.xbar, kFrCluster);
    sm.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  /* nobody writes into a peer's shared memory before the peer has set its barriers up */
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int R = p.hdr->R, V = p.src.V;
  const uint32_t rank = (uint32_t)blockIdx.x % kFrCluster;
  const int cid = (int)blockIdx.x / kFrCluster, ncl = (int)gridDim.x / kFrCluster;
  const int nvec_row = V / VEC;                              /* whole 128-bit vectors of a row; the rest by plain loads */
  const int nv_half = (nvec_row + kFrCluster - 1) / kFrCluster;
  const int vbase = min((int)rank * nv_half, nvec_row);      /* this CTA's vectors: [vbase, vbase + nvec) */
  const int nvec = min(nv_half, nvec_row - vbase);
  const int nchunk = (nvec + kStageVecs - 1) / kStageVecs;
  const bool has_tail = rank == kFrCluster - 1;              /* the last CTA of the pair takes the ragged end */
  if (warp == kFrWarps) {
    /* ---------------- producer ---------------- */
    if (lane == 0) {
      uint32_t n = 0;
      bool ok = true;
      for (int r = cid; r < R && ok; r += ncl) {
        const int2 bk = p.rows[r];
        const int tok = p.tokens[(size_t)bk.x * p.Lt + bk.y];
        const int passes = (tok >= 0 && tok < V) ? 2 : 1;
        const unsigned char* row = reinterpret_cast<const unsigned char*>(row_ptr<T>(p.src, bk.x, bk.y)) + (size_t)vbase * 16;
        for (int pass = 0; pass < passes && ok; ++pass)
          for (int c = 0; c < nchunk; ++c, ++n) {
            const uint32_t s = n % kFrStages, ph = (n / kFrStages) & 1u;
            if (!fr_wait(&sm.empty[s], ph ^ 1u, sm, p.hdr)) { ok = false; break; }
            const uint32_t bytes = (uint32_t)min(kStageVecs, nvec - c * kStageVecs) * 16u;
            mbar_arrive_expect_tx(&sm.full[s], bytes);
            bulk_copy_g2s(ring + (size_t)s * kFrStageBytes, row + (size_t)c * kFrStageBytes, bytes, &sm.full[s]);
          }
      }
      if (!ok) {                                             /* do not leave with copies still landing */
        const uint32_t first = n > (uint32_t)kFrStages ? n - (uint32_t)kFrStages : 0u;
        for (uint32_t q = first; q < n; ++q) {
          unsigned long long* bar = &sm.full[q % kFrStages];
          const uint32_t par = (q / kFrStages) & 1u;
          for (uint32_t i = 0; i < kFrSpinLimit && !mbar_try_wait(bar, par); ++i) {}
        }
      }
    }
  } else {
    /* ---------------- consumers ---------------- */
    uint32_t n = 0, rows_done = 0;
    bool ok = true;
    for (int r = cid; r < R && ok; r += ncl, ++rows_done) {
      const int2 bk = p.rows[r];
      const size_t at = (size_t)bk.x * p.Lt + bk.y;
      const int tok = p.tokens[at];
      const bool tok_ok = tok >= 0 && tok < V;
      const T* row = row_ptr<T>(p.src, bk.x, bk.y);
      T* grow = reinterpret_cast<T*>(p.grad) + ((long long)bk.x * p.gstride_b + (long long)(bk.y - p.src.pos0) * p.gstride_l);
      float x_tok = 0.f, lp_old = 0.f, adv = 0.f, sc = 0.f;
      if (tid == 0) {
        if (tok_ok) x_tok = to_f32(row[tok]);
        lp_old = p.logp_old[at]; adv = p.adv[bk.x]; sc = p.scale[bk.x];
      }
      /* ---- first pass over this CTA's half ---- */
      LseAcc acc;
      acc.init();
      for (int c = 0; c < nchunk; ++c, ++n) {
        const uint32_t s = n % kFrStages, ph = (n / kFrStages) & 1u;
        if (!__all_sync(0xffffffffu, fr_wait(&sm.full[s], ph, sm, p.hdr))) { ok = false; break; }   /* the whole warp stays or goes */
        const uint4* st = reinterpret_cast<const uint4*>(ring + (size_t)s * kFrStageBytes);
        const int nv = min(kStageVecs, nvec - c * kStageVecs);
        uint4 q[kStageVecs / kFrConsumers];
#pragma unroll
        for (int j = 0; j < kStageVecs / kFrConsumers; ++j) {
          const int i = tid + j * kFrConsumers;
          q[j] = (i < nv) ? st[i] : minus_inf_vector<T>();
        }
        float vm = -INFINITY;
#pragma unroll
        for (int j = 0; j < kStageVecs / kFrConsumers; ++j) {
          float x[VEC];
          unpack_vector<T>(q[j], x);
#pragma unroll
          for (int e = 0; e < VEC; ++e) vm = fmaxf(vm, x[e]);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.empty[s]);            /* every loaded word has been used, so the values sit in registers: the stage may be refilled */
        acc.meet(vm);
#pragma unroll
        for (int j = 0; j < kStageVecs / kFrConsumers; ++j) {
          float x[VEC];
          unpack_vector<T>(q[j], x);
#pragma unroll
          for (int e = 0; e < VEC; ++e) acc.add(x[e]);
        }
      }
      if (!ok) break;
      if (has_tail)
        for (int e = nvec_row * VEC + tid; e < V; e += kFrConsumers) {   /* the ragged end of the row */
          const float x = to_f32(row[e]);
          acc.meet(x);
          acc.add(x);
        }
      const Part mine = part_warp_reduce(acc.part());
      if (lane == 0) { sm.part[warp] = mine; mbar_arrive(&sm.red); }
      if (warp == 0) {
        if (!__all_sync(0xffffffffu, fr_wait(&sm.red, rows_done & 1u, sm, p.hdr))) { ok = false; break; }
        const Part half = part_warp_reduce(lane < kFrWarps ? sm.part[lane] : part_empty());
        if (lane == 0) {
          /* this half's (m, s) into the same slot of both CTAs, then one arrival on each CTA's barrier;
             the arrival releases the store, the wait below acquires the peer's */
          const uint32_t par = rows_done & 1u;
          const float4 mine4 = make_float4(half.m, half.s, 0.f, 0.f);
          for (uint32_t j = 0; j < (uint32_t)kFrCluster; ++j) {
            const uint32_t slot = fr_peer_addr(&sm.xpart[par][rank], j), bar = fr_peer_addr(&sm.xbar, j);
            asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};"
                         :: "r"(slot), "f"(mine4.x), "f"(mine4.y), "f"(mine4.z), "f"(mine4.w) : "memory");
            asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" :: "r"(bar) : "memory");
          }
          if (!fr_wait<true>(&sm.xbar, par, sm, p.hdr)) ok = false;
          Part part = part_empty();
          for (int j = 0; j < kFrCluster; ++j) {
            const volatile float* h = reinterpret_cast<const volatile float*>(&sm.xpart[par][j]);
            part = part_merge(part, Part{h[0], h[1], 0.f, kIdxNone});
          }
          const bool bad = !isfinite(part.s) || !(part.m > -INFINITY) || part.m == INFINITY;
          const float lns = ln_approx(part.s);
          uint32_t stt = bad ? (uint32_t)FORK_ROW_NONFINITE : 0u;
          const float qnan = __int_as_float(0x7fc00000);
          float lp;
          if (!tok_ok) { stt |= FORK_ROW_BAD_TOKEN; lp = 0.f; }
          else if (bad) lp = qnan;
          else lp = (x_tok - part.m) - lns;                   /* x_tok - m - ln s */
          const float lse = bad ? qnan : part.m + lns;
          float rho, term, d;
          grpo_token(lp, lp_old, adv, sc < 0.f, sc < 0.f ? 0.f : sc, p.eps_lo, p.eps_hi, rho, term, d);
          if (rank == 0 && ok) {
            p.logp[at] = lp;
            if (p.lse) p.lse[at] = lse;
            if (p.row_status) p.row_status[at] = stt;
            if (p.dlogp) p.dlogp[at] = d;
            if (p.ratio) p.ratio[at] = rho;
          }
          sm.w = d; sm.nl = -lse * kLog2e;
          if (ok) mbar_arrive(&sm.go);
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
      }
      if (!__all_sync(0xffffffffu, fr_wait(&sm.go, rows_done & 1u, sm, p.hdr))) { ok = false; break; }
      if (!tok_ok) continue;                                 /* scored as FORK_ROW_BAD_TOKEN: no gradient, and no second pass was copied */
      /* ---- second pass ---- */
      const float w = sm.w, nl = sm.nl;
      uint4* gv = reinterpret_cast<uint4*>(grow) + vbase;
      for (int c = 0; c < nchunk; ++c, ++n) {
        const uint32_t s = n % kFrStages, ph = (n / kFrStages) & 1u;
        if (!__all_sync(0xffffffffu, fr_wait(&sm.full[s], ph, sm, p.hdr))) { ok = false; break; }
        const uint4* st = reinterpret_cast<const uint4*>(ring + (size_t)s * kFrStageBytes);
        const int nv = min(kStageVecs, nvec - c * kStageVecs);
        uint4 q[kStageVecs / kFrConsumers];
#pragma unroll
        for (int j = 0; j < kStageVecs / kFrConsumers; ++j) {
          const int i = tid + j * kFrConsumers;
          if (i < nv) q[j] = st[i];
        }
        uint4 out[kStageVecs / kFrConsumers];
#pragma unroll
        for (int j = 0; j < kStageVecs / kFrConsumers; ++j) {
          const int i = tid + j * kFrConsumers;
          if (i < nv) {
            const int e0 = (vbase + c * kStageVecs + i) * VEC;
            float x[VEC], gr[VEC];
            unpack_vector<T>(q[j], x);
#pragma unroll
            for (int e = 0; e < VEC; ++e) gr[e] = w * ((e0 + e == tok ? 1.f : 0.f) - ex2_approx(fmaf(x[e], kLog2e, nl)));
            uint4& o = out[j];
            if (sizeof(T) == 2) {
              o.x = pack_bf16x2(gr[0], gr[1]); o.y = pack_bf16x2(gr[2 % VEC], gr[3 % VEC]);
              o.z = pack_bf16x2(gr[4 % VEC], gr[5 % VEC]); o.w = pack_bf16x2(gr[6 % VEC], gr[7 % VEC]);
            } else {
              o.x = __float_as_uint(gr[0]); o.y = __float_as_uint(gr[1]); o.z = __float_as_uint(gr[2]); o.w = __float_as_uint(gr[3]);
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.empty[s]);            /* the gradients are computed: every loaded word has been used */
#pragma unroll
        for (int j = 0; j < kStageVecs / kFrConsumers; ++j) {
          const int i = tid + j * kFrConsumers;
          if (i < nv) __stcs(gv + (size_t)c * kStageVecs + i, out[j]);
        }
      }
      if (!ok) break;
      if (has_tail)
        for (int e = nvec_row * VEC + tid; e < V; e += kFrConsumers) {
          const float pr = exp2f(fmaf(to_f32(row[e]), kLog2e, nl));
          store_grad(grow + e, w * ((e == tok ? 1.f : 0.f) - pr));
        }
    }
  }
  __syncthreads();
  /* nobody leaves while its peer may still store into its shared memory */
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

extern "C" fork_status fork_grpo_fused(const fork_grpo_fused_args* a, void* ws, size_t ws_bytes, void* stream) {
  if (!a) return FORK_ERR_INVALID_ARG;
  if (bad_source(a->logits, a->stride_b, a->stride_l, 0, a->B, a->Lt, a->Lt, a->V, a->dtype)) return FORK_ERR_INVALID_ARG;
  if (!a->tokens || !a->select || !a->logp_old || !a->reward || !a->grad || !a->logp || !a->seq_obj) return FORK_ERR_INVALID_ARG;
  if (a->group <= 0 || a->B % a->group != 0) return FORK_ERR_INVALID_ARG;
  if (!(a->eps_lo >= 0.f) || !(a->eps_hi >= 0.f)) return FORK_ERR_INVALID_ARG;
  if (a->grad_stride_l < a->V || a->grad_stride_b < 0) return FORK_ERR_INVALID_ARG;
  fork_status s = check_workspace(ws, ws_bytes, a->B, a->Lt);
  if (s != FORK_OK) return s;
  if (a->B == 0) {
    if (a->objective && cudaMemsetAsync(a->objective, 0, sizeof(float), (cudaStream_t)stream) != cudaSuccess) return FORK_ERR_CUDA;
    return FORK_OK;
  }
  cudaStream_t st = (cudaStream_t)stream;
  DeviceInfo* dev;
  if (!device_info(&dev)) return FORK_ERR_CUDA;
  WsView w = ws_view(ws, a->B, a->Lt);
  const bool pdl = g_tune[FORK_TUNE_PDL].load() >= 0;
  /* the rows to score: the selected positions (the fallback steps F_i of every rollout) */
  SetupParams sp;
  memset(&sp, 0, sizeof(sp));
  sp.flags = a->select; sp.lo = nullptr; sp.hi = nullptr;
  sp.B = a->B; sp.Lt = a->Lt; sp.pos0 = 0; sp.Ll = a->Lt; sp.C = 1; sp.G = 1; sp.min_units = 1;
  sp.hdr = w.hdr; sp.seq_off = w.seq_off; sp.expected = w.expected; sp.ticket = w.ticket; sp.rows = w.rows;
  if (launch(active_set_kernel, dim3(1), dim3(kSetupNT), st, pdl, sp) != cudaSuccess) return FORK_ERR_CUDA;
  /* advantage and 1 / (B |F_i|) per rollout, in a corner of the workspace this path does not use otherwise */
  float* adv_ws = reinterpret_cast<float*>(w.final_rec);
  float* scale_ws = adv_ws + a->B;
  {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)(a->B / a->group)); cfg.blockDim = dim3(kGrpoNT); cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (pdl) {
      attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[0].val.programmaticStreamSerializationAllowed = 1;
      cfg.attrs = attr; cfg.numAttrs = 1;
    }
    if (cudaLaunchKernelEx(&cfg, grpo_rollout_kernel, a->reward, a->select, a->B, a->Lt, a->group, adv_ws, scale_ws) != cudaSuccess)
      return FORK_ERR_CUDA;
    g_launches.fetch_add(1);
  }
  GrpoFusedParams fp;
  memset(&fp, 0, sizeof(fp));
  fp.src = RowSource{a->logits, (long long)a->stride_b, (long long)a->stride_l, 0, a->Lt, a->V};
  fp.grad = a->grad; fp.gstride_b = a->grad_stride_b; fp.gstride_l = a->grad_stride_l;
  fp.hdr = w.hdr; fp.rows = w.rows; fp.tokens = a->tokens; fp.logp_old = a->logp_old; fp.adv = adv_ws; fp.scale = scale_ws;
  fp.logp = a->logp; fp.lse = a->lse; fp.row_status = a->row_status; fp.dlogp = a->dlogp; fp.ratio = a->ratio;
  fp.Lt = a->Lt; fp.eps_lo = a->eps_lo; fp.eps_hi = a->eps_hi;
  fp.vector_ok = (source_is_vector_aligned(a->logits, a->stride_b, a->stride_l, a->dtype) &&
                  source_is_vector_aligned(a->grad, a->grad_stride_b, a->grad_stride_l, a->dtype)) ? 1 : 0;
  cudaError_t e;
  if (fp.vector_ok && g_tune[FORK_TUNE_VARIANT].load() != 1) {
    static std::once_flag smem_once[64];
    int di = 0;
    if (cudaGetDevice(&di) != cudaSuccess || di < 0 || di >= 64) return FORK_ERR_CUDA;
    std::call_once(smem_once[di], [] {
      cudaFuncSetAttribute(grpo_fused_ring_kernel<bf16_t>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFrSmemBytes);
      cudaFuncSetAttribute(grpo_fused_ring_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFrSmemBytes);
    });
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)(dev->sms * kFrPerSm / kFrCluster * kFrCluster)); cfg.blockDim = dim3(kFrThreads);
    cfg.dynamicSmemBytes = kFrSmemBytes; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kFrCluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    {
      /* a persistent grid: no more clusters than can be resident together (a cluster that had to wait for
         another to finish would start its share of the rows when the others are done with theirs) */
      static int max_clusters[64][2];
      static std::once_flag occ_once[64][2];
      const int ti = a->dtype == FORK_BF16 ? 0 : 1;
      std::call_once(occ_once[di][ti], [&] {
        int n = 0;
        cudaError_t oe = ti == 0 ? cudaOccupancyMaxActiveClusters(&n, grpo_fused_ring_kernel<bf16_t>, &cfg)
                                 : cudaOccupancyMaxActiveClusters(&n, grpo_fused_ring_kernel<float>, &cfg);
        max_clusters[di][ti] = (oe == cudaSuccess && n > 0) ? n : 0;
      });
      const int want = dev->sms * kFrPerSm / kFrCluster;
      const int ncl = max_clusters[di][ti] > 0 && max_clusters[di][ti] < want ? max_clusters[di][ti] : want;
      cfg.gridDim = dim3((unsigned)(ncl * kFrCluster));
    }
    if (pdl) {
      attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[1].val.programmaticStreamSerializationAllowed = 1;
      cfg.numAttrs = 2;
    }
    e = a->dtype == FORK_BF16 ? cudaLaunchKernelEx(&cfg, grpo_fused_ring_kernel<bf16_t>, fp)
                              : cudaLaunchKernelEx(&cfg, grpo_fused_ring_kernel<float>, fp);
    if (e == cudaSuccess) g_launches.fetch_add(1);
    else (void)cudaGetLastError();                          /* e.g. no room for clusters on this device: the plain kernel below */
  }
  if (!(fp.vector_ok && g_tune[FORK_TUNE_VARIANT].load() != 1) || e != cudaSuccess) {
    /* rows that are not 16-byte aligned (or variant 1): loads from registers */
    e = a->dtype == FORK_BF16 ? launch(grpo_fused_kernel<bf16_t>, dim3(dev->sms), dim3(kFusedNT), st, pdl, fp)
                              : launch(grpo_fused_kernel<float>, dim3(dev->sms), dim3(kFusedNT), st, pdl, fp);
  }
  if (e != cudaSuccess) return FORK_ERR_CUDA;
  /* the objective itself and the per-rollout outputs, from the log-probabilities just written */
  fork_grpo_args g;
  memset(&g, 0, sizeof(g));
  g.B = a->B; g.Lt = a->Lt; g.group = a->group;
  g.logp_new = a->logp; g.logp_old = a->logp_old; g.select = a->select; g.reward = a->reward;
  g.eps_lo = a->eps_lo; g.eps_hi = a->eps_hi;
  g.seq_obj = a->seq_obj; g.objective = a->objective; g.adv = a->adv; g.skipped = a->skipped;
  return fork_grpo_loss(&g, stream);
}

/* ---- vocabulary-parallel entry points ------------------------------------------------------- */
extern "C" fork_status fork_vp_reduce(const fork_step_args* a, int32_t vocab_offset, void* part_out, void* key_out,
                                      void* ws, size_t ws_bytes, void* stream) {
  fork_status s = check_step_args(a, true);
  if (s != FORK_OK) return s;
  if (!part_out || vocab_offset < 0 || (int64_t)vocab_offset + a->V > 0x7fffffffLL) return FORK_ERR_INVALID_ARG;
  if (a->temperature > 0.f && !key_out) return FORK_ERR_INVALID_ARG;
  if (((uintptr_t)part_out % 16) != 0 || ((uintptr_t)key_out % 16) != 0) return FORK_ERR_INVALID_ARG;
  s = check_workspace(ws, ws_bytes, a->B, a->Lt);
  if (s != FORK_OK) return s;
  if (a->B == 0) return FORK_OK;
  VpLocal vp{vocab_offset, (float4*)part_out, (float4*)key_out};
  return step_impl(a, a->blk_lo, a->blk_hi, ws, (cudaStream_t)stream, &vp);
}

extern "C" fork_status fork_vp_reduce_peers(const fork_step_args* a, int32_t vocab_offset, int32_t rank, int32_t n_ranks,
                                            void* const* peer_parts, void* const* peer_keys,
                                            void* ws, size_t ws_bytes, void* stream) {
  fork_status s = check_step_args(a, true);
  if (s != FORK_OK) return s;
  if (!peer_parts || n_ranks <= 0 || n_ranks > FORK_VP_MAX_RANKS || rank < 0 || rank >= n_ranks) return FORK_ERR_INVALID_ARG;
  if (vocab_offset < 0 || (int64_t)vocab_offset + a->V > 0x7fffffffLL) return FORK_ERR_INVALID_ARG;
  if (a->temperature > 0.f && !peer_keys) return FORK_ERR_INVALID_ARG;
  for (int j = 0; j < n_ranks; ++j) {
    if (!peer_parts[j] || ((uintptr_t)peer_parts[j] % 16) != 0) return FORK_ERR_INVALID_ARG;
    if (a->temperature > 0.f && (!peer_keys[j] || ((uintptr_t)peer_keys[j] % 16) != 0)) return FORK_ERR_INVALID_ARG;
  }
  s = check_workspace(ws, ws_bytes, a->B, a->Lt);
  if (s != FORK_OK) return s;
  if (a->B == 0) return FORK_OK;
  VpLocal vp{vocab_offset, nullptr, nullptr};
  vp.rank = rank; vp.peers = n_ranks; vp.peer_parts = peer_parts; vp.peer_keys = a->temperature > 0.f ? peer_keys : nullptr;
  return step_impl(a, a->blk_lo, a->blk_hi, ws, (cudaStream_t)stream, &vp);
}

extern "C" fork_status fork_vp_select(const fork_step_args* a, const void* parts, const void* keys, int32_t n_ranks,
                                      void* ws, size_t ws_bytes, void* stream) {
  if (!a || a->B < 0 || a->Lt <= 0 || !a->tokens || !a->mask || !a->blk_lo || !a->blk_hi) return FORK_ERR_INVALID_ARG;
  if ((int64_t)a->B * a->Lt > (int64_t)1 << 30) return FORK_ERR_INVALID_ARG;
  if (a->threshold != a->threshold) return FORK_ERR_INVALID_ARG;
  if (a->fallback_mode < FORK_FALLBACK_LEFTMOST || a->fallback_mode > FORK_FALLBACK_RANDOM) return FORK_ERR_INVALID_ARG;
  if (a->fallback_mode == FORK_FALLBACK_RANDOM && !a->fallback_rand) return FORK_ERR_INVALID_ARG;
  if (!(a->temperature >= 0.f) || a->temperature > 3.0e38f) return FORK_ERR_INVALID_ARG;
  if (!parts || n_ranks <= 0 || (a->temperature > 0.f && !keys)) return FORK_ERR_INVALID_ARG;
  if (((uintptr_t)parts % 16) != 0 || ((uintptr_t)keys % 16) != 0) return FORK_ERR_INVALID_ARG;
  fork_status s = check_workspace(ws, ws_bytes, a->B, a->Lt);
  if (s != FORK_OK) return s;
  if (a->B == 0) return FORK_OK;
  cudaStream_t st = (cudaStream_t)stream;
  WsView w = ws_view(ws, a->B, a->Lt);
  const bool pdl = g_tune[FORK_TUNE_PDL].load() >= 0;
  SetupParams sp;
  memset(&sp, 0, sizeof(sp));
  sp.flags = a->mask; sp.lo = a->blk_lo; sp.hi = a->blk_hi;
  sp.B = a->B; sp.Lt = a->Lt; sp.pos0 = 0; sp.Ll = a->Lt; sp.C = 1; sp.G = 1; sp.min_units = 1;
  if (a->Ll > 0) { sp.pos0 = a->pos0; sp.Ll = a->Ll; }      /* the window the slices covered */
  sp.hdr = w.hdr; sp.seq_off = w.seq_off; sp.expected = w.expected; sp.ticket = w.ticket; sp.rows = w.rows;
  sp.n_unmasked = a->n_unmasked; sp.is_fallback = a->is_fallback; sp.fallback_pos = a->fallback_pos;
  if (launch(active_set_kernel, dim3(1), dim3(kSetupNT), st, pdl, sp) != cudaSuccess) return FORK_ERR_CUDA;
  ReduceParams rp;
  memset(&rp, 0, sizeof(rp));
  rp.B = a->B; rp.Lt = a->Lt; rp.C = 1; rp.min_units = 1;
  rp.hdr = w.hdr; rp.seq_off = w.seq_off; rp.expected = w.expected; rp.ticket = w.ticket;
  rp.rows = w.rows; rp.final_rec = w.final_rec; rp.parts = w.parts;
  rp.tokens = a->tokens; rp.mask = a->mask; rp.threshold = a->threshold; rp.step = a->step;
  rp.conf = a->conf; rp.cand = a->cand; rp.entropy = a->entropy; rp.logp = a->logp; rp.row_status = a->row_status;
  rp.commit_step = a->commit_step; rp.commit_fallback = a->commit_fallback; rp.commit_logp = a->commit_logp;
  rp.n_unmasked = a->n_unmasked; rp.is_fallback = a->is_fallback; rp.fallback_pos = a->fallback_pos;
  rp.nfe = a->nfe; rp.n_fallback = a->n_fallback;
  rp.fallback_mode = a->fallback_mode; rp.fallback_rand = a->fallback_rand;
  rp.vp_parts_in = (const float4*)parts; rp.vp_keys_in = (const float4*)keys; rp.vp_ranks = n_ranks;
  if (a->temperature > 0.f) rp.noise_c = (float)(1.4426950408889634 / (double)a->temperature);
  rp.sample_seed = a->sample_seed;
  const dim3 grid((unsigned)((a->B + kVpNT / 32 - 1) / (kVpNT / 32)));
  cudaError_t e = a->temperature > 0.f ? launch(vp_select_kernel<true>, grid, dim3(kVpNT), st, pdl, rp)
                                       : launch(vp_select_kernel<false>, grid, dim3(kVpNT), st, pdl, rp);
  return e == cudaSuccess ? FORK_OK : FORK_ERR_CUDA;
}

/* ---- the step fused into the LM-head GEMM -------------------------------------------------- */
typedef CUresult (*tensor_map_encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                         const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                         CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static tensor_map_encode_fn g_tensor_map_encode = nullptr;
static std::once_flag g_head_once;
static bool g_head_ready = false;

static void head_init() {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn) return;
  g_tensor_map_encode = (tensor_map_encode_fn)fn;
  g_head_ready = true;
}

/* a [rows, d] bf16 matrix, d contiguous, row stride `ld` elements, cut into boxes of box_rows x 64 with the 128-byte swizzle */
constexpr int FORK_HEAD_MAX_SPLITS = 256;                   /* column ranges (CTAs along the vocabulary) of a launch: at most the SM count */
static bool head_tensor_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t d, uint64_t ld, uint32_t box_rows) {
  const cuuint64_t dims[2] = {d, rows};
  const cuuint64_t strides[1] = {ld * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kHeadK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return g_tensor_map_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

extern "C" size_t fork_head_sample_scratch_bytes(int32_t B, int32_t Ll, int32_t V) {
  if (B < 0 || Ll <= 0 || V <= 0) return 0;
  const size_t rows_pad = (((size_t)(B > 0 ? B : 1) * (size_t)Ll + kHeadM - 1) / kHeadM) * kHeadM;
  const size_t cells = (size_t)((V + kHeadGroup - 1) / kHeadGroup) * rows_pad;
  return 2 * align_up(cells * 4, 256) + align_up(cells, 256) + align_up(rows_pad * sizeof(float4), 256) +
         align_up((size_t)FORK_HEAD_MAX_SPLITS * rows_pad * sizeof(float), 256);
}

static fork_status check_head_args(const fork_step_args* a, const fork_head_args* h, bool need_bounds) {
  if (!a || !h) return FORK_ERR_INVALID_ARG;
  if (a->B < 0 || a->Lt <= 0 || a->Ll <= 0 || a->V <= 0 || a->pos0 < 0 || !a->tokens || !a->mask) return FORK_ERR_INVALID_ARG;
  if (need_bounds && (!a->blk_lo || !a->blk_hi)) return FORK_ERR_INVALID_ARG;
  if ((int64_t)a->B * a->Lt > (int64_t)1 << 30) return FORK_ERR_INVALID_ARG;
  if (need_bounds && !h->row_pos0 && a->pos0 + (int64_t)a->Ll > a->Lt) return FORK_ERR_INVALID_ARG;
  if (a->threshold != a->threshold) return FORK_ERR_INVALID_ARG;
  if (a->fallback_mode < FORK_FALLBACK_LEFTMOST || a->fallback_mode > FORK_FALLBACK_RANDOM) return FORK_ERR_INVALID_ARG;
  if (a->fallback_mode == FORK_FALLBACK_RANDOM && !a->fallback_rand) return FORK_ERR_INVALID_ARG;
  if (!(a->temperature >= 0.f) || a->temperature > 3.0e38f) return FORK_ERR_INVALID_ARG;
  if (!h->hidden || !h->weight || h->d <= 0 || h->d % kHeadK != 0) return FORK_ERR_INVALID_ARG;
  if (h->hidden_stride < h->d || h->weight_stride < h->d) return FORK_ERR_INVALID_ARG;
  if (((uintptr_t)h->hidden % 16) != 0 || ((uintptr_t)h->weight % 16) != 0 || (h->hidden_stride % 8) != 0 ||
      (h->weight_stride % 8) != 0) return FORK_ERR_INVALID_ARG;        /* tensor copies need 16-byte aligned rows */
  if (a->temperature > 0.f && (!a->sample_scratch || ((uintptr_t)a->sample_scratch % 256) != 0 ||
                               a->sample_scratch_bytes < fork_head_sample_scratch_bytes(a->B, a->Ll, a->V)))
    return FORK_ERR_WORKSPACE;                                         /* drawn candidates need their scratch */
  return FORK_OK;
}

/* one fused-head step on the stream: windows [row_pos0[b] (or pos0), + Ll) of every sequence, blocks lo / hi */
static fork_status head_step_impl(const fork_step_args* a, const fork_head_args* h, const int32_t* lo, const int32_t* hi,
                                  const int32_t* row_pos0, void* ws, cudaStream_t st, LoopCtl* loop) {
  DeviceInfo* dev;
  if (!device_info(&dev)) return FORK_ERR_CUDA;
  std::call_once(g_head_once, head_init);
  if (!g_head_ready) return FORK_ERR_CUDA;
  {
    static std::once_flag smem_once[64];
    int di = 0;
    if (cudaGetDevice(&di) != cudaSuccess || di < 0 || di >= 64) return FORK_ERR_CUDA;
    std::call_once(smem_once[di], [] {
      cudaFuncSetAttribute(head_gemm_reduce_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kHeadSmemLimit);
      cudaFuncSetAttribute(head_gemm_reduce_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kHeadSmemLimit);
    });
  }
  WsView w = ws_view(ws, a->B, a->Lt);
  const bool pdl = g_tune[FORK_TUNE_PDL].load() >= 0;

  HeadParams hp;
  memset(&hp, 0, sizeof(hp));
  hp.rows = a->B * a->Ll; hp.V = a->V; hp.d = h->d;
  hp.n_groups = (a->V + kHeadGroup - 1) / kHeadGroup;
  hp.m_blocks = (hp.rows + kHeadM - 1) / kHeadM;
  hp.unit = hp.m_blocks == 1 ? 1 : kHeadN / kHeadGroup;
  const int n_units = (hp.n_groups + hp.unit - 1) / hp.unit;
  int splits = dev->sms / hp.m_blocks;
  if (splits < 1) splits = 1;
  if (splits > FORK_HEAD_MAX_SPLITS) splits = FORK_HEAD_MAX_SPLITS;   /* (what the sample scratch has room for) */
  if (splits > n_units) splits = n_units;
  hp.n_splits = splits;
  hp.u_base = n_units / splits; hp.u_rem = n_units % splits;
  hp.a_box_rows = head_a_box_rows(hp.rows);
  hp.stages = head_stages(hp.a_box_rows);
  const size_t head_smem = (size_t)hp.stages * head_stage_bytes(hp.a_box_rows) + kHeadSmemExtra;
  if ((size_t)hp.n_splits * hp.m_blocks * kHeadM > (size_t)a->B * a->Lt + kHeadPartsExtra) return FORK_ERR_WORKSPACE;
  hp.parts = w.head_parts; hp.hdr = w.hdr;
  const bool drawn = a->temperature > 0.f;
  if (drawn) {
    /* per 32-column chunk and window row: log2-weight, drawn logit, drawn index; then a draw record per row */
    const size_t cells = (size_t)hp.n_groups * hp.m_blocks * kHeadM;
    char* base = (char*)a->sample_scratch;
    hp.lw = (float*)base;
    hp.xt = (float*)(base + align_up(cells * 4, 256));
    hp.jt = (unsigned char*)(base + 2 * align_up(cells * 4, 256));
    hp.draw = (float4*)(base + 2 * align_up(cells * 4, 256) + align_up(cells, 256));
    hp.lws = (float*)(base + 2 * align_up(cells * 4, 256) + align_up(cells, 256) + align_up((size_t)hp.m_blocks * kHeadM * sizeof(float4), 256));
    hp.merged = w.parts;
    hp.c_tau = (float)(1.4426950408889634 / (double)a->temperature);
    hp.seed = a->sample_seed; hp.step = a->step; hp.Ll = a->Ll; hp.pos0 = a->pos0; hp.row_pos0 = row_pos0;
  }
  HeadMaps maps;
  memset(&maps, 0, sizeof(maps));
  if (!head_tensor_map(&maps.h, h->hidden, (uint64_t)hp.rows, (uint64_t)h->d, (uint64_t)h->hidden_stride, (uint32_t)hp.a_box_rows))
    return FORK_ERR_INVALID_ARG;
  bool have[kHeadN / kHeadGroup] = {};
  for (int ns = 0; ns < splits; ++ns) {                                    /* the tile widths this launch uses (see the kernel) */
    const int g = head_split_groups(hp, ns), per = kHeadN / kHeadGroup, tiles = (g + per - 1) / per;
    for (int wg = g / tiles; wg <= g / tiles + (g % tiles ? 1 : 0); ++wg) {
      if (have[wg - 1]) continue;
      if (!head_tensor_map(&maps.w[wg - 1], h->weight, (uint64_t)a->V, (uint64_t)h->d, (uint64_t)h->weight_stride, (uint32_t)(wg * kHeadGroup)))
        return FORK_ERR_INVALID_ARG;
      have[wg - 1] = true;
    }
  }

  /* the active set (Algorithm 2, line 3): row list and per-sequence ranges for the select phase */
  SetupParams sp;
  memset(&sp, 0, sizeof(sp));
  sp.flags = a->mask; sp.lo = lo; sp.hi = hi;
  sp.B = a->B; sp.Lt = a->Lt; sp.pos0 = a->pos0; sp.Ll = a->Ll; sp.C = 1; sp.G = 1; sp.min_units = 1;
  sp.pos0_seq = row_pos0;
  sp.hdr = w.hdr; sp.seq_off = w.seq_off; sp.expected = w.expected; sp.ticket = w.ticket; sp.rows = w.rows;
  sp.n_unmasked = a->n_unmasked; sp.is_fallback = a->is_fallback; sp.fallback_pos = a->fallback_pos;
  sp.loop = loop; sp.step = a->step;
  if (launch(active_set_kernel, dim3(1), dim3(kSetupNT), st, pdl, sp) != cudaSuccess) return FORK_ERR_CUDA;

  /* logits tile by tile in tensor memory, reduced to one part per row and vocabulary split */
  {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)(hp.m_blocks * hp.n_splits)); cfg.blockDim = dim3(kHeadThreads);
    cfg.dynamicSmemBytes = head_smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (pdl) {
      attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[0].val.programmaticStreamSerializationAllowed = 1;
      cfg.attrs = attr; cfg.numAttrs = 1;
    }
    if ((drawn ? cudaLaunchKernelEx(&cfg, head_gemm_reduce_kernel<true>, maps, hp)
               : cudaLaunchKernelEx(&cfg, head_gemm_reduce_kernel<false>, maps, hp)) != cudaSuccess) return FORK_ERR_CUDA;
    g_launches.fetch_add(1);
  }

  /* the splits of a row merged (ties to the lowest column, like the slices of a vocabulary-parallel step) ... */
  if ((size_t)hp.m_blocks * kHeadM > (size_t)a->B * a->Lt + 2048) return FORK_ERR_WORKSPACE;
  {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)((hp.rows + kHeadMergeNT / 32 - 1) / (kHeadMergeNT / 32))); cfg.blockDim = dim3(kHeadMergeNT);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (pdl) {
      attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[0].val.programmaticStreamSerializationAllowed = 1;
      cfg.attrs = attr; cfg.numAttrs = 1;
    }
    if (cudaLaunchKernelEx(&cfg, head_merge_kernel, hp, w.parts) != cudaSuccess) return FORK_ERR_CUDA;
    g_launches.fetch_add(1);
    if (drawn) {                                             /* the chunk of every row, now that the rows' maxima are known */
      cfg.gridDim = dim3((unsigned)((hp.rows + 31) / 32)); cfg.blockDim = dim3(kHeadDrawNT);
      /* many short column ranges (few window rows): the range first, then its chunks; else all chunks in two passes */
      const bool by_ranges = hp.n_splits <= 256 && (hp.u_base + 1) * hp.unit <= kHeadDrawMaxRangeChunks;
      if ((by_ranges ? cudaLaunchKernelEx(&cfg, head_draw_ranges_kernel, hp)
                     : cudaLaunchKernelEx(&cfg, head_draw_kernel, hp)) != cudaSuccess) return FORK_ERR_CUDA;
      g_launches.fetch_add(1);
    }
  }
  /* ... then the unmask rule on one record per row */
  ReduceParams rp;
  memset(&rp, 0, sizeof(rp));
  rp.src.pos0 = a->pos0; rp.src.Ll = a->Ll; rp.src.V = a->V;
  rp.B = a->B; rp.Lt = a->Lt; rp.C = 1; rp.min_units = 1;
  rp.hdr = w.hdr; rp.seq_off = w.seq_off; rp.expected = w.expected; rp.ticket = w.ticket;
  rp.rows = w.rows; rp.final_rec = w.final_rec; rp.parts = w.parts;
  rp.tokens = a->tokens; rp.mask = a->mask; rp.threshold = a->threshold; rp.step = a->step;
  rp.conf = a->conf; rp.cand = a->cand; rp.entropy = a->entropy; rp.logp = a->logp; rp.row_status = a->row_status;
  rp.commit_step = a->commit_step; rp.commit_fallback = a->commit_fallback; rp.commit_logp = a->commit_logp;
  rp.n_unmasked = a->n_unmasked; rp.is_fallback = a->is_fallback; rp.fallback_pos = a->fallback_pos;
  rp.nfe = a->nfe; rp.n_fallback = a->n_fallback;
  rp.fallback_mode = a->fallback_mode; rp.fallback_rand = a->fallback_rand;
  rp.vp_parts_in = w.parts; rp.vp_ranks = 1; rp.vp_row_stride = hp.m_blocks * kHeadM;
  rp.vp_pos0_seq = row_pos0;
  rp.loop = loop; rp.blk_lo = lo; rp.blk_hi = hi;
  if (drawn) { rp.head_draw = hp.draw; rp.sample_seed = a->sample_seed; rp.noise_c = hp.c_tau; }
  const dim3 grid((unsigned)((a->B + kVpNT / 32 - 1) / (kVpNT / 32)));
  if ((drawn ? launch(vp_select_kernel<true>, grid, dim3(kVpNT), st, pdl, rp)
             : launch(vp_select_kernel<false>, grid, dim3(kVpNT), st, pdl, rp)) != cudaSuccess) return FORK_ERR_CUDA;
  return FORK_OK;
}

extern "C" fork_status fork_step_fused_head(const fork_step_args* a, const fork_head_args* h, void* ws, size_t ws_bytes,
                                            void* stream) {
  fork_status s = check_head_args(a, h, true);
  if (s != FORK_OK) return s;
  s = check_workspace(ws, ws_bytes, a->B, a->Lt);
  if (s != FORK_OK) return s;
  if (a->B == 0) return FORK_OK;
  return head_step_impl(a, h, a->blk_lo, a->blk_hi, h->row_pos0, ws, (cudaStream_t)stream, nullptr);
}

extern "C" fork_status fork_decode_loop_fused_head(const fork_step_args* proto, const fork_head_args* head, int32_t block_len,
                                                   int32_t gen_lo, int32_t gen_hi, fork_logits_fn provider, void* ctx,
                                                   int32_t max_steps, int32_t* steps_taken, void* ws, size_t ws_bytes,
                                                   void* stream) {
  if (steps_taken) *steps_taken = 0;
  fork_status s = check_head_args(proto, head, false);
  if (s != FORK_OK) return s;
  if (!provider || block_len <= 0 || block_len > proto->Ll || gen_lo < 0 || gen_hi > proto->Lt || gen_lo > gen_hi || max_steps < 0)
    return FORK_ERR_INVALID_ARG;
  s = check_workspace(ws, ws_bytes, proto->B, proto->Lt);
  if (s != FORK_OK) return s;
  if (proto->B == 0) return FORK_OK;
  cudaStream_t st = (cudaStream_t)stream;
  /* every sequence's window is its own block: row 0 of sequence b is position lo[b] of the step's cursors */
  return decode_loop_impl(proto, const_cast<void*>(head->hidden), block_len, gen_lo, gen_hi, provider, ctx, max_steps, steps_taken,
                          ws, stream, [&](const fork_step_args& a, const int32_t* lo, const int32_t* hi, LoopCtl* loop) {
                            return head_step_impl(&a, head, lo, hi, lo, ws, st, loop);
                          });
}

/* ---- host-buffer entry point --------------------------------------------------------------- */
struct StagingView {
  char* logits; int32_t* tokens; uint8_t* mask; int32_t* lo; int32_t* hi;
  float* conf; int32_t* cand; float* entropy; float* logp; uint32_t* row_status;
  int32_t* commit_step; uint8_t* commit_fallback; float* commit_logp;
  int32_t* n_unmasked; uint8_t* is_fallback; int32_t* fallback_pos; int32_t* nfe; int32_t* n_fallback;
  uint32_t* fallback_rand;
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
  v.fallback_rand = (uint32_t*)take(nb * 4);
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
  FORK_H2D(v.fallback_rand, h->fallback_rand, nb * 4);
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
  d.fallback_rand = h->fallback_rand ? v.fallback_rand : nullptr;
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

/* ---- read-only streaming probe ---------------------------------------------------------------- */
/* The rate at which this GPU delivers a buffer that is only read (128-bit streaming loads, a
   persistent grid, nothing computed but an XOR): the practical ceiling for the reduction kernels,
   which never write more than a few bytes per row.  The benchmark reports it beside the measured
   copy rate. */
__global__ void __launch_bounds__(256, 4) read_probe_kernel(const uint4* __restrict__ p, long long nvec, uint32_t* sink) {
  /* every CTA reads one contiguous share, like the reduction kernels */
  const long long per = (nvec + gridDim.x - 1) / gridDim.x;
  const long long lo = (long long)blockIdx.x * per, hi = (lo + per < nvec) ? lo + per : nvec;
  uint32_t x = 0;
  long long i = lo + threadIdx.x;
  for (; i + 3 * 256 < hi; i += 256 * 4) {
    uint4 v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = ld_stream(p + i + j * 256);
#pragma unroll
    for (int j = 0; j < 4; ++j) x ^= v[j].x ^ v[j].y ^ v[j].z ^ v[j].w;
  }
  for (; i < hi; i += 256) { const uint4 v = ld_stream(p + i); x ^= v.x ^ v.y ^ v.z ^ v.w; }
  if (x == 0x9e3779b9u) *sink = x;                           /* practically never: keeps the loads alive */
}

extern "C" fork_status fork_read_probe(const void* buffer, size_t bytes, void* sink4, void* stream) {
  if (!buffer || !sink4 || (reinterpret_cast<uintptr_t>(buffer) & 15u) != 0) return FORK_ERR_INVALID_ARG;
  DeviceInfo* dev;
  if (!device_info(&dev)) return FORK_ERR_CUDA;
  read_probe_kernel<<<dev->sms * 4, 256, 0, (cudaStream_t)stream>>>((const uint4*)buffer, (long long)(bytes / 16), (uint32_t*)sink4);
  if (cudaGetLastError() != cudaSuccess) return FORK_ERR_CUDA;
  g_launches.fetch_add(1);
  return FORK_OK;
}

/* ---- host-side view of the partition, for tests ------------------------------------------- */
extern "C" int64_t fork_debug_part_begin(int64_t U, int32_t G, int32_t g) { return fork_part_begin(U, G, g); }
extern "C" int32_t fork_debug_part_owner(int64_t U, int32_t G, int64_t x) { return fork_part_owner(U, G, x); }
extern "C" int32_t fork_debug_row_parts(int64_t U, int32_t G, int32_t C, int64_t r) { return fork_row_parts(U, G, C, r); }
extern "C" int32_t fork_debug_chunk(void) { return FORK_CHUNK; }
extern "C" int32_t fork_debug_effective_grid(int64_t U, int32_t G, int32_t min_units) { return fork_effective_grid(U, G, min_units); }
