"""Seeded synthetic logits for the Fork-dLLM confidence pass (input making only).

The generator is counter based: every logit is a pure function of (seed, nonce, step, b, l, v),
and the host build (gcc) and the device build (nvcc) of the same inline core give bit-identical
rows.  This package contains none of the sampler's arithmetic; it serves both the CPU oracle's
tests and the CUDA path's tests / benchmark with the same inputs.

Workload recipes (``workload(name)``) follow the five benchmark configurations: shapes, dtypes,
background std, peak-height distributions and fork-row fractions.  In the "calibrated" variant a
peak of height h is SET to ``ln V + sigma^2/2 - 1.4 + h`` so that h is measured from the row's
background log-sum-exp (a position then clears threshold 0.9 when h is above about 3.6); the
"literal" variant ADDS h to the background draw, which almost never clears the threshold and so
degenerates to left-to-right decoding.
"""
from __future__ import annotations

import ctypes as C
import math
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_HERE, "csrc")
_CPU_LIB = os.path.join(_HERE, "libfork_synth_cpu.so")
_CUDA_LIB = os.path.join(_HERE, "libfork_synth_cuda.so")

BF16, F32 = 0, 1
PEAK_ADD, PEAK_SET = 0, 1


class Cfg(C.Structure):
    _fields_ = [("seed", C.c_uint64), ("B", C.c_int32), ("Lt", C.c_int32), ("V", C.c_int32),
                ("dtype", C.c_int32), ("sigma", C.c_float), ("peak_mode", C.c_int32),
                ("peak_base", C.c_float), ("peak_prob", C.c_float), ("h_lo", C.c_float),
                ("h_span", C.c_float), ("fork_prob", C.c_float), ("fork_h", C.c_float),
                ("fork_gap", C.c_float)]


class RowPlan(C.Structure):
    _fields_ = [("n_planted", C.c_int32), ("is_fork", C.c_int32), ("tok", C.c_int32 * 4),
                ("val", C.c_float * 4)]


def _stale(out, srcs):
    return (not os.path.exists(out)) or any(os.path.getmtime(out) < os.path.getmtime(s) for s in srcs)


def build_cpu(force=False) -> str:
    srcs = [os.path.join(_CSRC, "fork_synth_cpu.c"), os.path.join(_CSRC, "fork_synth.h")]
    if force or _stale(_CPU_LIB, srcs):
        tmp = _CPU_LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=gnu11", "-ffp-contract=off", "-fPIC", "-shared", "-pthread",
                               "-o", tmp, srcs[0], "-lm"])
        os.replace(tmp, _CPU_LIB)
    return _CPU_LIB


def build_cuda(force=False) -> str:
    srcs = [os.path.join(_CSRC, "fork_synth_cuda.cu"), os.path.join(_CSRC, "fork_synth.h")]
    if force or _stale(_CUDA_LIB, srcs):
        tmp = _CUDA_LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["nvcc", "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a",
                               "-lineinfo", "-fmad=false", "-Xcompiler", "-fPIC", "-shared",
                               "-o", tmp, srcs[0]])
        os.replace(tmp, _CUDA_LIB)
    return _CUDA_LIB


_cpu = None
_cuda = None


def cpu():
    global _cpu
    if _cpu is None:
        L = C.CDLL(build_cpu())
        L.fork_synth_tables.restype = None
        L.fork_synth_tables.argtypes = [C.c_void_p, C.c_void_p]
        L.fork_synth_row_host.restype = None
        L.fork_synth_row_host.argtypes = [C.POINTER(Cfg), C.c_uint32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
        L.fork_synth_fill_host.restype = C.c_int64
        L.fork_synth_fill_host.argtypes = [C.POINTER(Cfg), C.c_uint32, C.c_int32, C.c_void_p, C.c_void_p,
                                           C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int32, C.c_int32,
                                           C.c_int32]
        L.fork_synth_plan_host.restype = None
        L.fork_synth_plan_host.argtypes = [C.POINTER(Cfg), C.c_int32, C.c_int32, C.POINTER(RowPlan)]
        _cpu = L
    return _cpu


def cuda():
    """The device-side generator (needs a GPU to run, not to load)."""
    global _cuda
    if _cuda is None:
        L = C.CDLL(build_cuda())
        L.fork_synth_cuda_init.restype = C.c_int
        L.fork_synth_cuda_init.argtypes = [C.c_void_p, C.c_void_p]
        L.fork_synth_cuda_fill.restype = C.c_int
        L.fork_synth_cuda_fill.argtypes = [C.POINTER(Cfg), C.c_uint32, C.c_int32, C.c_void_p, C.c_void_p,
                                           C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int32, C.c_int32,
                                           C.c_void_p]
        L.fork_synth_cuda_canary.restype = C.c_int
        L.fork_synth_cuda_canary.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_void_p]
        L.fork_synth_provider_create.restype = C.c_void_p
        L.fork_synth_provider_create.argtypes = [C.POINTER(Cfg), C.c_int64, C.c_int64, C.c_int32, C.c_int32,
                                                 C.c_void_p, C.c_int32]
        L.fork_synth_provider_destroy.restype = None
        L.fork_synth_provider_destroy.argtypes = [C.c_void_p]
        L.fork_synth_provider_calls.restype = C.c_int64
        L.fork_synth_provider_calls.argtypes = [C.c_void_p]
        L.fork_synth_provider_fail_at.restype = None
        L.fork_synth_provider_fail_at.argtypes = [C.c_void_p, C.c_int32]
        tm, tt = C.c_void_p(), C.c_void_p()
        cpu().fork_synth_tables(C.byref(tm), C.byref(tt))
        L._tables = (tm, tt)
        _cuda = L
    return _cuda


def provider_address() -> int:
    """Address of the C callback `fork_synth_provider` (has the decode loop's fork_logits_fn signature)."""
    return C.cast(cuda().fork_synth_provider, C.c_void_p).value


class Provider:
    """Owns a generator context for the decode loop: `address` + `ctx` go to fork_decode_loop."""

    def __init__(self, cfg: Cfg, stride_b: int, stride_l: int, pos0: int, Ll: int, nonce=None):
        L = cuda_init()
        arr = None if nonce is None else np.ascontiguousarray(nonce, np.uint32)
        self._L = L
        self.ctx = L.fork_synth_provider_create(C.byref(cfg), stride_b, stride_l, pos0, Ll,
                                                None if arr is None else arr.ctypes.data,
                                                0 if arr is None else len(arr))
        self.address = provider_address()

    @property
    def calls(self) -> int:
        return int(self._L.fork_synth_provider_calls(self.ctx))

    def fail_at(self, step: int):
        self._L.fork_synth_provider_fail_at(self.ctx, step)

    def close(self):
        if self.ctx:
            self._L.fork_synth_provider_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def cuda_fill(cfg: Cfg, step: int, mask_ptr: int, lo_ptr, hi_ptr, logits_ptr: int, stride_b: int, stride_l: int,
              pos0: int, Ll: int, stream_ptr: int = 0, nonce: int = 0):
    """Enqueue the fill of every live row of a device logits buffer (raw device pointers)."""
    rc = cuda_init().fork_synth_cuda_fill(C.byref(cfg), nonce, step, mask_ptr, lo_ptr, hi_ptr, logits_ptr,
                                          stride_b, stride_l, pos0, Ll, stream_ptr)
    if rc != 0:
        raise RuntimeError("fork_synth_cuda_fill: CUDA error %d" % rc)


def cuda_canary(logits_ptr: int, n_elems: int, dtype: int, stream_ptr: int = 0):
    rc = cuda().fork_synth_cuda_canary(logits_ptr, n_elems, dtype, stream_ptr)
    if rc != 0:
        raise RuntimeError("fork_synth_cuda_canary: CUDA error %d" % rc)


def cuda_init():
    """Upload the host-built quantile tables to the current device (once per process and device)."""
    L = cuda()
    rc = L.fork_synth_cuda_init(L._tables[0], L._tables[1])
    if rc != 0:
        raise RuntimeError("fork_synth_cuda_init failed with CUDA error %d" % rc)
    return L


# ------------------------------------------------------------------------------------------------
@dataclass
class Workload:
    """One benchmark configuration: shapes, sampler settings and the generator's parameters."""
    name: str
    B: int
    Lt: int
    block_len: int
    V: int
    dtype: int
    sigma: float
    threshold: float
    seed: int
    peak_mode: int = PEAK_SET
    peak_prob: float = 1.0
    h_lo: float = 0.0
    h_hi: float = 0.0
    fork_prob: float = 0.0
    fork_h: float = 6.0
    fork_gap: float = 0.1
    thresholds: tuple = field(default_factory=tuple)
    select_prob: float = 0.0       # ForkGRPO scoring: density of the fallback-step mask
    off_peak_prob: float = 0.0     # ForkGRPO scoring: P(sampled token is not the row's peak token)

    @property
    def es(self) -> int:
        return 2 if self.dtype == BF16 else 4

    @property
    def np_dtype(self):
        return np.uint16 if self.dtype == BF16 else np.float32

    def peak_base(self) -> float:
        if self.peak_mode == PEAK_ADD:
            return 0.0
        return float(np.float32(math.log(self.V) + 0.5 * self.sigma * self.sigma - 1.4))

    def cfg(self, B=None) -> Cfg:
        c = Cfg()
        c.seed = self.seed
        c.B, c.Lt, c.V, c.dtype = (self.B if B is None else B), self.Lt, self.V, self.dtype
        c.sigma, c.peak_mode, c.peak_base = self.sigma, self.peak_mode, self.peak_base()
        c.peak_prob, c.h_lo, c.h_span = self.peak_prob, self.h_lo, float(np.float32(self.h_hi - self.h_lo))
        c.fork_prob, c.fork_h, c.fork_gap = self.fork_prob, self.fork_h, self.fork_gap
        return c

    def literal(self) -> "Workload":
        """The configuration read literally: the peak height is added to the background draw."""
        from dataclasses import replace
        return replace(self, name=self.name + "-literal", peak_mode=PEAK_ADD)


def workload(name: str) -> Workload:
    """The five benchmark configurations ("calibrated" variant)."""
    if name == "tiny":       # B=1, one block of 32, V=1024, fp32, N(0,2^2), 25% peaks of height 8
        return Workload("tiny", B=1, Lt=32, block_len=32, V=1024, dtype=F32, sigma=2.0, threshold=0.9,
                        seed=0x39859_0001, peak_prob=0.25, h_lo=8.0, h_hi=8.0)
    if name == "b8":         # B=8, 256 = 8 blocks of 32, V=126464 bf16, N(0,3^2), every row a peak h~U(0,12)
        return Workload("b8", B=8, Lt=256, block_len=32, V=126464, dtype=BF16, sigma=3.0, threshold=0.9,
                        seed=0x39859_0002, peak_prob=1.0, h_lo=0.0, h_hi=12.0)
    if name == "passk":      # B=64 rollouts; 10% fork rows with 2..4 near-equal tops, the rest peaked (+10)
        return Workload("passk", B=64, Lt=256, block_len=32, V=126464, dtype=BF16, sigma=3.0, threshold=0.9,
                        seed=0x39859_0003, peak_prob=0.9, h_lo=10.0, h_hi=10.0, fork_prob=0.1, fork_h=6.0)
    if name == "grpo":       # 16 prompts x 8 rollouts, fp32, log-likelihood at ~20% of positions
        return Workload("grpo", B=128, Lt=256, block_len=32, V=126464, dtype=F32, sigma=3.0, threshold=0.9,
                        seed=0x39859_0004, peak_prob=1.0, h_lo=0.0, h_hi=12.0, select_prob=0.2,
                        off_peak_prob=0.2)
    if name == "sweep":      # B=32, 1024 = 16 blocks of 64, V=152064 bf16, h~U(0,14), five thresholds
        return Workload("sweep", B=32, Lt=1024, block_len=64, V=152064, dtype=BF16, sigma=3.0, threshold=0.9,
                        seed=0x39859_0005, peak_prob=1.0, h_lo=0.0, h_hi=14.0,
                        thresholds=(0.5, 0.7, 0.9, 0.95, 0.99))
    raise KeyError(name)


WORKLOADS = ("tiny", "b8", "passk", "grpo", "sweep")


# ------------------------------------------------------------------------------------------------
def row_host(cfg: Cfg, step: int, b: int, l: int, nonce: int = 0) -> np.ndarray:
    out = np.empty(cfg.V, np.uint16 if cfg.dtype == BF16 else np.float32)
    cpu().fork_synth_row_host(C.byref(cfg), nonce, step, b, l, out.ctypes.data)
    return out


def plan_host(cfg: Cfg, b: int, l: int) -> dict:
    p = RowPlan()
    cpu().fork_synth_plan_host(C.byref(cfg), b, l, C.byref(p))
    n = p.n_planted
    return dict(n_planted=n, is_fork=bool(p.is_fork), tok=list(p.tok)[:n], val=list(p.val)[:n])


def fill_host(cfg: Cfg, step: int, mask: np.ndarray, lo: np.ndarray, hi: np.ndarray, logits: np.ndarray,
              pos0: int = 0, nonce: int = 0, nthreads: int = 0) -> int:
    """Write every live row of ``logits`` ([B, Ll, V], C-contiguous) in host memory."""
    B, Ll, V = logits.shape
    assert B == cfg.B and V == cfg.V and logits.flags.c_contiguous
    mask = np.ascontiguousarray(mask, np.uint8)
    lo = np.ascontiguousarray(lo, np.int32)
    hi = np.ascontiguousarray(hi, np.int32)
    return int(cpu().fork_synth_fill_host(C.byref(cfg), nonce, step, mask.ctypes.data, lo.ctypes.data,
                                          hi.ctypes.data, logits.ctypes.data, Ll * V, V, pos0, Ll, nthreads))


def canary_host(logits: np.ndarray):
    """Fill a host logits buffer with NaN so that any read of a row that is not live shows up."""
    if logits.dtype == np.uint16:
        logits[...] = 0x7FC0
    else:
        logits[...] = np.nan


def bf16_bits_to_f32(a: np.ndarray) -> np.ndarray:
    return (a.astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even conversion of finite float32 values to bf16 bit patterns."""
    u = np.ascontiguousarray(a, np.float32).view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return (u >> 16).astype(np.uint16)


def scoring_inputs(w: Workload, cfg: Cfg):
    """Tokens and fallback-step mask for the ForkGRPO scoring workload: the sampled token is the
    row's planted peak with probability 1-off_peak_prob, else a uniform token; positions are
    selected with probability select_prob.  Pure integer hashing of (seed, b, l)."""
    B, Lt, V = cfg.B, cfg.Lt, cfg.V
    rng = np.random.Generator(np.random.PCG64(w.seed ^ 0xF0F0))
    select = (rng.random((B, Lt)) < w.select_prob).astype(np.uint8)
    off = rng.random((B, Lt)) < w.off_peak_prob
    uni = rng.integers(0, V, size=(B, Lt), dtype=np.int64)
    tokens = np.empty((B, Lt), np.int32)
    for b in range(B):
        for l in range(Lt):
            p = plan_host(cfg, b, l)
            tokens[b, l] = uni[b, l] if (off[b, l] or p["n_planted"] == 0) else p["tok"][0]
    return tokens, select


def head_weight(V: int, d: int, seed: int) -> np.ndarray:
    """A seeded stand-in for an LM-head weight [V, d] (bf16 bit patterns): independent N(0,1) entries."""
    rng = np.random.Generator(np.random.PCG64(seed))
    out = np.empty((V, d), np.uint16)
    step = 8192
    for v0 in range(0, V, step):
        out[v0:v0 + step] = f32_to_bf16_bits(rng.standard_normal((min(step, V - v0), d), dtype=np.float32))
    return out


def head_hidden(weight_bits: np.ndarray, n_rows: int, seed: int, sigma: float = 3.0, h_lo: float = 0.0, h_hi: float = 12.0):
    """Seeded hidden states [n_rows, d] (bf16 bit patterns) whose logits under `weight_bits` look like
    the calibrated workloads: a N(0, sigma^2) background (hidden = sigma / sqrt(d) * noise), plus, on
    a random token per row, a peak of height ln V + sigma^2/2 - 1.4 + h, h ~ U(h_lo, h_hi) (hidden +=
    height / d * weight[token]: the token's own logit rises by about `height`, the others hardly).
    Returns (hidden_bits, tokens)."""
    V, d = weight_bits.shape
    rng = np.random.Generator(np.random.PCG64(seed))
    hid = rng.standard_normal((n_rows, d), dtype=np.float32) * np.float32(sigma / math.sqrt(d))
    tok = rng.integers(0, V, size=n_rows)
    height = (math.log(V) + 0.5 * sigma * sigma - 1.4 + rng.uniform(h_lo, h_hi, size=n_rows)).astype(np.float32)
    hid += (height / np.float32(d))[:, None] * bf16_bits_to_f32(weight_bits[tok])
    return f32_to_bf16_bits(hid), tok.astype(np.int64)
