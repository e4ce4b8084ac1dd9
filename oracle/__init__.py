"""fp64 CPU oracle for the Fork-dLLM sampling step -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
The product package never does, and this package never imports the product package.

It is a ctypes wrapper around ``fork_oracle.c`` (plain C, fp64), which states Algorithm 2
(Fork-dLLM), the softmax confidence / entropy / log-probability definitions of Section 2 and
Section 3.2, and the semi-autoregressive loop of Section 4.1 (Setup) as directly as possible.

Arrays are numpy: bf16 logits are ``uint16`` bit patterns, fp32 logits are ``float32``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fork_oracle.c")
_LIB = os.path.join(_HERE, "libfork_oracle.so")

BF16, F32 = 0, 1
OK, ERR_ARG, ERR_MAX_STEPS, ERR_PROVIDER = 0, -1, -4, -5
ROW_BAD, ROW_BAD_TOKEN = 1, 2
FB_LEFTMOST, FB_MAX_CONF, FB_MIN_CONF, FB_MAX_ENTROPY, FB_RANDOM = 0, 1, 2, 3, 4


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-pthread",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _StepArgs(C.Structure):
    _fields_ = [
        ("logits", C.c_void_p), ("stride_b", C.c_int64), ("stride_l", C.c_int64), ("pos0", C.c_int32),
        ("B", C.c_int32), ("Lt", C.c_int32), ("Ll", C.c_int32), ("V", C.c_int32), ("dtype", C.c_int32),
        ("tokens", C.c_void_p), ("mask", C.c_void_p), ("blk_lo", C.c_void_p), ("blk_hi", C.c_void_p),
        ("threshold", C.c_float), ("step", C.c_int32),
        ("conf", C.c_void_p), ("cand", C.c_void_p), ("entropy", C.c_void_p), ("logp", C.c_void_p),
        ("commit_step", C.c_void_p), ("commit_fallback", C.c_void_p), ("commit_logp", C.c_void_p),
        ("n_unmasked", C.c_void_p), ("is_fallback", C.c_void_p), ("fallback_pos", C.c_void_p),
        ("nfe", C.c_void_p), ("n_fallback", C.c_void_p),
        ("row_status", C.c_void_p),
        ("nthreads", C.c_int32),
        ("fallback_mode", C.c_int32), ("fallback_rand", C.c_void_p),
        ("temperature", C.c_float), ("sample_seed", C.c_uint64),
        ("fallback_margin", C.c_void_p), ("sample_margin", C.c_void_p),
        ("slice_off", C.c_void_p), ("n_slices", C.c_int32),
    ]


_PROVIDER = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                        C.c_void_p)

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.fork_oracle_row_stats.restype = None
        L.fork_oracle_row_stats.argtypes = [C.c_void_p, C.c_int32, C.c_int32] + [C.c_void_p] * 8
        L.fork_oracle_row_logp.restype = C.c_double
        L.fork_oracle_row_logp.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
        L.fork_oracle_step.restype = C.c_int
        L.fork_oracle_step.argtypes = [C.POINTER(_StepArgs)]
        L.fork_oracle_logprob.restype = C.c_int
        L.fork_oracle_logprob.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int32, C.c_int32, C.c_int32,
                                          C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32]
        L.fork_oracle_block_cursors.restype = None
        L.fork_oracle_block_cursors.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                                C.c_int32, C.c_void_p, C.c_void_p]
        L.fork_oracle_decode_loop.restype = C.c_int
        L.fork_oracle_decode_loop.argtypes = [C.POINTER(_StepArgs), C.c_int32, C.c_int32, C.c_int32,
                                              _PROVIDER, C.c_void_p, C.c_int32, C.c_void_p]
        L.fork_oracle_threads_used.restype = C.c_int
        L.fork_oracle_threads_used.argtypes = [C.c_int32, C.c_int64]
        L.fork_oracle_noise.restype = None
        L.fork_oracle_noise.argtypes = [C.c_uint64, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        L.fork_oracle_select_top_entropy.restype = C.c_int
        L.fork_oracle_select_top_entropy.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_float,
                                                     C.c_void_p, C.c_void_p]
        L.fork_oracle_grpo_loss.restype = C.c_int
        L.fork_oracle_grpo_loss.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.c_float, C.c_float] + [C.c_void_p] * 6
        L.fork_oracle_row_logp_grad.restype = C.c_int
        L.fork_oracle_row_logp_grad.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_double, C.c_void_p]
        L.fork_oracle_row_lse.restype = C.c_double
        L.fork_oracle_row_lse.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
        _lib = L
    return _lib


def _dtype_of(a: np.ndarray) -> int:
    if a.dtype == np.uint16:
        return BF16
    if a.dtype == np.float32:
        return F32
    raise TypeError("logits must be uint16 (bf16 bits) or float32, got %s" % a.dtype)


def _ptr(a):
    return None if a is None else a.ctypes.data


def threads_used(nthreads: int, n_rows: int) -> int:
    return int(lib().fork_oracle_threads_used(nthreads, n_rows))


def row_stats(row: np.ndarray) -> dict:
    """conf, cand, entropy, logp of the candidate, and (m, s, t) for one contiguous logits row."""
    row = np.ascontiguousarray(row)
    conf, ent, lp, m, s, t = (C.c_double() for _ in range(6))
    cand, st = C.c_int32(), C.c_uint32()
    lib().fork_oracle_row_stats(row.ctypes.data, row.shape[0], _dtype_of(row),
                                C.addressof(conf), C.addressof(cand), C.addressof(ent), C.addressof(lp),
                                C.addressof(m), C.addressof(s), C.addressof(t), C.addressof(st))
    return dict(conf=conf.value, cand=cand.value, entropy=ent.value, logp=lp.value,
                m=m.value, s=s.value, t=t.value, status=st.value)


def row_logp(row: np.ndarray, tok: int):
    row = np.ascontiguousarray(row)
    st = C.c_uint32()
    v = lib().fork_oracle_row_logp(row.ctypes.data, row.shape[0], _dtype_of(row), int(tok), C.addressof(st))
    return float(v), int(st.value)


class StepState:
    """Host buffers of one batch: the sequence, its mask, and every output of the step."""

    def __init__(self, B: int, Lt: int, tokens=None, mask=None):
        self.B, self.Lt = B, Lt
        self.tokens = np.zeros((B, Lt), np.int32) if tokens is None else np.ascontiguousarray(tokens, np.int32).copy()
        self.mask = np.ones((B, Lt), np.uint8) if mask is None else np.ascontiguousarray(mask, np.uint8).copy()
        self.conf = np.full((B, Lt), np.nan, np.float64)
        self.cand = np.full((B, Lt), -1, np.int32)
        self.entropy = np.full((B, Lt), np.nan, np.float64)
        self.logp = np.full((B, Lt), np.nan, np.float64)
        self.commit_step = np.full((B, Lt), -1, np.int32)
        self.commit_fallback = np.full((B, Lt), 255, np.uint8)
        self.commit_logp = np.full((B, Lt), np.nan, np.float64)
        self.n_unmasked = np.zeros(B, np.int32)
        self.is_fallback = np.zeros(B, np.uint8)
        self.fallback_pos = np.full(B, -1, np.int32)
        self.nfe = np.zeros(B, np.int32)
        self.n_fallback = np.zeros(B, np.int32)
        self.row_status = np.zeros((B, Lt), np.uint32)
        self.fallback_margin = np.full(B, np.inf, np.float64)
        self.sample_margin = np.full((B, Lt), np.inf, np.float64)


def _fill_args(st: StepState, logits: np.ndarray, lo, hi, threshold, step, pos0, nthreads,
               fallback_mode=FB_LEFTMOST, fallback_rand=None, temperature=0.0, sample_seed=0, slices=None) -> _StepArgs:
    assert logits.ndim == 3 and logits.flags.c_contiguous
    B, Ll, V = logits.shape
    assert B == st.B
    a = _StepArgs()
    a.logits = logits.ctypes.data
    a.stride_b, a.stride_l, a.pos0 = Ll * V, V, pos0
    a.B, a.Lt, a.Ll, a.V, a.dtype = B, st.Lt, Ll, V, _dtype_of(logits)
    a.tokens, a.mask = st.tokens.ctypes.data, st.mask.ctypes.data
    a.blk_lo, a.blk_hi = _ptr(lo), _ptr(hi)
    a.threshold, a.step = float(threshold), int(step)
    a.conf, a.cand, a.entropy, a.logp = (x.ctypes.data for x in (st.conf, st.cand, st.entropy, st.logp))
    a.commit_step, a.commit_fallback, a.commit_logp = (x.ctypes.data for x in
                                                        (st.commit_step, st.commit_fallback, st.commit_logp))
    a.n_unmasked, a.is_fallback, a.fallback_pos = (x.ctypes.data for x in
                                                   (st.n_unmasked, st.is_fallback, st.fallback_pos))
    a.nfe, a.n_fallback = st.nfe.ctypes.data, st.n_fallback.ctypes.data
    a.row_status = st.row_status.ctypes.data
    a.nthreads = nthreads
    a.fallback_mode = int(fallback_mode)
    a.fallback_rand = _ptr(fallback_rand)
    a.temperature = float(temperature)
    a.sample_seed = int(sample_seed)
    a.fallback_margin = st.fallback_margin.ctypes.data
    a.sample_margin = st.sample_margin.ctypes.data
    if slices is not None:                           # vocabulary cut into slices [off[r], off[r+1]): kept alive by the caller
        a.slice_off, a.n_slices = slices.ctypes.data, len(slices) - 1
    return a


def step(st: StepState, logits: np.ndarray, lo: np.ndarray, hi: np.ndarray, threshold: float,
         step_id: int = 0, pos0: int = 0, nthreads: int = 0, fallback_mode: int = FB_LEFTMOST,
         fallback_rand=None, temperature: float = 0.0, sample_seed: int = 0, slices=None) -> int:
    """One sampling step on host buffers; ``st`` is updated in place.  The defaults give Fork-dLLM
    (Algorithm 2) with arg-max candidates; ``fallback_mode`` selects Fast-dLLM's order (Algorithm 1)
    or an ablation order, ``temperature`` > 0 draws the candidates (uniform stream ``sample_seed``;
    ``slices`` = ascending offsets [0, ..., V] when the vocabulary is sharded, which fixes the order
    in which the draw visits it)."""
    if slices is not None:
        slices = np.ascontiguousarray(slices, np.int32)
    lo = np.ascontiguousarray(lo, np.int32)
    hi = np.ascontiguousarray(hi, np.int32)
    if fallback_rand is not None:
        fallback_rand = np.ascontiguousarray(fallback_rand, np.uint32)
    a = _fill_args(st, logits, lo, hi, threshold, step_id, pos0, nthreads, fallback_mode, fallback_rand,
                   temperature, sample_seed, slices)
    return int(lib().fork_oracle_step(C.byref(a)))


def logprob(logits: np.ndarray, tokens: np.ndarray, select: np.ndarray, pos0: int = 0, nthreads: int = 0):
    """Per-token log-likelihood at selected positions and its per-sequence sum (Section 3.2)."""
    assert logits.ndim == 3 and logits.flags.c_contiguous
    B, Ll, V = logits.shape
    tokens = np.ascontiguousarray(tokens, np.int32)
    select = np.ascontiguousarray(select, np.uint8)
    Lt = tokens.shape[1]
    lp = np.zeros((B, Lt), np.float64)
    ssum = np.zeros(B, np.float64)
    scnt = np.zeros(B, np.int32)
    status = np.zeros((B, Lt), np.uint32)
    rc = lib().fork_oracle_logprob(logits.ctypes.data, Ll * V, V, pos0, B, Lt, Ll, V, _dtype_of(logits),
                                   tokens.ctypes.data, select.ctypes.data, lp.ctypes.data, ssum.ctypes.data,
                                   scnt.ctypes.data, status.ctypes.data, nthreads)
    return int(rc), lp, ssum, scnt, status


def block_cursors(mask: np.ndarray, gen_lo: int, gen_hi: int, block_len: int, lo=None, hi=None):
    mask = np.ascontiguousarray(mask, np.uint8)
    B, Lt = mask.shape
    if lo is None:
        lo = np.full(B, gen_lo, np.int32)
        hi = np.full(B, gen_lo, np.int32)
    lib().fork_oracle_block_cursors(mask.ctypes.data, B, Lt, gen_lo, gen_hi, block_len,
                                    lo.ctypes.data, hi.ctypes.data)
    return lo, hi


def decode_loop(st: StepState, logits: np.ndarray, block_len: int, gen_lo: int, gen_hi: int, provider,
                threshold: float, max_steps: int, step0: int = 0, pos0: int = 0, nthreads: int = 0,
                fallback_mode: int = FB_LEFTMOST, fallback_rand=None, temperature: float = 0.0,
                sample_seed: int = 0):
    """Run the semi-autoregressive loop.  ``provider(step, tokens, mask, lo, hi, logits)`` fills
    ``logits`` (numpy views of the live host buffers) and returns 0, or non-zero to abort."""
    B, Lt = st.B, st.Lt

    def _cb(_ctx, step_id, _tok, _mask, lo_p, hi_p, _out):
        lo = np.ctypeslib.as_array(C.cast(lo_p, C.POINTER(C.c_int32)), shape=(B,))
        hi = np.ctypeslib.as_array(C.cast(hi_p, C.POINTER(C.c_int32)), shape=(B,))
        try:
            return int(provider(int(step_id), st.tokens, st.mask, lo, hi, logits) or 0)
        except Exception:  # a Python error must not unwind through C
            import traceback
            traceback.print_exc()
            return 1

    a = _fill_args(st, logits, None, None, threshold, step0, pos0, nthreads, fallback_mode, fallback_rand,
                   temperature, sample_seed)
    steps = C.c_int32(0)
    rc = lib().fork_oracle_decode_loop(C.byref(a), block_len, gen_lo, gen_hi, _PROVIDER(_cb), None,
                                       max_steps, C.addressof(steps))
    return int(rc), int(steps.value)


def noise(seed: int, step_id: int, b: int, k: int):
    """(u_token, u_slice): the two uniform variates of row (step, b, k) that draw its candidate."""
    u, g = C.c_double(), C.c_double()
    lib().fork_oracle_noise(int(seed), step_id, b, k, C.addressof(u), C.addressof(g))
    return u.value, g.value


def select_top_entropy(entropy: np.ndarray, eligible: np.ndarray, ratio: float):
    """JustGRPO-Fast's selection: per rollout the floor(ratio*n) eligible positions of highest entropy."""
    entropy = np.ascontiguousarray(entropy, np.float32)
    eligible = np.ascontiguousarray(eligible, np.uint8)
    B, Lt = entropy.shape
    select = np.zeros((B, Lt), np.uint8)
    cnt = np.zeros(B, np.int32)
    rc = lib().fork_oracle_select_top_entropy(entropy.ctypes.data, eligible.ctypes.data, B, Lt, float(ratio),
                                              select.ctypes.data, cnt.ctypes.data)
    return int(rc), select, cnt


def grpo_loss(logp_new: np.ndarray, logp_old: np.ndarray, select: np.ndarray, reward: np.ndarray, group: int,
              eps_lo: float, eps_hi: float) -> dict:
    """The ForkGRPO objective (Eq. 2) and its derivative with respect to logp_new."""
    logp_new = np.ascontiguousarray(logp_new, np.float32)
    logp_old = np.ascontiguousarray(logp_old, np.float32)
    select = np.ascontiguousarray(select, np.uint8)
    reward = np.ascontiguousarray(reward, np.float32)
    B, Lt = logp_new.shape
    adv = np.zeros(B, np.float64)
    ratio = np.zeros((B, Lt), np.float64)
    seq_obj = np.zeros(B, np.float64)
    obj = np.zeros(1, np.float64)
    dlogp = np.zeros((B, Lt), np.float64)
    skipped = np.zeros(max(B // max(group, 1), 1), np.uint8)
    rc = lib().fork_oracle_grpo_loss(B, Lt, group, logp_new.ctypes.data, logp_old.ctypes.data, select.ctypes.data,
                                     reward.ctypes.data, float(eps_lo), float(eps_hi), adv.ctypes.data,
                                     ratio.ctypes.data, seq_obj.ctypes.data, obj.ctypes.data, dlogp.ctypes.data,
                                     skipped.ctypes.data)
    return dict(rc=int(rc), adv=adv, ratio=ratio, seq_obj=seq_obj, objective=float(obj[0]), dlogp=dlogp,
                skipped=skipped)


def row_logp_grad(row: np.ndarray, tok: int, w: float = 1.0) -> np.ndarray:
    """d(w * log q(tok))/d logits of one row."""
    row = np.ascontiguousarray(row)
    g = np.zeros(row.shape[0], np.float64)
    rc = lib().fork_oracle_row_logp_grad(row.ctypes.data, row.shape[0], _dtype_of(row), int(tok), float(w),
                                         g.ctypes.data)
    if rc != 0:
        raise ValueError("row_logp_grad: bad arguments")
    return g


def row_lse(row: np.ndarray) -> float:
    row = np.ascontiguousarray(row)
    return float(lib().fork_oracle_row_lse(row.ctypes.data, row.shape[0], _dtype_of(row)))


def head_logits(hidden_bits: np.ndarray, weight_bits: np.ndarray) -> np.ndarray:
    """Logits of the LM head for the fused step (Section 2: the model's distribution at a position
    is the soft-max of hidden state times output embedding): ``logits[i, v] = <hidden[i], weight[v]>``
    with the bf16 inputs (``uint16`` bit patterns, [n, d] and [V, d]) widened exactly to fp64, the
    products summed in fp64 (a library matrix product), and the result rounded ONCE to fp32 -- the
    fused path's logits are its fp32 accumulators, never rounded to bf16."""
    h = (np.ascontiguousarray(hidden_bits, np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    out = np.empty((h.shape[0], weight_bits.shape[0]), np.float32)
    step = 8192                                    # weight rows per slab: bounds the fp64 copy of the weight
    for v0 in range(0, weight_bits.shape[0], step):
        w = (np.ascontiguousarray(weight_bits[v0:v0 + step], np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        out[:, v0:v0 + step] = (h @ w.T).astype(np.float32)
    return out
