"""Thin ctypes binding of libfork_dllm.so: argument marshalling only.

Every function here has the name and the meaning of the C entry point it forwards to
(see include/fork_dllm.h); all computation happens in the CUDA kernels behind them.  PyTorch is
used for device memory and streams.  There is no CPU fallback: if the library cannot be loaded
the import fails.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import _build

FORK_OK, FORK_ERR_INVALID_ARG, FORK_ERR_CUDA, FORK_ERR_WORKSPACE, FORK_ERR_MAX_STEPS, FORK_ERR_PROVIDER = \
    0, -1, -2, -3, -4, -5
FORK_BF16, FORK_F32 = 0, 1
FORK_ROW_NONFINITE, FORK_ROW_BAD_TOKEN = 1, 2
FORK_DEV_WINDOW_CLAMPED, FORK_DEV_TIMEOUT = 1, 2
FORK_FALLBACK_LEFTMOST, FORK_FALLBACK_MAX_CONF, FORK_FALLBACK_MIN_CONF, FORK_FALLBACK_MAX_ENTROPY, \
    FORK_FALLBACK_RANDOM = 0, 1, 2, 3, 4
FORK_TUNE_VARIANT, FORK_TUNE_CTAS_PER_SM, FORK_TUNE_PDL, FORK_TUNE_STAGES, FORK_TUNE_ONE_KERNEL, FORK_TUNE_LATE_CTA, \
    FORK_TUNE_L2_EVICT_FIRST, FORK_TUNE_MIN_UNITS, FORK_TUNE_LOOP_AHEAD = 0, 1, 2, 3, 4, 5, 6, 7, 8


class fork_step_args(C.Structure):
    _fields_ = [
        ("logits", C.c_void_p), ("stride_b", C.c_int64), ("stride_l", C.c_int64), ("pos0", C.c_int32),
        ("B", C.c_int32), ("Lt", C.c_int32), ("Ll", C.c_int32), ("V", C.c_int32), ("dtype", C.c_int32),
        ("tokens", C.c_void_p), ("mask", C.c_void_p), ("blk_lo", C.c_void_p), ("blk_hi", C.c_void_p),
        ("threshold", C.c_float), ("step", C.c_int32),
        ("conf", C.c_void_p), ("cand", C.c_void_p), ("entropy", C.c_void_p), ("logp", C.c_void_p),
        ("row_status", C.c_void_p),
        ("commit_step", C.c_void_p), ("commit_fallback", C.c_void_p), ("commit_logp", C.c_void_p),
        ("n_unmasked", C.c_void_p), ("is_fallback", C.c_void_p), ("fallback_pos", C.c_void_p),
        ("nfe", C.c_void_p), ("n_fallback", C.c_void_p),
        ("fallback_mode", C.c_int32), ("fallback_rand", C.c_void_p),
        ("temperature", C.c_float), ("sample_seed", C.c_uint64),
        ("sample_scratch", C.c_void_p), ("sample_scratch_bytes", C.c_size_t),
    ]


class fork_logprob_args(C.Structure):
    _fields_ = [
        ("logits", C.c_void_p), ("stride_b", C.c_int64), ("stride_l", C.c_int64), ("pos0", C.c_int32),
        ("B", C.c_int32), ("Lt", C.c_int32), ("Ll", C.c_int32), ("V", C.c_int32), ("dtype", C.c_int32),
        ("tokens", C.c_void_p), ("select", C.c_void_p), ("logp", C.c_void_p), ("seq_sum", C.c_void_p),
        ("seq_cnt", C.c_void_p), ("row_status", C.c_void_p), ("lse", C.c_void_p),
    ]


class fork_grpo_args(C.Structure):
    _fields_ = [
        ("B", C.c_int32), ("Lt", C.c_int32), ("group", C.c_int32),
        ("logp_new", C.c_void_p), ("logp_old", C.c_void_p), ("select", C.c_void_p), ("reward", C.c_void_p),
        ("eps_lo", C.c_float), ("eps_hi", C.c_float),
        ("seq_obj", C.c_void_p), ("objective", C.c_void_p), ("adv", C.c_void_p), ("ratio", C.c_void_p),
        ("dlogp", C.c_void_p), ("skipped", C.c_void_p),
    ]


class fork_logprob_bwd_args(C.Structure):
    _fields_ = [
        ("logits", C.c_void_p), ("stride_b", C.c_int64), ("stride_l", C.c_int64), ("pos0", C.c_int32),
        ("B", C.c_int32), ("Lt", C.c_int32), ("Ll", C.c_int32), ("V", C.c_int32), ("dtype", C.c_int32),
        ("tokens", C.c_void_p), ("select", C.c_void_p), ("lse", C.c_void_p), ("dlogp", C.c_void_p),
        ("grad", C.c_void_p), ("grad_stride_b", C.c_int64), ("grad_stride_l", C.c_int64),
    ]


class fork_grpo_fused_args(C.Structure):
    _fields_ = [
        ("logits", C.c_void_p), ("stride_b", C.c_int64), ("stride_l", C.c_int64),
        ("B", C.c_int32), ("Lt", C.c_int32), ("V", C.c_int32), ("dtype", C.c_int32),
        ("tokens", C.c_void_p), ("select", C.c_void_p), ("group", C.c_int32),
        ("logp_old", C.c_void_p), ("reward", C.c_void_p), ("eps_lo", C.c_float), ("eps_hi", C.c_float),
        ("grad", C.c_void_p), ("grad_stride_b", C.c_int64), ("grad_stride_l", C.c_int64),
        ("logp", C.c_void_p), ("lse", C.c_void_p), ("row_status", C.c_void_p),
        ("seq_obj", C.c_void_p), ("objective", C.c_void_p), ("adv", C.c_void_p), ("ratio", C.c_void_p),
        ("dlogp", C.c_void_p), ("skipped", C.c_void_p),
    ]


class fork_head_args(C.Structure):
    _fields_ = [("hidden", C.c_void_p), ("hidden_stride", C.c_int64), ("weight", C.c_void_p), ("weight_stride", C.c_int64),
                ("d", C.c_int32), ("row_pos0", C.c_void_p)]


fork_logits_fn = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                             C.c_void_p, C.c_void_p)

EXPORTS = ("fork_workspace_bytes", "fork_sample_scratch_bytes", "fork_step", "fork_step_static", "fork_step_fused_head", "fork_head_sample_scratch_bytes", "fork_logprob", "fork_decode_loop", "fork_decode_loop_fused_head", "fork_staging_bytes",
           "fork_select_top_entropy", "fork_grpo_loss", "fork_logprob_backward", "fork_grpo_fused", "fork_vp_reduce", "fork_vp_reduce_peers", "fork_vp_select", "fork_read_probe",
           "fork_step_host", "fork_device_status", "fork_status_string", "fork_set_tuning",
           "fork_kernel_launches", "fork_mask_handovers", "fork_workspace_release", "fork_set_timing_events",
           "fork_debug_part_begin", "fork_debug_part_owner", "fork_debug_row_parts", "fork_debug_chunk", "fork_debug_effective_grid")

_lib = None


def lib():
    """Load (building first if the shared object is missing or stale) the C-ABI library."""
    global _lib
    if _lib is not None:
        return _lib
    override = os.environ.get("FORK_DLLM_LIB")          # developer hook: load an experimental build instead
    try:
        path = override if override else _build.build()
    except Exception as e:  # no silent fallback: the CUDA library IS the product
        if not os.path.exists(_build.LIB):
            raise ImportError("libfork_dllm.so is missing and could not be built with nvcc: %r" % (e,)) from e
        path = _build.LIB
    L = C.CDLL(path)
    L.fork_workspace_bytes.restype = C.c_size_t
    L.fork_workspace_bytes.argtypes = [C.c_int32, C.c_int32]
    L.fork_sample_scratch_bytes.restype = C.c_size_t
    L.fork_sample_scratch_bytes.argtypes = [C.c_int32, C.c_int32]
    L.fork_step.restype = C.c_int
    L.fork_step.argtypes = [C.POINTER(fork_step_args), C.c_void_p, C.c_size_t, C.c_void_p]
    L.fork_step_static.restype = C.c_int
    L.fork_step_static.argtypes = [C.POINTER(fork_step_args), C.c_void_p]
    L.fork_step_fused_head.restype = C.c_int
    L.fork_step_fused_head.argtypes = [C.POINTER(fork_step_args), C.POINTER(fork_head_args), C.c_void_p, C.c_size_t, C.c_void_p]
    L.fork_logprob.restype = C.c_int
    L.fork_logprob.argtypes = [C.POINTER(fork_logprob_args), C.c_void_p, C.c_size_t, C.c_void_p]
    L.fork_decode_loop.restype = C.c_int
    L.fork_decode_loop.argtypes = [C.POINTER(fork_step_args), C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                   C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.c_void_p, C.c_size_t, C.c_void_p]
    L.fork_staging_bytes.restype = C.c_size_t
    L.fork_staging_bytes.argtypes = [C.POINTER(fork_step_args)]
    L.fork_step_host.restype = C.c_int
    L.fork_step_host.argtypes = [C.POINTER(fork_step_args), C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t, C.c_void_p]
    L.fork_device_status.restype = C.c_int
    L.fork_device_status.argtypes = [C.c_void_p, C.POINTER(C.c_uint32), C.c_void_p]
    L.fork_status_string.restype = C.c_char_p
    L.fork_status_string.argtypes = [C.c_int]
    L.fork_set_tuning.restype = C.c_int32
    L.fork_set_tuning.argtypes = [C.c_int32, C.c_int32]
    L.fork_kernel_launches.restype = C.c_int64
    L.fork_kernel_launches.argtypes = []
    L.fork_mask_handovers.restype = C.c_int64
    L.fork_mask_handovers.argtypes = []
    L.fork_workspace_release.restype = C.c_int
    L.fork_workspace_release.argtypes = [C.c_void_p]
    L.fork_vp_reduce_peers.restype = C.c_int
    L.fork_vp_reduce_peers.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.c_size_t, C.c_void_p]
    L.fork_select_top_entropy.restype = C.c_int
    L.fork_select_top_entropy.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_float, C.c_void_p,
                                          C.c_void_p, C.c_void_p]
    L.fork_grpo_loss.restype = C.c_int
    L.fork_grpo_loss.argtypes = [C.POINTER(fork_grpo_args), C.c_void_p]
    L.fork_logprob_backward.restype = C.c_int
    L.fork_logprob_backward.argtypes = [C.POINTER(fork_logprob_bwd_args), C.c_void_p, C.c_size_t, C.c_void_p]
    L.fork_head_sample_scratch_bytes.restype = C.c_size_t
    L.fork_head_sample_scratch_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32]
    L.fork_decode_loop_fused_head.restype = C.c_int
    L.fork_decode_loop_fused_head.argtypes = [C.POINTER(fork_step_args), C.POINTER(fork_head_args), C.c_int32, C.c_int32, C.c_int32,
                                              C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.c_void_p, C.c_size_t, C.c_void_p]
    L.fork_grpo_fused.restype = C.c_int
    L.fork_grpo_fused.argtypes = [C.POINTER(fork_grpo_fused_args), C.c_void_p, C.c_size_t, C.c_void_p]
    L.fork_vp_reduce.restype = C.c_int
    L.fork_vp_reduce.argtypes = [C.POINTER(fork_step_args), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                 C.c_void_p]
    L.fork_vp_select.restype = C.c_int
    L.fork_vp_select.argtypes = [C.POINTER(fork_step_args), C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t,
                                 C.c_void_p]
    L.fork_read_probe.restype = C.c_int
    L.fork_read_probe.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
    L.fork_set_timing_events.restype = None
    L.fork_set_timing_events.argtypes = [C.c_void_p, C.c_void_p]
    _lib = L
    return L


class ForkError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s" % (where, fork_status_string(status)))


def fork_status_string(status: int) -> str:
    return lib().fork_status_string(int(status)).decode()


def fork_workspace_bytes(B: int, Lt: int) -> int:
    return int(lib().fork_workspace_bytes(B, Lt))


def fork_set_tuning(key: int, value: int) -> int:
    return int(lib().fork_set_tuning(key, value))


def fork_kernel_launches() -> int:
    return int(lib().fork_kernel_launches())


def fork_mask_handovers() -> int:
    return int(lib().fork_mask_handovers())


def _p(t):
    return None if t is None else t.data_ptr()


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return FORK_BF16
    if t.dtype == torch.float32:
        return FORK_F32
    raise TypeError("logits must be bfloat16 or float32, got %s" % t.dtype)


class ForkState:
    """Device buffers of one batch: the sequence and its mask, every output of fork_step, and the
    scratch workspace.  Plain tensors; nothing here computes."""

    PER_POS = (("conf", torch.float32, float("nan")), ("cand", torch.int32, -1),
               ("entropy", torch.float32, float("nan")), ("logp", torch.float32, float("nan")),
               ("row_status", torch.int32, 0), ("commit_step", torch.int32, -1),
               ("commit_fallback", torch.uint8, 255), ("commit_logp", torch.float32, float("nan")))
    PER_SEQ = (("n_unmasked", torch.int32, 0), ("is_fallback", torch.uint8, 0), ("fallback_pos", torch.int32, -1),
               ("nfe", torch.int32, 0), ("n_fallback", torch.int32, 0))

    def __init__(self, B: int, Lt: int, device="cuda", tokens=None, mask=None):
        self.B, self.Lt, self.device = B, Lt, torch.device(device)
        dev = self.device
        self.tokens = (torch.zeros((B, Lt), dtype=torch.int32, device=dev) if tokens is None
                       else torch.as_tensor(tokens, dtype=torch.int32).to(dev).contiguous().clone())
        self.mask = (torch.ones((B, Lt), dtype=torch.uint8, device=dev) if mask is None
                     else torch.as_tensor(mask, dtype=torch.uint8).to(dev).contiguous().clone())
        for name, dt, fill in self.PER_POS:
            setattr(self, name, torch.full((B, Lt), fill, dtype=dt, device=dev))
        for name, dt, fill in self.PER_SEQ:
            setattr(self, name, torch.full((B,), fill, dtype=dt, device=dev))
        nbytes = fork_workspace_bytes(B, Lt)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=dev)
        off = (-self.workspace.data_ptr()) % 256
        self.ws_ptr, self.ws_bytes = self.workspace.data_ptr() + off, nbytes

    def sample_scratch_ptr(self):
        """Device scratch of a step that draws its candidates, allocated when first asked for."""
        if getattr(self, "_sample_scratch", None) is None:
            n = int(lib().fork_sample_scratch_bytes(self.B, self.Lt))
            self._sample_scratch = torch.zeros(n + 256, dtype=torch.uint8, device=self.device)   # (the library wants it zero-filled once)
            self._sample_bytes = n
        p = self._sample_scratch.data_ptr()
        return p + (-p) % 256, self._sample_bytes

    def close(self):
        """Give the control block the library keeps for this workspace address back (one-kernel
        steps).  Waits for the device first: the library's condition is that every call that used
        the workspace has completed."""
        ptr, self.ws_ptr = getattr(self, "ws_ptr", None), None
        if ptr and _lib is not None:
            with torch.cuda.device(self.device):
                torch.cuda.synchronize()
                _lib.fork_workspace_release(C.c_void_p(ptr))

    def __del__(self):
        try:
            self.close()
        except Exception:                  # interpreter or CUDA context already going away
            pass

    def host(self) -> dict:
        names = ["tokens", "mask"] + [n for n, _, _ in self.PER_POS] + [n for n, _, _ in self.PER_SEQ]
        return {n: getattr(self, n).cpu().numpy() for n in names}


def make_step_args(st: ForkState, logits: torch.Tensor, blk_lo, blk_hi, threshold: float, step: int = 0,
                   pos0: int = 0, fallback_mode: int = FORK_FALLBACK_LEFTMOST, fallback_rand=None,
                   temperature: float = 0.0, sample_seed: int = 0) -> fork_step_args:
    a = fork_step_args()
    if logits is None:                   # fork_vp_select: the logits are not read
        a.B, a.Lt, a.pos0 = st.B, st.Lt, pos0
    else:
        assert logits.dim() == 3 and logits.stride(2) == 1, "logits must be [B, Ll, V] with V contiguous"
        B, Ll, V = logits.shape
        assert B == st.B
        a.logits = logits.data_ptr()
        a.stride_b, a.stride_l, a.pos0 = logits.stride(0), logits.stride(1), pos0
        a.B, a.Lt, a.Ll, a.V, a.dtype = B, st.Lt, Ll, V, _dtype_code(logits)
    a.tokens, a.mask = st.tokens.data_ptr(), st.mask.data_ptr()
    a.blk_lo, a.blk_hi = _p(blk_lo), _p(blk_hi)
    a.threshold, a.step = float(threshold), int(step)
    for name, _, _ in ForkState.PER_POS + ForkState.PER_SEQ:
        setattr(a, name, getattr(st, name).data_ptr())
    a.fallback_mode, a.fallback_rand = int(fallback_mode), _p(fallback_rand)
    a.temperature, a.sample_seed = float(temperature), int(sample_seed)
    if temperature > 0 and logits is not None:           # (the fused-head step brings its own scratch; the select phase needs none)
        a.sample_scratch, a.sample_scratch_bytes = st.sample_scratch_ptr()
    return a


def fork_step(st: ForkState, logits: torch.Tensor, blk_lo: torch.Tensor, blk_hi: torch.Tensor, threshold: float,
              step: int = 0, pos0: int = 0, stream=None, **variant) -> None:
    """One sampling step on device buffers (asynchronous on the stream).  `variant` takes the
    fallback_mode / fallback_rand / temperature / sample_seed fields of fork_step_args."""
    a = make_step_args(st, logits, blk_lo, blk_hi, threshold, step, pos0, **variant)
    rc = lib().fork_step(C.byref(a), C.c_void_p(st.ws_ptr), st.ws_bytes, _stream_ptr(stream))
    if rc != FORK_OK:
        raise ForkError(rc, "fork_step")


FORK_STATIC_SCRATCH_BYTES = 2 * 1024 * 1024


def fork_step_static(st: ForkState, logits: torch.Tensor, blk_lo: torch.Tensor, blk_hi: torch.Tensor,
                     threshold: float, step: int = 0, pos0: int = 0, stream=None) -> None:
    """fork_step on the library's built-in scratch: for callers that cannot allocate device memory
    (a server whose pool owns the device, a latency-critical path).  `st.workspace` is not used.
    Raises ForkError(FORK_ERR_WORKSPACE) when the batch needs more than FORK_STATIC_SCRATCH_BYTES."""
    a = make_step_args(st, logits, blk_lo, blk_hi, threshold, step, pos0)
    rc = lib().fork_step_static(C.byref(a), _stream_ptr(stream))
    if rc != FORK_OK:
        raise ForkError(rc, "fork_step_static")


def _head_sample_scratch(st: ForkState, a: fork_step_args, B: int, Ll: int, V: int, device) -> None:
    """Scratch of a fused-head step that draws its candidates; kept on the state and reused while it is large enough."""
    if not a.temperature > 0:
        return
    n = int(lib().fork_head_sample_scratch_bytes(B, Ll, V))
    buf = getattr(st, "_head_scratch", None)
    if buf is None or buf.numel() < n + 256:
        buf = torch.empty(n + 256, dtype=torch.uint8, device=device)
        st._head_scratch = buf
    off = (-buf.data_ptr()) % 256
    a.sample_scratch, a.sample_scratch_bytes = buf.data_ptr() + off, n


def _head_args(hidden: torch.Tensor, weight: torch.Tensor, row_pos0=None) -> fork_head_args:
    assert hidden.dtype == torch.bfloat16 and weight.dtype == torch.bfloat16
    assert hidden.dim() == 3 and hidden.stride(2) == 1 and hidden.stride(0) == hidden.shape[1] * hidden.stride(1)
    assert weight.dim() == 2 and weight.stride(1) == 1 and weight.shape[1] == hidden.shape[2]
    h = fork_head_args()
    h.hidden, h.hidden_stride, h.weight, h.weight_stride, h.d = hidden.data_ptr(), hidden.stride(1), weight.data_ptr(), weight.stride(0), hidden.shape[2]
    if row_pos0 is not None:
        assert row_pos0.dtype == torch.int32 and row_pos0.is_contiguous() and row_pos0.numel() == hidden.shape[0]
        h.row_pos0 = row_pos0.data_ptr()
    return h


def fork_decode_loop_fused_head(st: ForkState, hidden: torch.Tensor, weight: torch.Tensor, block_len: int, gen_lo: int, gen_hi: int,
                                provider, ctx, threshold: float, max_steps: int, step0: int = 0, stream=None,
                                raise_on_error: bool = True, **variant):
    """fork_decode_loop on hidden states: `provider` (as for fork_decode_loop) fills `hidden` [B, Ll, d] with each
    sequence's active block (row l of sequence b = position lo[b] + l); the step is the fused LM-head step.
    Returns (status, steps_taken)."""
    B, Ll, d = hidden.shape
    assert B == st.B
    a = make_step_args(st, None, None, None, threshold, step0, 0, **variant)
    a.Ll, a.V = Ll, weight.shape[0]
    _head_sample_scratch(st, a, B, Ll, a.V, hidden.device)
    h = _head_args(hidden, weight)
    keep = None
    if callable(provider) and not isinstance(provider, (int, C._CFuncPtr)):
        def _tramp(_ctx, step, _tok, _mask, lo, hi, _out, stream_p):
            try:
                return int(provider(int(step), lo, hi, stream_p) or 0)
            except Exception:
                import traceback
                traceback.print_exc()
                return 1
        keep = fork_logits_fn(_tramp)
        fn_ptr = C.cast(keep, C.c_void_p)
    elif isinstance(provider, int):
        fn_ptr = C.c_void_p(provider)
    else:
        fn_ptr = C.cast(provider, C.c_void_p)
    steps = C.c_int32(0)
    rc = lib().fork_decode_loop_fused_head(C.byref(a), C.byref(h), block_len, gen_lo, gen_hi, fn_ptr, C.c_void_p(ctx or 0), max_steps,
                                           C.byref(steps), C.c_void_p(st.ws_ptr), st.ws_bytes, _stream_ptr(stream))
    del keep
    if rc != FORK_OK and raise_on_error:
        raise ForkError(rc, "fork_decode_loop_fused_head")
    return int(rc), int(steps.value)


def fork_step_fused_head(st: ForkState, hidden: torch.Tensor, weight: torch.Tensor, blk_lo: torch.Tensor, blk_hi: torch.Tensor,
                         threshold: float, step: int = 0, pos0: int = 0, stream=None, row_pos0=None, **variant) -> None:
    """One sampling step from hidden states [B, Ll, d] (bf16) and the LM-head weight [V, d] (bf16): the
    logits are formed and reduced on the fly, never stored.  `row_pos0` [B] int32 (optional): every sequence's
    window starts at its own position.  Asynchronous on the stream."""
    assert hidden.dtype == torch.bfloat16 and weight.dtype == torch.bfloat16
    assert hidden.dim() == 3 and hidden.stride(2) == 1 and hidden.stride(0) == hidden.shape[1] * hidden.stride(1)
    assert weight.dim() == 2 and weight.stride(1) == 1 and weight.shape[1] == hidden.shape[2]
    B, Ll, d = hidden.shape
    assert B == st.B
    a = make_step_args(st, None, blk_lo, blk_hi, threshold, step, pos0, **variant)
    a.Ll, a.V = Ll, weight.shape[0]
    _head_sample_scratch(st, a, B, Ll, a.V, hidden.device)
    h = _head_args(hidden, weight, row_pos0)
    rc = lib().fork_step_fused_head(C.byref(a), C.byref(h), C.c_void_p(st.ws_ptr), st.ws_bytes, _stream_ptr(stream))
    if rc != FORK_OK:
        raise ForkError(rc, "fork_step_fused_head")


def fork_logprob(logits: torch.Tensor, tokens: torch.Tensor, select: torch.Tensor, st: ForkState, pos0: int = 0,
                 stream=None, want_lse: bool = False):
    """Log-likelihood of `tokens` at the selected positions; returns (logp [B,Lt], seq_sum [B],
    seq_cnt [B], row_status [B,Lt]) as device tensors (asynchronous on the stream), plus the
    rows' log-sum-exp [B,Lt] (for fork_logprob_backward) when `want_lse`."""
    assert logits.dim() == 3 and logits.stride(2) == 1
    B, Ll, V = logits.shape
    Lt = tokens.shape[1]
    dev = logits.device
    logp = torch.empty((B, Lt), dtype=torch.float32, device=dev)
    seq_sum = torch.empty((B,), dtype=torch.float32, device=dev)
    seq_cnt = torch.empty((B,), dtype=torch.int32, device=dev)
    status = torch.zeros((B, Lt), dtype=torch.int32, device=dev)
    a = fork_logprob_args()
    a.logits = logits.data_ptr()
    a.stride_b, a.stride_l, a.pos0 = logits.stride(0), logits.stride(1), pos0
    a.B, a.Lt, a.Ll, a.V, a.dtype = B, Lt, Ll, V, _dtype_code(logits)
    assert tokens.dtype == torch.int32 and select.dtype == torch.uint8 and tokens.is_contiguous() and select.is_contiguous()
    a.tokens, a.select = tokens.data_ptr(), select.data_ptr()
    a.logp, a.seq_sum, a.seq_cnt, a.row_status = logp.data_ptr(), seq_sum.data_ptr(), seq_cnt.data_ptr(), status.data_ptr()
    lse = torch.zeros((B, Lt), dtype=torch.float32, device=dev) if want_lse else None
    a.lse = _p(lse)
    rc = lib().fork_logprob(C.byref(a), C.c_void_p(st.ws_ptr), st.ws_bytes, _stream_ptr(stream))
    if rc != FORK_OK:
        raise ForkError(rc, "fork_logprob")
    return (logp, seq_sum, seq_cnt, status, lse) if want_lse else (logp, seq_sum, seq_cnt, status)


def fork_decode_loop(st: ForkState, logits: torch.Tensor, block_len: int, gen_lo: int, gen_hi: int, provider,
                     ctx, threshold: float, max_steps: int, step0: int = 0, pos0: int = 0, stream=None,
                     raise_on_error: bool = True, **variant):
    """Semi-autoregressive decoding.  `provider` is either a C function pointer (int address or
    ctypes function) with the fork_logits_fn signature plus its `ctx` pointer, or a Python callable
    ``provider(step, lo_ptr, hi_ptr, stream_ptr) -> int`` that enqueues the work filling `logits`.
    Returns (status, steps_taken)."""
    a = make_step_args(st, logits, None, None, threshold, step0, pos0, **variant)
    keep = None
    if callable(provider) and not isinstance(provider, (int, C._CFuncPtr)):
        def _tramp(_ctx, step, _tok, _mask, lo, hi, _out, stream_p):
            try:
                return int(provider(int(step), lo, hi, stream_p) or 0)
            except Exception:
                import traceback
                traceback.print_exc()
                return 1
        keep = fork_logits_fn(_tramp)
        fn_ptr = C.cast(keep, C.c_void_p)
    elif isinstance(provider, int):
        fn_ptr = C.c_void_p(provider)
    else:
        fn_ptr = C.cast(provider, C.c_void_p)
    steps = C.c_int32(0)
    rc = lib().fork_decode_loop(C.byref(a), block_len, gen_lo, gen_hi, fn_ptr, C.c_void_p(ctx or 0), max_steps,
                                C.byref(steps), C.c_void_p(st.ws_ptr), st.ws_bytes, _stream_ptr(stream))
    del keep
    if rc != FORK_OK and raise_on_error:
        raise ForkError(rc, "fork_decode_loop")
    return int(rc), int(steps.value)


def fork_device_status(st, stream=None) -> int:
    """Device status word (FORK_DEV_* bits) of the last call on `st`'s workspace; `st` = None asks
    about the library's built-in scratch (fork_step_static)."""
    out = C.c_uint32(0)
    rc = lib().fork_device_status(C.c_void_p(st.ws_ptr) if st is not None else None, C.byref(out), _stream_ptr(stream))
    if rc != FORK_OK:
        raise ForkError(rc, "fork_device_status")
    return int(out.value)


def fork_select_top_entropy(entropy: torch.Tensor, eligible: torch.Tensor, ratio: float, stream=None):
    """JustGRPO-Fast's selection: returns (select [B,Lt] uint8, n_selected [B] int32) device tensors."""
    assert entropy.dtype == torch.float32 and eligible.dtype == torch.uint8
    assert entropy.is_contiguous() and eligible.is_contiguous() and entropy.shape == eligible.shape
    B, Lt = entropy.shape
    select = torch.empty((B, Lt), dtype=torch.uint8, device=entropy.device)
    cnt = torch.empty((B,), dtype=torch.int32, device=entropy.device)
    rc = lib().fork_select_top_entropy(C.c_void_p(entropy.data_ptr()), C.c_void_p(eligible.data_ptr()), B, Lt,
                                       C.c_float(ratio), C.c_void_p(select.data_ptr()), C.c_void_p(cnt.data_ptr()),
                                       _stream_ptr(stream))
    if rc != FORK_OK:
        raise ForkError(rc, "fork_select_top_entropy")
    return select, cnt


def fork_grpo_loss(logp_new: torch.Tensor, logp_old: torch.Tensor, select: torch.Tensor, reward: torch.Tensor,
                   group: int, eps_lo: float, eps_hi: float, stream=None) -> dict:
    """The ForkGRPO objective (Eq. 2) and its derivative with respect to logp_new; device tensors."""
    for t, dt in ((logp_new, torch.float32), (logp_old, torch.float32), (select, torch.uint8), (reward, torch.float32)):
        assert t.dtype == dt and t.is_contiguous()
    B, Lt = logp_new.shape
    dev = logp_new.device
    out = dict(seq_obj=torch.empty(B, dtype=torch.float32, device=dev),
               objective=torch.empty(1, dtype=torch.float32, device=dev),
               adv=torch.empty(B, dtype=torch.float32, device=dev),
               ratio=torch.empty((B, Lt), dtype=torch.float32, device=dev),
               dlogp=torch.empty((B, Lt), dtype=torch.float32, device=dev),
               skipped=torch.empty(max(B // max(group, 1), 1), dtype=torch.uint8, device=dev))
    a = fork_grpo_args()
    a.B, a.Lt, a.group = B, Lt, group
    a.logp_new, a.logp_old, a.select, a.reward = (t.data_ptr() for t in (logp_new, logp_old, select, reward))
    a.eps_lo, a.eps_hi = float(eps_lo), float(eps_hi)
    for name, t in out.items():
        setattr(a, name, t.data_ptr())
    rc = lib().fork_grpo_loss(C.byref(a), _stream_ptr(stream))
    if rc != FORK_OK:
        raise ForkError(rc, "fork_grpo_loss")
    return out


def fork_grpo_fused(logits: torch.Tensor, tokens: torch.Tensor, select: torch.Tensor, logp_old: torch.Tensor,
                    reward: torch.Tensor, group: int, eps_lo: float, eps_hi: float, grad: torch.Tensor, st: ForkState,
                    stream=None) -> dict:
    """Scoring, Eq. 2 and the log-softmax backward in one pass over `logits` [B,Lt,V]: returns the outputs of
    fork_logprob and fork_grpo_loss as a dict and writes d J / d logits into the selected rows of `grad`."""
    assert logits.dim() == 3 and logits.stride(2) == 1 and grad.dim() == 3 and grad.stride(2) == 1
    assert grad.dtype == logits.dtype and grad.shape == logits.shape
    B, Lt, V = logits.shape
    for t, dt in ((tokens, torch.int32), (select, torch.uint8), (logp_old, torch.float32), (reward, torch.float32)):
        assert t.dtype == dt and t.is_contiguous()
    assert tuple(tokens.shape) == (B, Lt) and st.B == B and st.Lt == Lt
    dev = logits.device
    out = dict(logp=torch.zeros((B, Lt), dtype=torch.float32, device=dev),
               lse=torch.zeros((B, Lt), dtype=torch.float32, device=dev),
               row_status=torch.zeros((B, Lt), dtype=torch.int32, device=dev),
               seq_obj=torch.empty(B, dtype=torch.float32, device=dev),
               objective=torch.empty(1, dtype=torch.float32, device=dev),
               adv=torch.empty(B, dtype=torch.float32, device=dev),
               ratio=torch.zeros((B, Lt), dtype=torch.float32, device=dev),
               dlogp=torch.zeros((B, Lt), dtype=torch.float32, device=dev),
               skipped=torch.empty(max(B // max(group, 1), 1), dtype=torch.uint8, device=dev))
    a = fork_grpo_fused_args()
    a.logits, a.stride_b, a.stride_l = logits.data_ptr(), logits.stride(0), logits.stride(1)
    a.B, a.Lt, a.V, a.dtype = B, Lt, V, _dtype_code(logits)
    a.tokens, a.select, a.group = tokens.data_ptr(), select.data_ptr(), group
    a.logp_old, a.reward, a.eps_lo, a.eps_hi = logp_old.data_ptr(), reward.data_ptr(), float(eps_lo), float(eps_hi)
    a.grad, a.grad_stride_b, a.grad_stride_l = grad.data_ptr(), grad.stride(0), grad.stride(1)
    for name, t in out.items():
        setattr(a, name, t.data_ptr())
    rc = lib().fork_grpo_fused(C.byref(a), C.c_void_p(st.ws_ptr), st.ws_bytes, _stream_ptr(stream))
    if rc != FORK_OK:
        raise ForkError(rc, "fork_grpo_fused")
    return out


def fork_logprob_backward(logits: torch.Tensor, tokens: torch.Tensor, select: torch.Tensor, lse: torch.Tensor,
                          dlogp: torch.Tensor, grad: torch.Tensor, st: ForkState, pos0: int = 0, stream=None) -> None:
    """Writes d(sum dlogp * logp)/d logits into the rows of `grad` ([B,Ll,V] like `logits`) that belong
    to selected positions; other rows are left as they are."""
    assert logits.dim() == 3 and logits.stride(2) == 1 and grad.dim() == 3 and grad.stride(2) == 1
    assert grad.dtype == logits.dtype and grad.shape == logits.shape
    B, Ll, V = logits.shape
    a = fork_logprob_bwd_args()
    a.logits = logits.data_ptr()
    a.stride_b, a.stride_l, a.pos0 = logits.stride(0), logits.stride(1), pos0
    a.B, a.Lt, a.Ll, a.V, a.dtype = B, tokens.shape[1], Ll, V, _dtype_code(logits)
    a.tokens, a.select, a.lse, a.dlogp = tokens.data_ptr(), select.data_ptr(), lse.data_ptr(), dlogp.data_ptr()
    a.grad, a.grad_stride_b, a.grad_stride_l = grad.data_ptr(), grad.stride(0), grad.stride(1)
    rc = lib().fork_logprob_backward(C.byref(a), C.c_void_p(st.ws_ptr), st.ws_bytes, _stream_ptr(stream))
    if rc != FORK_OK:
        raise ForkError(rc, "fork_logprob_backward")


# ---- vocabulary-parallel step -------------------------------------------------------------------
def vocab_shards(V: int, n_ranks: int, elem_size: int):
    """(offset, length) of every rank's slice of the vocabulary: equal sizes rounded so that each
    slice starts on a 16-byte boundary (the last rank takes the remainder)."""
    per = 16 // elem_size
    base = -(-V // n_ranks)
    base = -(-base // per) * per
    out = []
    for r in range(n_ranks):
        lo = min(r * base, V)
        out.append((lo, max(0, min(V, lo + base) - lo)))
    return out


def fork_vp_reduce(st: ForkState, logits_slice: torch.Tensor, blk_lo, blk_hi, threshold: float, vocab_offset: int,
                   step: int = 0, pos0: int = 0, stream=None, **variant):
    """Local phase on this rank's slice [B, Ll, V_local]: returns (parts [B,Lt,4] float32, keys
    [B,Lt,4] float32 or None) for the exchange; nothing is committed."""
    a = make_step_args(st, logits_slice, blk_lo, blk_hi, threshold, step, pos0, **variant)
    dev = logits_slice.device
    parts = torch.zeros((st.B, st.Lt, 4), dtype=torch.float32, device=dev)
    keys = torch.zeros((st.B, st.Lt, 4), dtype=torch.float32, device=dev) if a.temperature > 0 else None
    rc = lib().fork_vp_reduce(C.byref(a), int(vocab_offset), C.c_void_p(parts.data_ptr()), C.c_void_p(_p(keys) or 0),
                              C.c_void_p(st.ws_ptr), st.ws_bytes, _stream_ptr(stream))
    if rc != FORK_OK:
        raise ForkError(rc, "fork_vp_reduce")
    return parts, keys


def fork_vp_reduce_peers(st: ForkState, logits_slice: torch.Tensor, blk_lo, blk_hi, threshold: float, vocab_offset: int,
                         rank: int, gather_parts, gather_keys=None, step: int = 0, pos0: int = 0, stream=None,
                         **variant) -> None:
    """Local phase with the exchange fused in: this rank's slice results go straight into slot `rank`
    of EVERY rank's gather buffer.  gather_parts[j] (and gather_keys[j] with drawn candidates) is rank
    j's buffer [N, B, Lt, 4] float32 as addressable from this GPU: a tensor, or an integer device
    address of peer-mapped memory.  The caller orders the select phase after the completion of this
    call on all ranks."""
    a = make_step_args(st, logits_slice, blk_lo, blk_hi, threshold, step, pos0, **variant)
    n = len(gather_parts)

    def addresses(bufs):
        arr = (C.c_void_p * n)()
        for j, t in enumerate(bufs):
            if isinstance(t, torch.Tensor):
                assert t.dtype == torch.float32 and t.is_contiguous() and tuple(t.shape) == (n, st.B, st.Lt, 4)
                arr[j] = t.data_ptr()
            else:
                arr[j] = int(t)
        return arr

    parts_arr = addresses(gather_parts)
    keys_arr = addresses(gather_keys) if (a.temperature > 0 and gather_keys is not None) else None
    rc = lib().fork_vp_reduce_peers(C.byref(a), int(vocab_offset), int(rank), n, parts_arr, keys_arr,
                                    C.c_void_p(st.ws_ptr), st.ws_bytes, _stream_ptr(stream))
    if rc != FORK_OK:
        raise ForkError(rc, "fork_vp_reduce_peers")


def fork_vp_select(st: ForkState, parts: torch.Tensor, keys, blk_lo, blk_hi, threshold: float, step: int = 0,
                   pos0: int = 0, Ll: int = 0, stream=None, **variant) -> None:
    """Select phase on the gathered slices: parts (and keys) are [N, B, Lt, 4] in rank order."""
    assert parts.dim() == 4 and parts.is_contiguous() and parts.dtype == torch.float32
    a = make_step_args(st, None, blk_lo, blk_hi, threshold, step, pos0, **variant)
    a.Ll = Ll
    rc = lib().fork_vp_select(C.byref(a), C.c_void_p(parts.data_ptr()), C.c_void_p(_p(keys) or 0), parts.shape[0],
                              C.c_void_p(st.ws_ptr), st.ws_bytes, _stream_ptr(stream))
    if rc != FORK_OK:
        raise ForkError(rc, "fork_vp_select")


def gather_rank_major(t: torch.Tensor, group=None) -> torch.Tensor:
    """All-gather of one tensor per rank into [world, ...] in rank order (torch.distributed)."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    out = [torch.empty_like(t) for _ in range(world)]
    dist.all_gather(out, t.contiguous(), group=group)
    return torch.stack(out, 0)


def fork_step_vocab_parallel(st: ForkState, logits_slice: torch.Tensor, blk_lo, blk_hi, threshold: float,
                             vocab_offset: int, step: int = 0, pos0: int = 0, group=None, stream=None,
                             peer_buffers=None, **variant) -> None:
    """One sampling step with the vocabulary sharded over the ranks of `group`: local reduction, an
    exchange of 16 (32 with drawn candidates) bytes per position, selection on every rank.  Slices
    must ascend with the rank (vocab_shards).
    The exchange is one all-gather (torch.distributed), or, with `peer_buffers` = (gather_parts,
    gather_keys or None) as fork_vp_reduce_peers takes them (every rank's gather buffer mapped on
    this GPU), stores issued by the reduction kernel itself followed by a barrier of the group."""
    if peer_buffers is not None:
        import torch.distributed as dist
        rank = dist.get_rank(group)
        g_parts_all, g_keys_all = peer_buffers
        fork_vp_reduce_peers(st, logits_slice, blk_lo, blk_hi, threshold, vocab_offset, rank, g_parts_all, g_keys_all,
                             step, pos0, stream, **variant)
        (stream or torch.cuda.current_stream()).synchronize()      # this rank's stores are out ...
        dist.barrier(group)                                        # ... and so are everybody else's
        mine = g_parts_all[rank]
        keys_mine = g_keys_all[rank] if (g_keys_all is not None and variant.get("temperature", 0.0) > 0) else None
        fork_vp_select(st, mine, keys_mine, blk_lo, blk_hi, threshold, step, pos0, logits_slice.shape[1], stream, **variant)
        return
    parts, keys = fork_vp_reduce(st, logits_slice, blk_lo, blk_hi, threshold, vocab_offset, step, pos0, stream, **variant)
    g_parts = gather_rank_major(parts, group)
    g_keys = gather_rank_major(keys, group) if keys is not None else None
    fork_vp_select(st, g_parts, g_keys, blk_lo, blk_hi, threshold, step, pos0, logits_slice.shape[1], stream, **variant)
