"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the header
declares, rejects bad arguments before touching CUDA, and its work partition is consistent."""
import ctypes as C
import os
import re

import pytest

import paper_2609_39859_b200 as pkg

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "fork_dllm.h")


def declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    names = set(re.findall(r"\b(fork_[a-z_]+)\s*\(", src))
    names.discard("fork_logits_fn")
    return sorted(names)


def test_library_exports_every_declared_symbol():
    L = pkg.lib()
    names = declared_functions()
    assert {"fork_step", "fork_logprob", "fork_decode_loop", "fork_workspace_bytes", "fork_step_host"} <= set(names)
    for n in names:
        assert hasattr(L, n), n
    assert set(pkg.binding.EXPORTS) == set(names)


def test_status_strings_and_workspace_size():
    assert pkg.fork_status_string(0) == "FORK_OK"
    assert pkg.fork_status_string(-4) == "FORK_ERR_MAX_STEPS"
    assert pkg.fork_status_string(99) == "FORK_UNKNOWN_STATUS"
    a, b = pkg.fork_workspace_bytes(8, 256), pkg.fork_workspace_bytes(64, 256)
    assert 0 < a < b and a % 256 == 0
    assert pkg.fork_workspace_bytes(-1, 256) == 0 and pkg.fork_workspace_bytes(4, 0) == 0


def good_step_args():
    a = pkg.fork_step_args()
    a.logits = 0x1000
    a.stride_b, a.stride_l, a.pos0 = 32 * 1024, 1024, 0
    a.B, a.Lt, a.Ll, a.V, a.dtype = 2, 32, 32, 1024, pkg.FORK_BF16
    a.tokens, a.mask, a.blk_lo, a.blk_hi = 0x2000, 0x3000, 0x4000, 0x5000
    a.threshold, a.step = 0.9, 0
    return a


def test_invalid_arguments_are_rejected_on_the_host():
    """None of these reach a CUDA call (the pointers are fake, and this machine has no GPU)."""
    L = pkg.lib()
    ws, nbytes = C.c_void_p(0x100000), pkg.fork_workspace_bytes(2, 32)
    assert L.fork_step(None, ws, nbytes, None) == pkg.FORK_ERR_INVALID_ARG
    for field, value in (("logits", None), ("tokens", None), ("mask", None), ("blk_lo", None), ("blk_hi", None),
                         ("V", 0), ("Lt", 0), ("Ll", 0), ("B", -1), ("dtype", 7), ("stride_l", 100), ("pos0", -1),
                         ("threshold", float("nan"))):
        a = good_step_args()
        setattr(a, field, value)
        assert L.fork_step(C.byref(a), ws, nbytes, None) == pkg.FORK_ERR_INVALID_ARG, field
    a = good_step_args()
    assert L.fork_step(C.byref(a), None, nbytes, None) == pkg.FORK_ERR_WORKSPACE
    assert L.fork_step(C.byref(a), ws, nbytes - 1, None) == pkg.FORK_ERR_WORKSPACE
    assert L.fork_step(C.byref(a), C.c_void_p(0x100010), nbytes, None) == pkg.FORK_ERR_WORKSPACE   # not 256-aligned
    a.B = 0
    assert L.fork_step(C.byref(a), ws, nbytes, None) == pkg.FORK_OK                                # nothing to do
    # decode loop
    steps = C.c_int32(-1)
    a = good_step_args()
    assert L.fork_decode_loop(C.byref(a), 32, 0, 32, None, None, 10, C.byref(steps), ws, nbytes, None) == pkg.FORK_ERR_INVALID_ARG
    fn = C.c_void_p(0x1234)
    for bl, glo, ghi, ms in ((0, 0, 32, 10), (32, -1, 32, 10), (32, 0, 33, 10), (32, 8, 4, 10), (32, 0, 32, -1)):
        assert L.fork_decode_loop(C.byref(a), bl, glo, ghi, fn, None, ms, C.byref(steps), ws, nbytes, None) == pkg.FORK_ERR_INVALID_ARG
    assert steps.value == 0
    # scoring
    lp = pkg.fork_logprob_args()
    assert L.fork_logprob(None, ws, nbytes, None) == pkg.FORK_ERR_INVALID_ARG
    lp.logits, lp.stride_b, lp.stride_l, lp.B, lp.Lt, lp.Ll, lp.V, lp.dtype = 0x1000, 32 * 1024, 1024, 2, 32, 32, 1024, 1
    lp.tokens, lp.select, lp.logp = 0x2000, 0x3000, None
    assert L.fork_logprob(C.byref(lp), ws, nbytes, None) == pkg.FORK_ERR_INVALID_ARG
    # host entry point
    a = good_step_args()
    assert L.fork_staging_bytes(C.byref(a)) > 2 * 32 * 1024 * 2
    assert L.fork_step_host(C.byref(a), None, 1 << 30, ws, nbytes, None) == pkg.FORK_ERR_WORKSPACE
    a.stride_b = 32 * 1024 + 8
    assert L.fork_step_host(C.byref(a), C.c_void_p(0x200000), 1 << 30, ws, nbytes, None) == pkg.FORK_ERR_INVALID_ARG
    assert L.fork_device_status(None, None, None) == pkg.FORK_ERR_INVALID_ARG


def test_tuning_knobs_round_trip():
    assert pkg.fork_set_tuning(99, 1) == -1
    old = pkg.fork_set_tuning(pkg.FORK_TUNE_CTAS_PER_SM, 2)
    assert pkg.fork_set_tuning(pkg.FORK_TUNE_CTAS_PER_SM, old) == 2
    assert pkg.fork_kernel_launches() >= 0


def test_partition_is_a_partition():
    """Brute force: CTA ranges tile [0,U) in order, the owner formula inverts them, the number of
    parts per row matches a direct count, and the slot r+g is unique and below R+G."""
    L = pkg.lib()
    L.fork_debug_part_begin.restype = C.c_int64
    L.fork_debug_part_begin.argtypes = [C.c_int64, C.c_int32, C.c_int32]
    L.fork_debug_part_owner.restype = C.c_int32
    L.fork_debug_part_owner.argtypes = [C.c_int64, C.c_int32, C.c_int64]
    L.fork_debug_row_parts.restype = C.c_int32
    L.fork_debug_row_parts.argtypes = [C.c_int64, C.c_int32, C.c_int32, C.c_int64]
    assert L.fork_debug_chunk() == 2048
    L.fork_debug_effective_grid.restype = C.c_int32
    L.fork_debug_effective_grid.argtypes = [C.c_int64, C.c_int32, C.c_int32]
    for R in (1, 2, 3, 8, 31, 32, 33, 256, 700):
        for Cc in (1, 2, 5, 62, 75):
            for G0, mu in ((1, 1), (3, 1), (148, 1), (592, 1), (2048, 1), (296, 8), (296, 3), (592, 64)):
                U = R * Cc
                G = L.fork_debug_effective_grid(U, G0, mu)
                assert G == min(G0, -(-U // mu)) and 1 <= G <= U        # every CTA owns a unit; small steps use fewer CTAs
                begins = [L.fork_debug_part_begin(U, G, g) for g in range(G + 1)]
                assert begins[0] == 0 and begins[-1] == U and all(x <= y for x, y in zip(begins, begins[1:]))
                assert max(y - x for x, y in zip(begins, begins[1:])) - min(y - x for x, y in zip(begins, begins[1:])) <= 1
                slots = set()
                for r in range(R):
                    owners = sorted({L.fork_debug_part_owner(U, G, u) for u in range(r * Cc, (r + 1) * Cc)})
                    for u in (r * Cc, (r + 1) * Cc - 1):
                        g = L.fork_debug_part_owner(U, G, u)
                        assert begins[g] <= u < begins[g + 1]
                    assert owners == list(range(owners[0], owners[-1] + 1))
                    assert L.fork_debug_row_parts(U, G, Cc, r) == len(owners)
                    for g in owners:
                        assert (r + g) not in slots and r + g < R + G
                        slots.add(r + g)
    # sizes of the real workloads: no overflow in the 64-bit arithmetic
    U = 32768 * 75
    assert L.fork_debug_part_begin(U, 2048, 2048) == U and L.fork_debug_part_owner(U, 2048, U - 1) == 2047


def test_invalid_arguments_of_the_variant_entry_points():
    """Fallback order / temperature fields, selection, objective, backward and the vocabulary-parallel
    pair: every bad argument is refused before any CUDA call."""
    L = pkg.lib()
    ws, nbytes = C.c_void_p(0x100000), pkg.fork_workspace_bytes(2, 32)
    INV = pkg.FORK_ERR_INVALID_ARG
    for field, value in (("fallback_mode", 5), ("fallback_mode", -1), ("fallback_mode", pkg.FORK_FALLBACK_RANDOM),
                         ("temperature", -0.5), ("temperature", float("nan")), ("temperature", float("inf"))):
        a = good_step_args()
        setattr(a, field, value)
        assert L.fork_step(C.byref(a), ws, nbytes, None) == INV, field
        assert L.fork_vp_reduce(C.byref(a), 0, C.c_void_p(0x9000), C.c_void_p(0xA000), ws, nbytes, None) == INV, field
    a = good_step_args()
    assert L.fork_vp_reduce(C.byref(a), 0, None, None, ws, nbytes, None) == INV              # no output buffer
    assert L.fork_vp_reduce(C.byref(a), -1, C.c_void_p(0x9000), None, ws, nbytes, None) == INV
    assert L.fork_vp_reduce(C.byref(a), 0, C.c_void_p(0x9004), None, ws, nbytes, None) == INV  # not 16-byte aligned
    a.temperature = 0.8
    assert L.fork_vp_reduce(C.byref(a), 0, C.c_void_p(0x9000), None, ws, nbytes, None) == INV  # keys needed
    assert L.fork_vp_select(C.byref(a), C.c_void_p(0x9000), None, 2, ws, nbytes, None) == INV
    a.temperature = 0.0
    assert L.fork_vp_select(C.byref(a), None, None, 2, ws, nbytes, None) == INV
    assert L.fork_vp_select(C.byref(a), C.c_void_p(0x9000), None, 0, ws, nbytes, None) == INV
    assert L.fork_vp_select(C.byref(a), C.c_void_p(0x9000), None, 2, ws, 16, None) == pkg.FORK_ERR_WORKSPACE
    p = C.c_void_p(0x9000)
    assert L.fork_select_top_entropy(None, p, 2, 8, 0.2, p, None, None) == INV
    assert L.fork_select_top_entropy(p, p, 2, 8, 1.5, p, None, None) == INV
    assert L.fork_select_top_entropy(p, p, 2, 8, -0.1, p, None, None) == INV
    assert L.fork_select_top_entropy(p, p, 2, 40000, 0.2, p, None, None) == INV
    assert L.fork_select_top_entropy(p, p, 0, 8, 0.2, p, None, None) == pkg.FORK_OK          # empty batch
    g = pkg.fork_grpo_args()
    g.B, g.Lt, g.group = 4, 8, 2
    g.logp_new = g.logp_old = g.select = g.reward = g.seq_obj = 0x9000
    g.eps_lo = g.eps_hi = 0.2
    for field, value in (("group", 3), ("group", 0), ("Lt", 0), ("logp_new", None), ("reward", None), ("seq_obj", None),
                         ("eps_lo", -1.0), ("eps_hi", float("nan"))):
        bad = pkg.fork_grpo_args.from_buffer_copy(g)
        setattr(bad, field, value)
        assert L.fork_grpo_loss(C.byref(bad), None) == INV, field
    assert L.fork_grpo_loss(None, None) == INV
    b = pkg.fork_logprob_bwd_args()
    b.logits = 0x1000
    b.stride_b, b.stride_l, b.pos0 = 32 * 1024, 1024, 0
    b.B, b.Lt, b.Ll, b.V, b.dtype = 2, 32, 32, 1024, pkg.FORK_BF16
    b.tokens = b.select = b.lse = b.dlogp = b.grad = 0x9000
    b.grad_stride_b, b.grad_stride_l = 32 * 1024, 1024
    for field, value in (("grad", None), ("lse", None), ("dlogp", None), ("grad_stride_l", 100), ("V", 0)):
        bad = pkg.fork_logprob_bwd_args.from_buffer_copy(b)
        setattr(bad, field, value)
        assert L.fork_logprob_backward(C.byref(bad), ws, nbytes, None) == INV, field
    assert L.fork_logprob_backward(C.byref(b), ws, 16, None) == pkg.FORK_ERR_WORKSPACE
    # the step fused into the LM-head product
    hd = pkg.fork_head_args()
    hd.hidden, hd.weight, hd.d, hd.hidden_stride, hd.weight_stride = 0x20000, 0x40000, 256, 256, 256
    a = good_step_args()
    assert L.fork_step_fused_head(None, C.byref(hd), ws, nbytes, None) == INV
    assert L.fork_step_fused_head(C.byref(a), None, ws, nbytes, None) == INV
    for field, value in (("hidden", None), ("weight", None), ("d", 0), ("d", 100), ("hidden_stride", 64), ("weight_stride", 64),
                         ("hidden_stride", 260), ("hidden", 0x20008)):   # d must be a multiple of 64; rows 16-byte aligned
        bad = pkg.fork_head_args.from_buffer_copy(hd)
        setattr(bad, field, value)
        assert L.fork_step_fused_head(C.byref(a), C.byref(bad), ws, nbytes, None) == INV, field
    a.temperature = 0.8                                                   # drawn candidates need their scratch
    assert L.fork_step_fused_head(C.byref(a), C.byref(hd), ws, nbytes, None) == pkg.FORK_ERR_WORKSPACE
    a.sample_scratch, a.sample_scratch_bytes = 0x80000, L.fork_head_sample_scratch_bytes(a.B, a.Ll, a.V) - 1
    assert L.fork_step_fused_head(C.byref(a), C.byref(hd), ws, nbytes, None) == pkg.FORK_ERR_WORKSPACE
    a.temperature = -1.0
    assert L.fork_step_fused_head(C.byref(a), C.byref(hd), ws, nbytes, None) == INV
    assert L.fork_head_sample_scratch_bytes(8, 32, 126464) == 2 * 3952 * 256 * 4 + 3952 * 256 + 256 * 16 + 256 * 256 * 4
    a = good_step_args()
    cb = pkg.binding.fork_logits_fn(lambda *x: 0)
    fn = C.cast(cb, C.c_void_p)
    n = C.c_int32(7)
    loop = L.fork_decode_loop_fused_head
    assert loop(C.byref(a), C.byref(hd), 8, 0, 32, None, None, 10, C.byref(n), ws, nbytes, None) == INV and n.value == 0   # no provider
    assert loop(C.byref(a), None, 8, 0, 32, fn, None, 10, C.byref(n), ws, nbytes, None) == INV
    assert loop(C.byref(a), C.byref(hd), 0, 0, 32, fn, None, 10, C.byref(n), ws, nbytes, None) == INV          # block length
    assert loop(C.byref(a), C.byref(hd), a.Ll + 1, 0, 32, fn, None, 10, C.byref(n), ws, nbytes, None) == INV   # block longer than the window
    assert loop(C.byref(a), C.byref(hd), 8, 0, a.Lt + 1, fn, None, 10, C.byref(n), ws, nbytes, None) == INV
    assert loop(C.byref(a), C.byref(hd), 8, 0, 32, fn, None, -1, C.byref(n), ws, nbytes, None) == INV
    assert loop(C.byref(a), C.byref(hd), 8, 0, 32, fn, None, 10, C.byref(n), ws, 16, None) == pkg.FORK_ERR_WORKSPACE
    a = good_step_args()
    assert L.fork_step_fused_head(C.byref(a), C.byref(hd), ws, 16, None) == pkg.FORK_ERR_WORKSPACE
    f = pkg.fork_grpo_fused_args()
    f.logits = 0x1000
    f.stride_b, f.stride_l = 32 * 1024, 1024
    f.B, f.Lt, f.V, f.dtype, f.group = 4, 32, 1024, pkg.FORK_F32, 2
    f.tokens = f.select = f.logp_old = f.reward = f.grad = f.logp = f.seq_obj = 0x9000
    f.grad_stride_b, f.grad_stride_l = 32 * 1024, 1024
    f.eps_lo = f.eps_hi = 0.2
    for field, value in (("grad", None), ("logp", None), ("seq_obj", None), ("reward", None), ("logp_old", None), ("group", 3),
                         ("group", 0), ("grad_stride_l", 100), ("V", 0), ("eps_hi", float("nan")), ("dtype", 7)):
        bad = pkg.fork_grpo_fused_args.from_buffer_copy(f)
        setattr(bad, field, value)
        assert L.fork_grpo_fused(C.byref(bad), ws, nbytes, None) == INV, field
    assert L.fork_grpo_fused(None, ws, nbytes, None) == INV
    assert L.fork_grpo_fused(C.byref(f), ws, 16, None) == pkg.FORK_ERR_WORKSPACE
