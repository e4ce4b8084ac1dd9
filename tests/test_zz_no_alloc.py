"""fork_step_static: the step for callers that cannot allocate device memory (for instance a
server whose own pool already holds the whole device, or a latency-critical path that must not hit
cudaMalloc's implicit synchronisation).  It runs on a fixed scratch array inside the library.  The
checks: it gives what the fp64 oracle gives and what fork_step gives -- on two calls in a row,
because the second call finds the scratch as the first one left it --, both when the batch is small
enough for the one-kernel step and when it takes the set-up kernel first; a warm call leaves the
amount of free device memory where it was and asks torch's allocator for nothing; and the device status word of such a call can
be read although the caller has no workspace pointer to ask with.  Kept in a file that pytest
collects last."""
import ctypes as C
import gc

import numpy as np
import pytest
import torch

import fork_synth as fs
import oracle
from helpers import assert_close, assert_equal, compare_step_state

pytestmark = pytest.mark.gpu


def _inputs(rng, B, Lt, V):
    x = (rng.standard_normal((B, Lt, V)) * 3).astype(np.float32)
    peaks = rng.integers(0, V, size=(B, Lt))
    x[np.arange(B)[:, None], np.arange(Lt)[None, :], peaks] += rng.uniform(8, 22, size=(B, Lt)).astype(np.float32)
    return fs.f32_to_bf16_bits(x)


def _free_bytes():
    free, _ = torch.cuda.mem_get_info()
    return free


def _allocations():
    """Number of allocation requests torch's caching allocator has served so far (frees do not
    lower it, so objects of earlier tests that the garbage collector happens to drop do not matter)."""
    return torch.cuda.memory_stats().get("allocation.all.allocated", 0)


@pytest.mark.parametrize("B,Lt,V,kernels", [(6, 48, 20000, 1), (300, 64, 2056, 2)])
def test_static_scratch_step_matches_oracle_and_fork_step_twice_in_a_row(B, Lt, V, kernels):
    import paper_2609_39859_b200 as pkg
    rng = np.random.default_rng(2609 + B)
    assert pkg.fork_workspace_bytes(B, Lt) <= pkg.FORK_STATIC_SCRATCH_BYTES
    lo_h = (rng.integers(0, 3, size=B) * 16).astype(np.int32)
    hi_h = (lo_h + 16).astype(np.int32)
    hi_h[-1] = lo_h[-1]                                # the last sequence sits out
    lo, hi = torch.from_numpy(lo_h).cuda(), torch.from_numpy(hi_h).cuda()
    mask0 = (rng.random((B, Lt)) < 0.8).astype(np.uint8)
    ref = pkg.ForkState(B, Lt, mask=mask0)            # fork_step: caller-provided workspace
    got = pkg.ForkState(B, Lt, mask=mask0)            # fork_step_static: no workspace used
    want = oracle.StepState(B, Lt, mask=mask0)
    for call in range(2):                             # the second call starts from the first one's state
        bits = _inputs(rng, B, Lt, V)
        logits = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
        assert oracle.step(want, bits, lo_h, hi_h, 0.9, step_id=call) == 0
        pkg.fork_step(ref, logits, lo, hi, 0.9, step=call)
        torch.cuda.synchronize()
        gc.collect()
        n0, free0, alloc0 = pkg.fork_kernel_launches(), _free_bytes(), _allocations()
        pkg.fork_step_static(got, logits, lo, hi, 0.9, step=call)
        torch.cuda.synchronize()
        assert pkg.fork_kernel_launches() - n0 == kernels       # one-kernel step, or set-up kernel + streaming kernel
        if call == 1:                                           # a warm call: nothing was allocated, by anybody
            assert _free_bytes() >= free0 and _allocations() == alloc0
        assert pkg.fork_device_status(None) == 0                # the static call's own status word
        r, g = ref.host(), got.host()
        assert int(r["n_unmasked"].sum()) > 0
        compare_step_state(g, want)                             # integers bit-exact, floats within 1e-5 + 1e-4 |oracle|
        for name in ("tokens", "mask", "cand", "commit_step", "commit_fallback", "row_status",
                     "n_unmasked", "is_fallback", "fallback_pos", "nfe", "n_fallback"):
            assert_equal(name, g[name], r[name])
        for name in ("conf", "entropy", "logp", "commit_logp"):
            assert_close(name, g[name], r[name])
    assert int(got.host()["nfe"].max()) == 2


def test_static_scratch_rejects_batches_beyond_its_limit():
    import paper_2609_39859_b200 as pkg
    L = pkg.lib()
    B, Lt = 512, 1024                                  # needs far more than the 2 MiB built in
    assert pkg.fork_workspace_bytes(B, Lt) > pkg.FORK_STATIC_SCRATCH_BYTES
    a = pkg.fork_step_args()
    a.logits = 0x1000
    a.stride_b, a.stride_l, a.pos0 = Lt * 1024, 1024, 0
    a.B, a.Lt, a.Ll, a.V, a.dtype = B, Lt, Lt, 1024, pkg.FORK_BF16
    a.tokens, a.mask, a.blk_lo, a.blk_hi = 0x2000, 0x3000, 0x4000, 0x5000
    a.threshold = 0.9
    assert L.fork_step_static(C.byref(a), None) == pkg.FORK_ERR_WORKSPACE
    assert pkg.fork_status_string(pkg.FORK_ERR_WORKSPACE) == "FORK_ERR_WORKSPACE"
    a.mask = None
    assert L.fork_step_static(C.byref(a), None) == pkg.FORK_ERR_INVALID_ARG
