"""fork_step_static: the step for callers that cannot allocate device memory (for instance a
server whose own pool already holds the whole device, or a latency-critical path that must not hit
cudaMalloc's implicit synchronisation).  It runs on a fixed scratch array inside the library, so
the check is simply that it gives what fork_step gives -- on two calls in a row, because the second
call finds the scratch as the first one left it.  Kept in a file that pytest collects last."""
import ctypes as C

import numpy as np
import pytest
import torch

import fork_synth as fs
from helpers import assert_close, assert_equal

pytestmark = pytest.mark.gpu


def test_static_scratch_step_matches_fork_step_twice_in_a_row():
    import paper_2609_39859_b200 as pkg
    rng = np.random.default_rng(2609)
    B, Lt, V = 6, 48, 20000
    lo = torch.tensor([0, 0, 16, 16, 32, 8], dtype=torch.int32, device="cuda")
    hi = torch.tensor([16, 16, 32, 32, 48, 8], dtype=torch.int32, device="cuda")      # the last sequence sits out
    mask0 = (rng.random((B, Lt)) < 0.8).astype(np.uint8)
    ref = pkg.ForkState(B, Lt, mask=mask0)            # fork_step: caller-provided workspace
    got = pkg.ForkState(B, Lt, mask=mask0)            # fork_step_static: no workspace used
    for call in range(2):                             # the second call starts from the first one's state
        x = (rng.standard_normal((B, Lt, V)) * 3).astype(np.float32)
        peaks = rng.integers(0, V, size=(B, Lt))
        x[np.arange(B)[:, None], np.arange(Lt)[None, :], peaks] += rng.uniform(8, 22, size=(B, Lt)).astype(np.float32)
        logits = torch.from_numpy(fs.f32_to_bf16_bits(x).view(np.int16)).cuda().view(torch.bfloat16)
        pkg.fork_step(ref, logits, lo, hi, 0.9, step=call)
        pkg.fork_step_static(got, logits, lo, hi, 0.9, step=call)
        torch.cuda.synchronize()
        r, g = ref.host(), got.host()
        assert int(r["n_unmasked"].sum()) > 0
        for name in ("tokens", "mask", "cand", "commit_step", "commit_fallback", "row_status",
                     "n_unmasked", "is_fallback", "fallback_pos", "nfe", "n_fallback"):
            assert_equal(name, g[name], r[name])
        for name in ("conf", "entropy", "logp", "commit_logp"):
            assert_close(name, g[name], r[name])      # |g - r| <= 1e-5 + 1e-4 |r|, NaN where never written
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
