"""The five benchmark configurations on the GPU against the oracle: the device generator is
bit-identical to the host generator, so the oracle regenerates exactly the rows the kernels saw.
Whole decode loops are compared sequence by sequence (sequences are independent); at the full
batch sizes a prefix of the sequences is checked exactly and the rest through invariants."""
import math

import numpy as np
import pytest
import torch

import fork_synth as fs
import oracle
from helpers import (assert_close, assert_equal, compare_step_state, live_mask, oracle_reference_loop)

pytestmark = pytest.mark.gpu


def F():
    import paper_2609_39859_b200 as pkg
    return pkg


def torch_dtype(w):
    return torch.bfloat16 if w.dtype == fs.BF16 else torch.float32


def device_logits(w, B, Ll=None, canary=True):
    Ll = w.Lt if Ll is None else Ll
    t = torch.empty((B, Ll, w.V), dtype=torch_dtype(w), device="cuda")
    if canary:
        fs.cuda_canary(t.data_ptr(), t.numel(), w.dtype, torch.cuda.current_stream().cuda_stream)
    return t


def gpu_loop(w, threshold, nonces=None, max_steps=100000, B=None, raise_on_error=True, fail_at=None):
    pkg = F()
    B = w.B if B is None else B
    cfg = w.cfg(B=B)
    logits = device_logits(w, B)
    st = pkg.ForkState(B, w.Lt)
    prov = fs.Provider(cfg, w.Lt * w.V, w.V, 0, w.Lt, nonce=nonces)
    if fail_at is not None:
        prov.fail_at(fail_at)
    rc, steps = pkg.fork_decode_loop(st, logits, w.block_len, 0, w.Lt, prov.address, prov.ctx, threshold,
                                     max_steps, raise_on_error=raise_on_error)
    torch.cuda.synchronize()
    calls = prov.calls
    prov.close()
    return rc, steps, calls, st.host()


def check_loop_invariants(h, w, steps):
    """Properties that hold for every sequence at any size (Algorithm 2 and Section 3.2)."""
    B, Lt = h["mask"].shape
    assert (h["mask"] == 0).all()
    assert (h["commit_step"] >= 0).all() and (h["commit_step"] < steps).all()
    assert steps == h["nfe"].max()
    fb = h["commit_fallback"]
    assert set(np.unique(fb)) <= {0, 1}
    assert_equal("n_fallback", h["n_fallback"], fb.sum(1))          # one token per fallback step
    for b in range(B):
        cs = h["commit_step"][b]
        assert len(np.unique(cs)) == h["nfe"][b]                    # every step of the sequence commits something
        fsteps = cs[fb[b] == 1]
        assert len(np.unique(fsteps)) == len(fsteps)                # exactly one commit at a fallback step
        for s in fsteps:                                            # ... and it is the leftmost still-masked position
            k = int(np.flatnonzero((cs == s))[0])
            blk = (k // w.block_len) * w.block_len
            assert (cs[blk:k] < s).all()
    assert (h["tokens"] == h["cand"]).all()
    lp_ok = np.abs(h["commit_logp"] - np.log(h["conf"])) <= 1e-5 + 1e-4 * np.abs(h["commit_logp"])
    assert lp_ok.all()


def test_device_generator_is_bit_identical_to_host_generator():
    for name in ("tiny", "b8", "passk", "grpo"):
        w = fs.workload(name)
        for wl in (w, w.literal()):
            B = min(w.B, 2)
            cfg = wl.cfg(B=B)
            Ll = 6
            t = device_logits(wl, B, Ll=Ll)
            mask = np.ones((B, wl.Lt), np.uint8)
            mask[0, 2] = 0
            lo, hi = np.zeros(B, np.int32), np.full(B, Ll, np.int32)
            mask_d, lo_d, hi_d = (torch.from_numpy(a).cuda() for a in (mask, lo, hi))   # kept alive until the sync
            fs.cuda_fill(cfg, 3, mask_d.data_ptr(), lo_d.data_ptr(), hi_d.data_ptr(), t.data_ptr(), Ll * wl.V, wl.V,
                         0, Ll, nonce=5)
            torch.cuda.synchronize()
            got = (t.view(torch.int16) if wl.dtype == fs.BF16 else t).cpu().numpy()
            got = got.view(np.uint16) if wl.dtype == fs.BF16 else got
            for b in range(B):
                for l in range(Ll):
                    if mask[b, l]:
                        assert (got[b, l] == fs.row_host(cfg, 3, b, l, nonce=5)).all(), (name, b, l)
                    else:
                        assert (got[b, l] == 0x7FC0).all() if wl.dtype == fs.BF16 else np.isnan(got[b, l]).all()


def test_tiny_one_step_and_full_loop_byte_for_byte():
    pkg = F()
    w = fs.workload("tiny")
    ost, nonces, osteps, _ = oracle_reference_loop(w, w.B, w.threshold)
    rc, steps, calls, h = gpu_loop(w, w.threshold, nonces)
    assert rc == 0 and steps == osteps == calls
    compare_step_state(h, ost)
    check_loop_invariants(h, w, steps)
    # a single step from the all-masked state
    cfg = w.cfg()
    x = np.empty((w.B, w.Lt, w.V), np.float32)
    mask = np.ones((w.B, w.Lt), np.uint8)
    lo, hi = np.zeros(w.B, np.int32), np.full(w.B, w.Lt, np.int32)
    fs.fill_host(cfg, 0, mask, lo, hi, x, nonce=int(nonces[0]))
    o = oracle.StepState(w.B, w.Lt)
    oracle.step(o, x, lo, hi, w.threshold)
    g = pkg.ForkState(w.B, w.Lt)
    pkg.fork_step(g, torch.from_numpy(x).cuda(), torch.from_numpy(lo).cuda(), torch.from_numpy(hi).cuda(), w.threshold)
    compare_step_state(g.host(), o)


@pytest.mark.parametrize("variant", ["calibrated", "literal"])
def test_b8_full_decode_loop(variant):
    w = fs.workload("b8")
    nseq = w.B
    if variant == "literal":
        w, nseq = w.literal(), 2
    ost, nonces, osteps, _ = oracle_reference_loop(w, nseq, w.threshold)
    rc, steps, calls, h = gpu_loop(w, w.threshold, nonces)
    assert rc == 0 and steps == calls and steps >= osteps
    compare_step_state(h, ost, nseq=nseq, last_step_outputs=(steps == osteps))
    check_loop_invariants(h, w, steps)
    if variant == "literal":            # almost nothing clears 0.9: close to pure left-to-right decoding
        assert steps > 0.8 * w.Lt and h["commit_fallback"].mean() > 0.8
    else:
        assert steps == osteps and 40 <= steps < w.Lt
        frac = h["commit_fallback"].mean()
        assert 0.15 < frac < 0.45, frac


def test_passk_decode_loop_every_sequence_exact():
    w = fs.workload("passk")
    nseq = w.B                               # all 64 sequences against the oracle (about 16,000 rows of fp64 work)
    ost, nonces, osteps, _ = oracle_reference_loop(w, nseq, w.threshold)
    rc, steps, calls, h = gpu_loop(w, w.threshold, nonces)
    assert rc == 0 and steps == calls
    compare_step_state(h, ost, nseq=nseq, last_step_outputs=(steps == osteps))
    check_loop_invariants(h, w, steps)
    assert steps < w.Lt                      # parallel decoding: fewer model evaluations than tokens
    assert 0.05 < h["commit_fallback"].mean() < 0.16
    # fork rows (exact or one-ulp ties in bf16) resolved to the lowest index of the maximum
    cfg = w.cfg()
    checked = 0
    for b in range(0, w.B, 7):
        for l in range(0, w.Lt, 5):
            p = fs.plan_host(cfg, b, l)
            if p["is_fork"]:
                cs = int(h["commit_step"][b, l])
                row = fs.row_host(cfg, cs, b, l, nonce=int(nonces[cs]) if cs < len(nonces) else 0)
                s = oracle.row_stats(row)
                assert h["tokens"][b, l] == s["cand"]
                assert_close("conf", h["conf"][b, l], s["conf"])
                assert_close("entropy", h["entropy"][b, l], s["entropy"])
                checked += 1
    assert checked >= 5


@pytest.mark.parametrize("lam", [0.5, 0.7, 0.9, 0.95, 0.99])
def test_sweep_decode_loop(lam):
    w = fs.workload("sweep")
    nseq = 8 if lam in (0.7, 0.95) else 1    # eight sequences exactly at two thresholds, one at the others, the rest by invariants
    ost, nonces, osteps, _ = oracle_reference_loop(w, nseq, lam)
    rc, steps, calls, h = gpu_loop(w, lam, nonces)
    assert rc == 0 and steps == calls
    compare_step_state(h, ost, nseq=nseq, last_step_outputs=(steps == osteps))
    check_loop_invariants(h, w, steps)


def test_full_block_step_at_benchmark_shapes_sampled_rows():
    """The launch the benchmark times (every position of one block live) at B=8 and B=64:
    sampled rows against the oracle, every sequence through the unmask rule's invariants."""
    pkg = F()
    rng = np.random.default_rng(1)
    for name in ("b8", "passk", "sweep"):
        w = fs.workload(name)
        cfg = w.cfg()
        BL = w.block_len
        t = device_logits(w, w.B, Ll=BL)                      # block-window logits, pos0 = first block
        st = pkg.ForkState(w.B, w.Lt)
        lo = torch.zeros(w.B, dtype=torch.int32, device="cuda")
        hi = torch.full((w.B,), BL, dtype=torch.int32, device="cuda")
        fs.cuda_fill(cfg, 0, st.mask.data_ptr(), lo.data_ptr(), hi.data_ptr(), t.data_ptr(), BL * w.V, w.V, 0, BL)
        pkg.fork_step(st, t, lo, hi, w.threshold, step=0)
        torch.cuda.synchronize()
        h = st.host()
        conf = h["conf"][:, :BL]
        for b in range(w.B):
            above = conf[b] > np.float32(w.threshold)
            want = above if above.any() else (np.arange(BL) == 0)
            assert ((h["mask"][b, :BL] == 0) == want).all()
            assert h["is_fallback"][b] == (0 if above.any() else 1)
            assert h["n_unmasked"][b] == want.sum()
            assert (h["mask"][b, BL:] == 1).all() and np.isnan(h["conf"][b, BL:]).all()
        for _ in range(24):
            b, l = int(rng.integers(0, w.B)), int(rng.integers(0, BL))
            s = oracle.row_stats(fs.row_host(cfg, 0, b, l))
            assert h["cand"][b, l] == s["cand"]
            assert_close("conf", h["conf"][b, l], s["conf"])
            assert_close("entropy", h["entropy"][b, l], s["entropy"])
            assert_close("logp", h["logp"][b, l], s["logp"])
            assert abs(s["conf"] - w.threshold) >= 1e-4


def test_grpo_scoring_full_size_sampled_rows():
    pkg = F()
    w = fs.workload("grpo")
    cfg = w.cfg()
    tokens, select = fs.scoring_inputs(w, cfg)
    t = device_logits(w, w.B)                                 # 16.6 GB of fp32, NaN except the selected rows
    sel_d = torch.from_numpy(select).cuda()
    fs.cuda_fill(cfg, 0, sel_d.data_ptr(), None, None, t.data_ptr(), w.Lt * w.V, w.V, 0, w.Lt)
    st = pkg.ForkState(w.B, w.Lt)
    lp, ssum, scnt, status = pkg.fork_logprob(t, torch.from_numpy(tokens).cuda(), sel_d, st)
    torch.cuda.synchronize()
    lp, ssum, scnt, status = lp.cpu().numpy(), ssum.cpu().numpy(), scnt.cpu().numpy(), status.cpu().numpy()
    assert_equal("seq_cnt", scnt, select.sum(1))
    assert (status == 0).all() and (lp[select == 0] == 0).all()
    assert 0.15 < select.mean() < 0.25
    rng = np.random.default_rng(2)
    bs, ks = np.nonzero(select)
    for i in rng.choice(len(bs), size=40, replace=False):
        b, k = int(bs[i]), int(ks[i])
        want, st_o = oracle.row_logp(fs.row_host(cfg, 0, b, k), int(tokens[b, k]))
        assert st_o == 0
        assert_close("logp", lp[b, k], want)
    for b in (0, 77):                                         # per-sequence sums, fully
        want = sum(oracle.row_logp(fs.row_host(cfg, 0, b, int(k)), int(tokens[b, k]))[0]
                   for k in np.flatnonzero(select[b]))
        assert_close("seq_sum", ssum[b], want)
    assert_close("seq_sum vs logp", ssum, lp.astype(np.float64).sum(1))


def test_decode_loop_error_paths_and_python_provider():
    pkg = F()
    w = fs.workload("tiny")
    rc, steps, calls, h = gpu_loop(w, 1.0, max_steps=5, raise_on_error=False)
    assert rc == pkg.FORK_ERR_MAX_STEPS and steps == 5 and h["mask"].sum() == w.Lt - 5
    assert h["commit_step"][0, :5].tolist() == [0, 1, 2, 3, 4]      # threshold 1.0: left to right
    rc, steps, calls, h = gpu_loop(w, 1.0, raise_on_error=False, fail_at=3)
    assert rc == pkg.FORK_ERR_PROVIDER and steps == 3 and h["mask"].sum() == w.Lt - 3
    with pytest.raises(pkg.ForkError):
        gpu_loop(w, 1.0, max_steps=2)
    # a Python callable as the model: same result as the C provider
    cfg = w.cfg()
    logits = device_logits(w, w.B)
    st = pkg.ForkState(w.B, w.Lt)

    def model(step, lo_ptr, hi_ptr, stream_ptr):
        fs.cuda_fill(cfg, step, st.mask.data_ptr(), lo_ptr, hi_ptr, logits.data_ptr(), w.Lt * w.V, w.V, 0, w.Lt,
                     stream_ptr=stream_ptr)
        return 0
    rc, steps = pkg.fork_decode_loop(st, logits, w.block_len, 0, w.Lt, model, None, w.threshold, 1000)
    rc2, steps2, _, h2 = gpu_loop(w, w.threshold)
    assert rc == 0 and steps == steps2
    h1 = st.host()
    for name in h1:
        assert h1[name].tobytes() == h2[name].tobytes(), name


def test_loop_that_runs_ahead_of_the_outcomes_gives_the_same_bytes():
    """With FORK_TUNE_LOOP_AHEAD the host enqueues model calls and steps before it has read the
    outcome of the earlier ones; the steps enqueued after the batch was complete must find nothing
    to do and change nothing (not even the per-sequence evaluation counts)."""
    pkg = F()
    for name, B in (("tiny", None), ("b8", 3)):
        w = fs.workload(name)
        rc0, steps0, calls0, h0 = gpu_loop(w, w.threshold, B=B)
        assert rc0 == 0 and calls0 == steps0
        for ahead in (1, 4, 6):
            old = pkg.fork_set_tuning(pkg.FORK_TUNE_LOOP_AHEAD, ahead)
            try:
                rc, steps, calls, h = gpu_loop(w, w.threshold, B=B)
            finally:
                pkg.fork_set_tuning(pkg.FORK_TUNE_LOOP_AHEAD, old)
            assert rc == 0 and steps == steps0 and steps0 <= calls <= steps0 + ahead
            for key in h:                    # (the three per-sequence outputs that describe the LAST step enqueued are those of an empty step)
                if calls == steps0 or key not in ("n_unmasked", "is_fallback", "fallback_pos"):
                    assert h[key].tobytes() == h0[key].tobytes(), (name, ahead, key)
        # the step limit and a failing model call behave as without look-ahead
        old = pkg.fork_set_tuning(pkg.FORK_TUNE_LOOP_AHEAD, 4)
        try:
            rc, steps, calls, h = gpu_loop(w, 1.0, max_steps=5, B=B, raise_on_error=False)
            assert rc == pkg.FORK_ERR_MAX_STEPS and steps == 5 and calls == 5
            assert int((h["commit_step"] >= 0).sum()) == 5 * h["mask"].shape[0]
            rc, steps, calls, h = gpu_loop(w, 1.0, B=B, raise_on_error=False, fail_at=3)
            assert rc == pkg.FORK_ERR_PROVIDER and steps == 3
        finally:
            pkg.fork_set_tuning(pkg.FORK_TUNE_LOOP_AHEAD, old)


def test_loop_resumes_from_its_buffers():
    """State is only the caller's buffers: stopping at max_steps and calling again continues."""
    pkg = F()
    w = fs.workload("tiny")
    rc_full, steps_full, _, h_full = gpu_loop(w, w.threshold)
    cfg = w.cfg()
    logits = device_logits(w, w.B)
    st = pkg.ForkState(w.B, w.Lt)
    prov = fs.Provider(cfg, w.Lt * w.V, w.V, 0, w.Lt)
    rc, s1 = pkg.fork_decode_loop(st, logits, w.block_len, 0, w.Lt, prov.address, prov.ctx, w.threshold, 3,
                                  raise_on_error=False)
    assert rc == pkg.FORK_ERR_MAX_STEPS and s1 == 3
    rc, s2 = pkg.fork_decode_loop(st, logits, w.block_len, 0, w.Lt, prov.address, prov.ctx, w.threshold, 1000, step0=3)
    assert rc == 0 and s1 + s2 == steps_full
    h = st.host()
    for name in h:
        assert h[name].tobytes() == h_full[name].tobytes(), name


def test_sampled_full_block_step_at_the_pass_at_k_shape():
    """The launch the benchmark times with --temperature 0.8 (B=64, every position of a block live):
    the first two sequences exactly against the oracle (inputs re-drawn until its decisions are
    clear), every sequence through invariants of the drawn candidates."""
    from helpers import decisions_are_clear
    pkg = F()
    w = fs.workload("passk")
    BL, tau, seed, nseq = w.block_len, 0.8, 4711, 2
    cfg_small = w.cfg(B=nseq)
    lo_h, hi_h = np.zeros(nseq, np.int32), np.full(nseq, BL, np.int32)
    for nonce in range(16):
        x = np.empty((nseq, BL, w.V), np.uint16)
        for b in range(nseq):
            for l in range(BL):
                x[b, l] = fs.row_host(cfg_small, 0, b, l, nonce=nonce)
        o = oracle.StepState(nseq, w.Lt)
        assert oracle.step(o, x, lo_h, hi_h, w.threshold, step_id=0, temperature=tau, sample_seed=seed) == 0
        if decisions_are_clear(o, live_mask(np.ones((nseq, w.Lt), np.uint8), lo_h, hi_h), w.threshold, 1e-4, 0, tau):
            break
    else:
        raise AssertionError("no nonce with clear margins")
    cfg = w.cfg()
    t = device_logits(w, w.B, Ll=BL)
    st = pkg.ForkState(w.B, w.Lt)
    lo = torch.zeros(w.B, dtype=torch.int32, device="cuda")
    hi = torch.full((w.B,), BL, dtype=torch.int32, device="cuda")
    fs.cuda_fill(cfg, 0, st.mask.data_ptr(), lo.data_ptr(), hi.data_ptr(), t.data_ptr(), BL * w.V, w.V, 0, BL, nonce=nonce)
    pkg.fork_step(st, t, lo, hi, w.threshold, step=0, temperature=tau, sample_seed=seed)
    torch.cuda.synchronize()
    h = st.host()
    compare_step_state(h, o, nseq=nseq)
    conf, logp = h["conf"][:, :BL], h["logp"][:, :BL]
    assert ((conf > 0) & (conf <= 1.0 + 1e-6)).all()
    assert (np.abs(np.log(conf) - logp) <= 1e-5 + 1e-4 * np.abs(logp)).all()       # both describe the drawn token
    committed = h["mask"][:, :BL] == 0
    assert (h["tokens"][:, :BL][committed] == h["cand"][:, :BL][committed]).all()
    for b in range(w.B):
        above = conf[b] > np.float32(w.threshold)
        want = above if above.any() else (np.arange(BL) == 0)
        assert (committed[b] == want).all()
    # a drawn token is not always the arg-max: some candidates differ from the greedy step's
    st2 = pkg.ForkState(w.B, w.Lt)
    pkg.fork_step(st2, t, lo, hi, w.threshold, step=0)
    torch.cuda.synchronize()
    assert (st2.host()["cand"][:, :BL] != h["cand"][:, :BL]).any()


def test_grpo_training_chain_full_size_sampled_rows():
    """Scoring -> Eq. 2 -> log-softmax backward at B=128, Lt=256, V=126464 fp32 (16.6 GB of logits and
    as much gradient): the objective on the whole batch, gradients on sampled rows."""
    pkg = F()
    w = fs.workload("grpo")
    cfg = w.cfg()
    tokens, select = fs.scoring_inputs(w, cfg)
    t = device_logits(w, w.B)
    sel_d, tok_d = torch.from_numpy(select).cuda(), torch.from_numpy(tokens).cuda()
    fs.cuda_fill(cfg, 0, sel_d.data_ptr(), None, None, t.data_ptr(), w.Lt * w.V, w.V, 0, w.Lt)
    st = pkg.ForkState(w.B, w.Lt)
    lp, ssum, scnt, status, lse = pkg.fork_logprob(t, tok_d, sel_d, st, want_lse=True)
    gen = torch.Generator(device="cuda").manual_seed(5)
    old = ((lp + 0.1 * torch.randn(lp.shape, device="cuda", generator=gen)) * (sel_d != 0)).contiguous()
    reward = (torch.rand(w.B, device="cuda", generator=gen) < 0.4).float()
    reward[:8] = 1.0                                              # one prompt group with equal rewards
    out = pkg.fork_grpo_loss(lp, old, sel_d, reward, 8, 0.2, 0.2)
    grad = torch.empty_like(t)
    fs.cuda_canary(grad.data_ptr(), grad.numel(), w.dtype, torch.cuda.current_stream().cuda_stream)
    pkg.fork_logprob_backward(t, tok_d, sel_d, lse, out["dlogp"], grad, st)
    torch.cuda.synchronize()
    o = oracle.grpo_loss(lp.cpu().numpy(), old.cpu().numpy(), select, reward.cpu().numpy(), 8, 0.2, 0.2)
    rho = o["ratio"][select != 0]
    near = (np.abs(rho - 0.8) < 1e-4) | (np.abs(rho - 1.2) < 1e-4)
    d = out["dlogp"].cpu().numpy()
    ok = np.abs(d - o["dlogp"]) <= 1e-9 + 1e-4 * np.abs(o["dlogp"])
    assert ok[select != 0][~near].all() and (d[select == 0] == 0).all() and (d[:8] == 0).all()
    assert abs(float(out["objective"].cpu()[0]) - o["objective"]) <= 1e-6 + 1e-4 * abs(o["objective"])
    assert o["skipped"][0] == 1 and out["skipped"].cpu().numpy()[0] == 1
    rng = np.random.default_rng(4)
    bs, ks = np.nonzero(select[8:])                               # rollouts with a non-zero advantage
    lse_h = lse.cpu().numpy()
    for i in rng.choice(len(bs), size=4, replace=False):
        b, k = int(bs[i]) + 8, int(ks[i])
        row = fs.row_host(cfg, 0, b, k)
        assert abs(lse_h[b, k] - oracle.row_lse(row)) <= 1e-5 + 1e-5 * abs(lse_h[b, k])
        want = oracle.row_logp_grad(row, int(tokens[b, k]), float(d[b, k]))
        got = grad[b, k].cpu().numpy().astype(np.float64)
        assert (np.abs(got - want) <= 2e-6 * abs(float(d[b, k])) + 1e-4 * np.abs(want)).all()
    b, k = map(int, np.argwhere(select == 0)[123])
    assert torch.isnan(grad[b, k]).all()                          # rows of unselected positions keep the canary


def test_grpo_fused_pass_full_size_sampled_rows():
    """fork_grpo_fused in the configuration bench.py times (B=128, Lt=256, V=126464 fp32, 6496 selected rows,
    16.6 GB of logits and as much gradient): log-probabilities and gradient rows of sampled positions against the
    oracle, Eq. 2 on the whole batch against the oracle on the call's own log-probabilities, canaries in every
    sampled row it must not touch."""
    pkg = F()
    w = fs.workload("grpo")
    cfg = w.cfg()
    tokens, select = fs.scoring_inputs(w, cfg)
    t = device_logits(w, w.B)
    sel_d, tok_d = torch.from_numpy(select).cuda(), torch.from_numpy(tokens).cuda()
    fs.cuda_fill(cfg, 0, sel_d.data_ptr(), None, None, t.data_ptr(), w.Lt * w.V, w.V, 0, w.Lt)
    st = pkg.ForkState(w.B, w.Lt)
    rng = np.random.default_rng(6)
    bs, ks = np.nonzero(select)
    picks = [(int(bs[i]), int(ks[i])) for i in rng.choice(len(bs), size=24, replace=False)]
    old_h = np.zeros(select.shape, np.float32)
    want_lp = {}
    for b in range(w.B):                                          # old-policy log-probabilities near the new ones
        for k in np.flatnonzero(select[b]):
            old_h[b, k] = -2.0
    for b, k in picks:
        want_lp[(b, k)] = oracle.row_logp(fs.row_host(cfg, 0, b, k), int(tokens[b, k]))[0]
        old_h[b, k] = np.float32(want_lp[(b, k)] + 0.05 * rng.standard_normal())
    gen = torch.Generator(device="cuda").manual_seed(9)
    reward = (torch.rand(w.B, device="cuda", generator=gen) < 0.4).float()
    reward[:8] = 1.0                                              # one prompt group with equal rewards
    grad = torch.empty_like(t)
    fs.cuda_canary(grad.data_ptr(), grad.numel(), w.dtype, torch.cuda.current_stream().cuda_stream)
    out = pkg.fork_grpo_fused(t, tok_d, sel_d, torch.from_numpy(old_h).cuda(), reward, 8, 0.2, 0.2, grad, st)
    torch.cuda.synchronize()
    assert pkg.fork_device_status(st) == 0
    h = {k: v.cpu().numpy() for k, v in out.items()}
    assert (h["row_status"][select != 0] == 0).all()
    for (b, k), want in want_lp.items():
        assert_close("logp", h["logp"][b, k], want)
    o = oracle.grpo_loss(h["logp"], old_h, select, reward.cpu().numpy(), 8, 0.2, 0.2)
    rho = o["ratio"][select != 0]
    near = (np.abs(rho - 0.8) < 1e-4) | (np.abs(rho - 1.2) < 1e-4)
    ok = np.abs(h["dlogp"] - o["dlogp"]) <= 1e-9 + 1e-4 * np.abs(o["dlogp"])
    assert ok[select != 0][~near].all() and (h["dlogp"][:8][select[:8] != 0] == 0).all()
    assert abs(float(h["objective"][0]) - o["objective"]) <= 1e-6 + 1e-4 * abs(o["objective"])
    assert o["skipped"][0] == 1 and h["skipped"][0] == 1
    for b, k in picks:
        row = fs.row_host(cfg, 0, b, k)
        d = float(h["dlogp"][b, k])
        want = oracle.row_logp_grad(row, int(tokens[b, k]), d)
        got = grad[b, k].cpu().numpy().astype(np.float64)
        assert (np.abs(got - want) <= 2e-6 * abs(d) + 1e-4 * np.abs(want)).all(), (b, k)
        assert abs(float(h["lse"][b, k]) - oracle.row_lse(row)) <= 1e-5 + 1e-5 * abs(float(h["lse"][b, k]))
    # rows of unselected positions keep the canary (NaN for fp32)
    ub, uk = np.nonzero(select == 0)
    for i in rng.choice(len(ub), size=6, replace=False):
        assert torch.isnan(grad[int(ub[i]), int(uk[i])]).all()
