"""The variants of the sampling step on the GPU against the oracle, through the C ABI: the
fallback orders the paper compares Fork-dLLM with (Algorithm 1 and the ablations of Section 4.1).
Inputs are re-drawn until every decision has a clear margin in the oracle (threshold, fallback
ranking), so that fp32 and fp64 take the same one."""
import numpy as np
import pytest
import torch

import fork_synth as fs
import oracle
from helpers import (FALLBACK_MARGIN, compare_step_state, decisions_are_clear, live_mask,
                     oracle_reference_loop, to_torch_logits)
from test_gpu_step import make_rows
from test_gpu_workloads import check_loop_invariants, gpu_loop

pytestmark = pytest.mark.gpu

MODES = {"leftmost": 0, "max_conf": 1, "min_conf": 2, "max_entropy": 3, "random": 4}


def F():
    import paper_2609_39859_b200 as pkg
    return pkg


def step_both(x, mask, lo, hi, lam, mode, rand, step=3):
    pkg = F()
    B, Ll, V = x.shape
    Lt = mask.shape[1]
    o = oracle.StepState(B, Lt, mask=mask)
    assert oracle.step(o, x, lo, hi, lam, step_id=step, fallback_mode=mode, fallback_rand=rand) == 0
    if not decisions_are_clear(o, live_mask(mask, lo, hi), lam, 1e-4, mode):
        return None, o
    g = pkg.ForkState(B, Lt, mask=mask)
    keep = [torch.from_numpy(np.asarray(a)).cuda() for a in (lo, hi, rand.view(np.int32))]
    pkg.fork_step(g, to_torch_logits(x), keep[0], keep[1], lam, step=step, fallback_mode=mode,
                  fallback_rand=keep[2])
    torch.cuda.synchronize()
    return g.host(), o


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("mode", sorted(MODES))
def test_fallback_orders_single_steps(mode, dtype):
    """Blocks of up to 24 live rows; about half of the sequences have no row above lambda."""
    checked = fallbacks = 0
    for seed in range(12):
        rng = np.random.default_rng(100 * MODES[mode] + seed)
        B, Lt, V = 6, 40, 4104
        mask = (rng.random((B, Lt)) < 0.7).astype(np.uint8)
        lo = rng.integers(0, 16, size=B).astype(np.int32)
        hi = (lo + rng.integers(1, 24, size=B)).astype(np.int32)
        x = make_rows(rng, (B, Lt), V, dtype, peak=4.0, peak_frac=0.15)
        rand = rng.integers(0, 2 ** 32, B, dtype=np.uint64).astype(np.uint32)
        g, o = step_both(x, mask, lo, hi, 0.9, MODES[mode], rand)
        if g is None:
            continue
        compare_step_state(g, o)
        checked += 1
        fallbacks += int(o.is_fallback.sum())
    assert checked >= 6 and fallbacks >= 10


@pytest.mark.parametrize("mode", ["max_conf", "min_conf", "max_entropy", "random"])
def test_fallback_orders_with_more_than_32_live_rows(mode):
    """The finaliser's multi-batch path: 100 and 70 live rows in one window, all below lambda."""
    for seed in range(8):
        rng = np.random.default_rng(7 + seed)
        B, Lt, V = 2, 100, 2048
        mask = np.ones((B, Lt), np.uint8)
        mask[1, 5:35] = 0
        lo, hi = np.zeros(B, np.int32), np.full(B, Lt, np.int32)
        x = make_rows(rng, (B, Lt), V, "bf16", peak_frac=0.0)        # no planted peaks: every confidence is far below lambda
        rand = rng.integers(0, 2 ** 32, B, dtype=np.uint64).astype(np.uint32)
        g, o = step_both(x, mask, lo, hi, 0.9, MODES[mode], rand)
        if g is None:
            continue
        assert o.is_fallback.all()
        compare_step_state(g, o)
        return
    raise AssertionError("no input with clear margins found")


def test_flagged_rows_are_passed_over_and_all_flagged_takes_leftmost():
    rng = np.random.default_rng(3)
    B, Lt, V = 2, 8, 1024
    mask = np.ones((B, Lt), np.uint8)
    lo, hi = np.zeros(B, np.int32), np.full(B, Lt, np.int32)
    x = make_rows(rng, (B, Lt), V, "f32", peak=1.0, peak_frac=0.0)
    x[0, 0, 5] = np.nan                 # sequence 0: its leftmost row is flagged
    x[0, 3, 9] = np.inf
    x[1, :, 1] = np.nan                 # sequence 1: every row flagged
    rand = np.zeros(B, np.uint32)
    for mode in ("max_conf", "min_conf", "max_entropy"):
        g, o = step_both(x, mask, lo, hi, 0.9, MODES[mode], rand)
        assert g is not None
        compare_step_state(g, o)
        assert g["fallback_pos"][0] not in (0, 3) and g["fallback_pos"][1] == 0


@pytest.mark.parametrize("mode", ["max_conf", "max_entropy", "random"])
def test_tiny_decode_loop_under_other_fallback_orders(mode):
    """Whole semi-autoregressive loops (V=1024 fp32, one block of 32) with the fallback position
    chosen by Fast-dLLM's rule or an ablation's; Fork-dLLM's own invariant on the commit order
    (leftmost first) must then fail somewhere, which shows that the mode reached the kernel."""
    w = fs.workload("tiny")
    B = 4
    rand = np.array([3, 17, 0xFFFFFFF0, 12345], np.uint32)
    ost, nonces, osteps, _ = oracle_reference_loop(w, B, w.threshold, fallback_mode=MODES[mode], fallback_rand=rand)
    pkg = F()
    cfg = w.cfg(B=B)
    logits = torch.empty((B, w.Lt, w.V), dtype=torch.float32, device="cuda")
    st = pkg.ForkState(B, w.Lt)
    prov = fs.Provider(cfg, w.Lt * w.V, w.V, 0, w.Lt, nonce=nonces)
    rand_d = torch.from_numpy(rand.view(np.int32)).cuda()
    rc, steps = pkg.fork_decode_loop(st, logits, w.block_len, 0, w.Lt, prov.address, prov.ctx, w.threshold, 10000,
                                     fallback_mode=MODES[mode], fallback_rand=rand_d)
    torch.cuda.synchronize()
    prov.close()
    assert rc == 0 and steps == osteps
    h = st.host()
    compare_step_state(h, ost)
    with pytest.raises(AssertionError):
        check_loop_invariants(h, w, steps)


def test_bad_variant_arguments_are_rejected():
    pkg = F()
    B, Lt, V = 1, 4, 64
    st = pkg.ForkState(B, Lt)
    lg = torch.zeros((B, Lt, V), dtype=torch.float32, device="cuda")
    lo = torch.zeros(B, dtype=torch.int32, device="cuda")
    hi = torch.full((B,), Lt, dtype=torch.int32, device="cuda")
    for kw in (dict(fallback_mode=5), dict(fallback_mode=-1), dict(fallback_mode=4), dict(temperature=-1.0),
               dict(temperature=float("nan"))):
        with pytest.raises(pkg.ForkError) as e:
            pkg.fork_step(st, lg, lo, hi, 0.9, **kw)
        assert e.value.status == pkg.FORK_ERR_INVALID_ARG


@pytest.mark.parametrize("Lt,ratio", [(256, 0.2), (1024, 0.25), (37, 0.5), (20000, 0.01), (64, 0.0), (64, 1.0)])
def test_top_entropy_selection_matches_the_oracle(Lt, ratio):
    """JustGRPO-Fast's selection: both sides rank the same fp32 entropies, so the result is exact."""
    pkg = F()
    rng = np.random.default_rng(Lt)
    B = 5
    H = rng.gamma(2.0, 1.0, (B, Lt)).astype(np.float32)
    H[1, : Lt // 2] = H[1, 0]                                   # many ties
    H[2, ::5] = np.nan
    elig = (rng.random((B, Lt)) < 0.7).astype(np.uint8)
    elig[3] = 1
    elig[4] = 0
    rc, want_sel, want_cnt = oracle.select_top_entropy(H, elig, ratio)
    assert rc == 0
    sel, cnt = pkg.fork_select_top_entropy(torch.from_numpy(H).cuda(), torch.from_numpy(elig).cuda(), ratio)
    torch.cuda.synchronize()
    assert np.array_equal(cnt.cpu().numpy(), want_cnt)
    assert np.array_equal(sel.cpu().numpy(), want_sel)


def test_top_entropy_selection_feeds_the_scoring_pass():
    """Entropies of a decode loop -> selection -> fork_logprob on the selected positions."""
    pkg = F()
    w = fs.workload("tiny")
    B = 4
    ost, nonces, osteps, _ = oracle_reference_loop(w, B, w.threshold)
    rc, steps, calls, h = gpu_loop(w, w.threshold, nonces, B=B)
    assert rc == 0
    ent = torch.from_numpy(h["entropy"]).cuda()
    elig = torch.ones((B, w.Lt), dtype=torch.uint8, device="cuda")
    sel, cnt = pkg.fork_select_top_entropy(ent, elig, 0.2)
    rc, osel, ocnt = oracle.select_top_entropy(h["entropy"], np.ones((B, w.Lt), np.uint8), 0.2)
    assert np.array_equal(sel.cpu().numpy(), osel) and (ocnt == 6).all()        # floor(0.2 * 32)
    rng = np.random.default_rng(1)
    x = (rng.standard_normal((B, w.Lt, w.V)) * 2).astype(np.float32)
    st = pkg.ForkState(B, w.Lt)
    tokens = torch.from_numpy(h["tokens"]).cuda()
    lp, ssum, scnt, status = pkg.fork_logprob(torch.from_numpy(x).cuda(), tokens, sel, st)
    torch.cuda.synchronize()
    rc, olp, osum, ocnt2, _ = oracle.logprob(x, h["tokens"], osel)
    from helpers import assert_close
    assert_close("logp", lp.cpu().numpy(), olp)
    assert_close("seq_sum", ssum.cpu().numpy(), osum)
    assert np.array_equal(scnt.cpu().numpy(), ocnt2)
