"""The step fused into the LM-head product (hidden states and weight in, logits never stored) against
the oracle: fp64 product of the same bf16 inputs, rounded once to fp32, then Algorithm 2 as always.
Shapes: the LLaDA-8B head the paper names (d = 4096, V = 126464) at 8, 256 and 2048 window rows, and
small ragged ones.  Inputs are re-drawn until no decision of the checked rows sits within rounding
distance of flipping (confidence against the threshold, the two largest logits against each other).

Tolerance.  The logits of this path are the tensor cores' fp32 accumulators.  A tcgen05.mma adds 16
products to the running sum with a rounding of at most one unit in the last place of that sum, and
a row's logit takes d / 16 = 256 of them; with |logit| <= 32 that bounds the error of a logit by
256 * 2^-23 * 32 = 1e-3 (observed: a few 1e-4 on the largest logits, where the partial sums are
largest).  Confidence and log-probability move by at most that much relatively / absolutely, the
entropy by that much times its own size plus the same absolute amount, so the floats are compared at
|gpu - oracle| <= 1e-4 + 1e-3 |oracle| (the step on stored logits: 1e-5 + 1e-4 |oracle|), and the
margins of the decisions are widened accordingly (2e-3 on confidences, 5e-3 on the top-two gap)."""
HEAD_RTOL, HEAD_ATOL = 1e-3, 1e-4
import numpy as np
import pytest
import torch

import fork_synth as fs
import oracle
from helpers import compare_step_state

pytestmark = pytest.mark.gpu

_W = {}


def weight(V, d):
    if (V, d) not in _W:
        bits = fs.head_weight(V, d, seed=0x39859_00A0 + V + d)
        _W.clear()                                    # one large weight at a time
        _W[(V, d)] = (bits, torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16))
    return _W[(V, d)]


def run_case(B, Ll, Lt, pos0, V, d, lam, n_check, mask_density=1.0, seed=1):
    import paper_2609_39859_b200 as pkg
    w_bits, w_dev = weight(V, d)
    rng = np.random.default_rng(seed)
    mask = (rng.random((B, Lt)) < mask_density).astype(np.uint8)
    lo = np.full(B, pos0, np.int32)
    hi = np.full(B, pos0 + Ll, np.int32)
    if B > 2:
        hi[-1] = lo[-1]                               # a sequence that sits out
        hi[1] = pos0 + max(1, Ll // 2)                # a shorter block
    for nonce in range(8):
        h_bits, _ = fs.head_hidden(w_bits, B * Ll, seed=seed * 100 + nonce)
        chk = n_check * Ll
        logits = oracle.head_logits(h_bits[:chk], w_bits).reshape(n_check, Ll, V)
        o = oracle.StepState(n_check, Lt, mask=mask[:n_check])
        assert oracle.step(o, logits, lo[:n_check], hi[:n_check], lam, step_id=3, pos0=pos0) == 0
        k = np.arange(Lt)[None, :]
        live = (mask[:n_check] != 0) & (k >= lo[:n_check, None]) & (k < hi[:n_check, None])
        top2 = np.partition(logits, V - 2, axis=2)[:, :, V - 2:]
        gap = (top2[:, :, 1] - top2[:, :, 0])
        gap_full = np.full((n_check, Lt), np.inf)
        gap_full[:, pos0:pos0 + Ll] = gap
        if (np.abs(o.conf[live] - np.float64(np.float32(lam))) >= 2e-3).all() and (gap_full[live] >= 5e-3).all():
            break
    else:
        raise AssertionError("no draw with clear margins")
    st = pkg.ForkState(B, Lt, mask=mask)
    hid = torch.from_numpy(h_bits.view(np.int16)).cuda().view(torch.bfloat16).view(B, Ll, d)
    n0 = pkg.fork_kernel_launches()
    pkg.fork_step_fused_head(st, hid, w_dev, torch.from_numpy(lo).cuda(), torch.from_numpy(hi).cuda(), lam, step=3, pos0=pos0)
    torch.cuda.synchronize()
    assert pkg.fork_kernel_launches() - n0 == 4
    assert pkg.fork_device_status(st) == 0
    g = st.host()
    compare_step_state(g, o, nseq=n_check, rtol=HEAD_RTOL, atol=HEAD_ATOL)
    # every sequence: the unmask rule on the step's own confidences
    for b in range(B):
        k = np.arange(Lt)
        live_b = (mask[b] != 0) & (k >= lo[b]) & (k < hi[b])
        if not live_b.any():
            assert g["n_unmasked"][b] == 0 and (g["mask"][b] == mask[b]).all()
            continue
        above = live_b & (g["conf"][b] > np.float32(lam))
        want = above if above.any() else (k == k[live_b][0])
        assert ((g["mask"][b] == 0) & (mask[b] != 0) == want).all()
        assert g["is_fallback"][b] == (0 if above.any() else 1)
        assert (g["mask"][b][~live_b] == mask[b][~live_b]).all()
    return g


def test_small_ragged_shapes():
    # V not a multiple of the 256-column tile, rows not a multiple of 128, a window inside a longer buffer
    run_case(B=3, Ll=5, Lt=16, pos0=4, V=1000, d=128, lam=0.9, n_check=3, mask_density=0.8, seed=2)
    run_case(B=5, Ll=40, Lt=40, pos0=0, V=5000, d=256, lam=0.5, n_check=5, mask_density=0.7, seed=3)
    # 33..64 window rows: the 64-row box of hidden states; a vocabulary that ends inside a 32-column group
    run_case(B=2, Ll=24, Lt=24, pos0=0, V=3001, d=192, lam=0.7, n_check=2, mask_density=0.9, seed=4)


@pytest.mark.parametrize("B,Ll,n_check", [(1, 8, 1), (8, 32, 8), (64, 32, 6)])
def test_llada_head_shapes(B, Ll, n_check):
    run_case(B=B, Ll=Ll, Lt=256, pos0=32, V=126464, d=4096, lam=0.9, n_check=n_check, seed=10 + B)


@pytest.mark.parametrize("mode", ["max_conf", "min_conf", "max_entropy", "random"])
def test_fallback_orders_on_the_fused_head(mode):
    """The comparison orders of a fallback step (Algorithm 1's arg-max confidence and the ablations) apply
    to the fused-head step as to the step on stored logits: with a threshold nothing clears, every live
    sequence commits exactly the position the oracle picks under that order."""
    import paper_2609_39859_b200 as pkg
    code = {"max_conf": pkg.FORK_FALLBACK_MAX_CONF, "min_conf": pkg.FORK_FALLBACK_MIN_CONF,
            "max_entropy": pkg.FORK_FALLBACK_MAX_ENTROPY, "random": pkg.FORK_FALLBACK_RANDOM}[mode]
    B, Ll, Lt, V, d = 4, 8, 8, 3000, 256
    w_bits, w_dev = weight(V, d)
    rng = np.random.default_rng(40 + code)
    mask = (rng.random((B, Lt)) < 0.8).astype(np.uint8)
    mask[:, 0] = 1
    lo, hi = np.zeros(B, np.int32), np.full(B, Ll, np.int32)
    rand = rng.integers(0, 2 ** 32, B, dtype=np.uint32) if mode == "random" else None
    for nonce in range(32):
        h_bits, _ = fs.head_hidden(w_bits, B * Ll, seed=900 + 32 * code + nonce, h_lo=0.0, h_hi=6.0)
        logits = oracle.head_logits(h_bits, w_bits).reshape(B, Ll, V)
        o = oracle.StepState(B, Lt, mask=mask)
        assert oracle.step(o, logits, lo, hi, 1.0, step_id=0, fallback_mode=code, fallback_rand=rand) == 0
        if (o.fallback_margin >= (5e-3 if mode == "max_entropy" else 2e-3)).all():   # the order's best and its runner-up are clearly apart
            break
    else:
        raise AssertionError("no draw with clear margins")
    st = pkg.ForkState(B, Lt, mask=mask)
    hid = torch.from_numpy(h_bits.view(np.int16)).cuda().view(torch.bfloat16).view(B, Ll, d)
    pkg.fork_step_fused_head(st, hid, w_dev, torch.from_numpy(lo).cuda(), torch.from_numpy(hi).cuda(), 1.0, step=0,
                             fallback_mode=code, fallback_rand=None if rand is None else torch.from_numpy(rand.view(np.int32)).cuda())
    torch.cuda.synchronize()
    g = st.host()
    assert (g["is_fallback"] == 1).all() and (g["n_unmasked"] == 1).all()
    assert (g["fallback_pos"] == o.fallback_pos).all()
    compare_step_state(g, o, rtol=HEAD_RTOL, atol=HEAD_ATOL)


@pytest.mark.parametrize("tau", [0.0, 0.8])
def test_decode_loop_on_hidden_states(tau):
    """fork_decode_loop_fused_head: every step the provider hands over the hidden states of each sequence's own
    active block (row l of sequence b = position lo[b] + l) and the step runs on the product with the head; the
    whole loop against the oracle's loop on the same products, sequences drifting apart in their blocks."""
    import paper_2609_39859_b200 as pkg
    from helpers import live_mask
    B, Lt, BL, V, d, lam = 3, 24, 8, 3000, 256, 0.6
    w_bits, w_dev = weight(V, d)
    slices = np.append(np.arange(0, V, 32), V).astype(np.int32)
    draw = dict(temperature=tau, sample_seed=99, slices=slices) if tau > 0 else {}
    o = oracle.StepState(B, Lt)
    lo, hi = oracle.block_cursors(o.mask, 0, Lt, BL)
    hidden_steps = []
    step = 0
    while (lo < hi).any():
        assert step < 200
        live = live_mask(o.mask, lo, hi)
        for nonce in range(64):
            h_bits, _ = fs.head_hidden(w_bits, B * BL, seed=7000 + 64 * step + nonce, h_lo=0.0 if tau == 0 else 3.0, h_hi=9.0 if tau == 0 else 12.0)
            blocks = oracle.head_logits(h_bits, w_bits).reshape(B, BL, V)
            full = np.full((B, Lt, V), np.nan, np.float32)      # rows outside a sequence's block must not be read
            for b in range(B):
                n = max(0, min(BL, Lt - int(lo[b])))
                full[b, lo[b]:lo[b] + n] = blocks[b, :n]
            import copy
            trial = copy.deepcopy(o)
            assert oracle.step(trial, full, lo, hi, lam, step_id=step, **draw) == 0
            rows = full[live]
            top2 = np.partition(rows, V - 2, axis=1)[:, V - 2:]
            if (np.abs(trial.conf[live] - np.float64(np.float32(lam))) >= 2e-3).all() and ((top2[:, 1] - top2[:, 0]) >= 5e-3).all() \
                    and (tau == 0 or (trial.sample_margin[live] >= 5e-4).all()):
                break
        else:
            raise AssertionError("no draw with clear margins at step %d" % step)
        o = trial
        hidden_steps.append(torch.from_numpy(h_bits.view(np.int16)).view(torch.bfloat16).view(B, BL, d).pin_memory())
        step += 1
        lo, hi = oracle.block_cursors(o.mask, 0, Lt, BL, lo, hi)
    assert tau > 0 or step > Lt // BL                            # more than one step per block: thresholds and fallbacks both occur
    st = pkg.ForkState(B, Lt)
    hid = torch.zeros((B, BL, d), dtype=torch.bfloat16, device="cuda")
    calls = []

    def model(s_, lo_ptr, hi_ptr, stream_ptr):
        calls.append(s_)
        hid.copy_(hidden_steps[min(s_, len(hidden_steps) - 1)], non_blocking=True)
        return 0

    rc, steps = pkg.fork_decode_loop_fused_head(st, hid, w_dev, BL, 0, Lt, model, None, lam, max_steps=200,
                                                **({"temperature": tau, "sample_seed": 99} if tau > 0 else {}))
    torch.cuda.synchronize()
    assert rc == 0 and steps == step and calls == list(range(step))
    assert pkg.fork_device_status(st) == 0
    g = st.host()
    assert g["mask"].sum() == 0
    compare_step_state(g, o, rtol=HEAD_RTOL, atol=HEAD_ATOL)
    assert (g["nfe"] == o.nfe).all() and (g["n_fallback"] == o.n_fallback).all()
    assert tau > 0 or g["n_fallback"].sum() > 0                # (the drawn case plants high peaks to keep its draws clear: no fallbacks there)


@pytest.mark.parametrize("B,Ll,V,d,tau", [(3, 7, 1000, 128, 0.8), (4, 8, 40000, 256, 0.8), (2, 16, 5003, 192, 1.3)])
def test_drawn_candidates_on_the_fused_head(B, Ll, V, d, tau):
    """Candidates at a temperature on the fused-head step: the two-stage draw (a chunk of 32 consecutive entries by
    the row's slice uniform, the token inside it by its entry uniform, both by inversion in ascending order) is the
    oracle's draw with the vocabulary in slices of 32; tokens are compared exactly on inputs whose draws keep clear of
    the boundaries of the running sums, confidence and log-probability are the untempered ones of the drawn token."""
    import paper_2609_39859_b200 as pkg
    Lt, lam, seed = Ll, 0.9, 77
    w_bits, w_dev = weight(V, d)
    rng = np.random.default_rng(3 * V + B)
    mask = (rng.random((B, Lt)) < 0.9).astype(np.uint8)
    lo, hi = np.zeros(B, np.int32), np.full(B, Ll, np.int32)
    slices = np.append(np.arange(0, V, 32), V).astype(np.int32)
    for nonce in range(48):
        h_bits, _ = fs.head_hidden(w_bits, B * Ll, seed=31000 + 48 * (V % 97) + nonce, h_lo=3.0, h_hi=12.0)
        logits = oracle.head_logits(h_bits, w_bits).reshape(B, Ll, V)
        o = oracle.StepState(B, Lt, mask=mask)
        assert oracle.step(o, logits, lo, hi, lam, step_id=4, temperature=tau, sample_seed=seed, slices=slices) == 0
        live = (mask != 0)
        # (with a chunk per 32 entries the running sum over the chunks has a boundary every 1/1250 of a flat row's
        # mass: the margin is what the draws of these few rows keep, not a bound on the kernels' error)
        if (np.abs(o.conf[live] - np.float64(np.float32(lam))) >= 2e-3).all() and (o.sample_margin[live] >= 5e-4).all():
            break
    else:
        raise AssertionError("no draw with clear margins")
    st = pkg.ForkState(B, Lt, mask=mask)
    hid = torch.from_numpy(h_bits.view(np.int16)).cuda().view(torch.bfloat16).view(B, Ll, d)
    n0 = pkg.fork_kernel_launches()
    pkg.fork_step_fused_head(st, hid, w_dev, torch.from_numpy(lo).cuda(), torch.from_numpy(hi).cuda(), lam, step=4,
                             temperature=tau, sample_seed=seed)
    torch.cuda.synchronize()
    assert pkg.fork_kernel_launches() - n0 == 5               # active set, product + reduction, merge, draw, unmask rule
    assert pkg.fork_device_status(st) == 0
    g = st.host()
    compare_step_state(g, o, rtol=HEAD_RTOL, atol=HEAD_ATOL)


def test_drawn_candidates_on_the_fused_head_at_a_block_of_eight_sequences():
    """256 window rows, V = 40000: per position, the drawn token is the oracle's wherever the oracle's draw keeps
    clear of the boundaries of its running sums (and nearly everywhere else), and confidence, log-probability and
    entropy of every position with the same token agree; it is a draw, not the arg-max."""
    import paper_2609_39859_b200 as pkg
    B, Ll, V, d, tau, seed = 8, 32, 40000, 256, 0.8, 78
    w_bits, w_dev = weight(V, d)
    mask = np.ones((B, Ll), np.uint8)
    lo, hi = np.zeros(B, np.int32), np.full(B, Ll, np.int32)
    slices = np.append(np.arange(0, V, 32), V).astype(np.int32)
    h_bits, _ = fs.head_hidden(w_bits, B * Ll, seed=4242, h_lo=0.0, h_hi=10.0)
    logits = oracle.head_logits(h_bits, w_bits).reshape(B, Ll, V)
    o = oracle.StepState(B, Ll, mask=mask)
    assert oracle.step(o, logits, lo, hi, 2.0, step_id=1, temperature=tau, sample_seed=seed, slices=slices) == 0
    st = pkg.ForkState(B, Ll, mask=mask)
    hid = torch.from_numpy(h_bits.view(np.int16)).cuda().view(torch.bfloat16).view(B, Ll, d)
    pkg.fork_step_fused_head(st, hid, w_dev, torch.from_numpy(lo).cuda(), torch.from_numpy(hi).cuda(), 2.0, step=1,
                             temperature=tau, sample_seed=seed)
    torch.cuda.synchronize()
    g = st.host()
    same = g["cand"] == o.cand
    clear = o.sample_margin >= 2e-3
    assert same[clear].all() and clear.mean() > 0.5
    assert same.mean() > 0.97
    for name in ("conf", "logp", "entropy"):
        got, want = g[name][same].astype(np.float64), getattr(o, name)[same]
        assert (np.abs(got - want) <= HEAD_ATOL + HEAD_RTOL * np.abs(want)).all(), name
    assert (g["cand"] != logits.argmax(-1)).mean() > 0.05       # it is a draw, not the arg-max
    assert (g["n_unmasked"] == 1).all() and (g["is_fallback"] == 1).all()   # threshold 2: every sequence commits its leftmost position


def test_drawn_candidates_on_the_fused_head_follow_the_tempered_softmax():
    """Distribution: one row's hidden state repeated over many positions and seeds; the drawn tokens against
    softmax(logits / tau) by chi-square on the likeliest tokens."""
    import paper_2609_39859_b200 as pkg
    from scipy import stats
    B, Ll, V, d, tau = 16, 32, 1000, 128, 0.9
    w_bits, w_dev = weight(V, d)
    h_bits, _ = fs.head_hidden(w_bits, 1, seed=5, sigma=2.0, h_lo=1.0, h_hi=1.0)
    logits = oracle.head_logits(h_bits, w_bits)[0].astype(np.float64)
    prob = np.exp((logits - logits.max()) / tau)
    prob /= prob.sum()
    hid = torch.from_numpy(np.repeat(h_bits, B * Ll, 0).view(np.int16)).cuda().view(torch.bfloat16).view(B, Ll, d)
    lo = torch.zeros(B, dtype=torch.int32, device="cuda")
    hi = torch.full((B,), Ll, dtype=torch.int32, device="cuda")
    counts = np.zeros(V, np.int64)
    for seed in range(24):
        st = pkg.ForkState(B, Ll)
        pkg.fork_step_fused_head(st, hid, w_dev, lo, hi, 2.0, step=seed, temperature=tau, sample_seed=1000 + seed)
        torch.cuda.synchronize()
        counts += np.bincount(st.host()["cand"].ravel(), minlength=V)
    n = counts.sum()
    top = np.flatnonzero(prob * n >= 8)                          # the tokens likely enough for a chi-square cell of their own
    obs = np.append(counts[top], n - counts[top].sum())
    exp = np.append(prob[top], 1 - prob[top].sum()) * n
    assert len(top) >= 20 and exp.min() > 5
    assert stats.chisquare(obs, exp).pvalue > 1e-4


def test_drawn_candidates_at_the_llada_head_shape():
    """d = 4096, V = 126464, 256 window rows (the shape at which every row's chunks are gone through in two passes
    rather than range by range): the first two sequences' positions against the oracle, as above."""
    import paper_2609_39859_b200 as pkg
    B, Ll, V, d, tau, seed, n_check = 8, 32, 126464, 4096, 0.8, 5, 2
    w_bits, w_dev = weight(V, d)
    mask = np.ones((B, Ll), np.uint8)
    lo, hi = np.zeros(B, np.int32), np.full(B, Ll, np.int32)
    slices = np.append(np.arange(0, V, 32), V).astype(np.int32)
    h_bits, _ = fs.head_hidden(w_bits, B * Ll, seed=99)
    logits = oracle.head_logits(h_bits[:n_check * Ll], w_bits).reshape(n_check, Ll, V)
    o = oracle.StepState(n_check, Ll, mask=mask[:n_check])
    assert oracle.step(o, logits, lo[:n_check], hi[:n_check], 2.0, step_id=1, temperature=tau, sample_seed=seed, slices=slices) == 0
    st = pkg.ForkState(B, Ll, mask=mask)
    hid = torch.from_numpy(h_bits.view(np.int16)).cuda().view(torch.bfloat16).view(B, Ll, d)
    pkg.fork_step_fused_head(st, hid, w_dev, torch.from_numpy(lo).cuda(), torch.from_numpy(hi).cuda(), 2.0, step=1,
                             temperature=tau, sample_seed=seed)
    torch.cuda.synchronize()
    assert pkg.fork_device_status(st) == 0
    g = st.host()
    same = g["cand"][:n_check] == o.cand
    clear = o.sample_margin >= 2e-3
    assert same[clear].all() and clear.mean() > 0.4 and same.mean() > 0.9
    for name in ("conf", "logp", "entropy"):
        got, want = g[name][:n_check][same].astype(np.float64), getattr(o, name)[same]
        assert (np.abs(got - want) <= HEAD_ATOL + HEAD_RTOL * np.abs(want)).all(), name
    assert (g["cand"][:n_check] != logits.argmax(-1)).mean() > 0.05


def test_decode_loop_on_hidden_states_error_paths():
    """The loop's own outcomes on the hidden-state form: the step limit, a failing provider, and a clean restart
    from the buffers as they were left."""
    import paper_2609_39859_b200 as pkg
    B, Lt, BL, V, d = 2, 16, 8, 1000, 128
    w_bits, w_dev = weight(V, d)
    h_bits, _ = fs.head_hidden(w_bits, B * BL, seed=3)
    hid = torch.from_numpy(h_bits.view(np.int16)).cuda().view(torch.bfloat16).view(B, BL, d)
    st = pkg.ForkState(B, Lt)
    rc, steps = pkg.fork_decode_loop_fused_head(st, hid, w_dev, BL, 0, Lt, lambda *a: 0, None, 2.0, max_steps=3, raise_on_error=False)
    torch.cuda.synchronize()
    assert rc == pkg.FORK_ERR_MAX_STEPS and steps == 3
    g = st.host()
    assert (g["mask"].sum(1) == Lt - 3).all() and g["commit_step"][0, :3].tolist() == [0, 1, 2]   # threshold 2: left to right
    calls = []

    def failing(step, lo, hi, stream_p):
        calls.append(step)
        return 1 if step == 5 else 0

    rc, steps = pkg.fork_decode_loop_fused_head(st, hid, w_dev, BL, 0, Lt, failing, None, 2.0, max_steps=100, step0=3, raise_on_error=False)
    torch.cuda.synchronize()
    assert rc == pkg.FORK_ERR_PROVIDER and steps == 2 and calls == [3, 4, 5]
    rc, steps = pkg.fork_decode_loop_fused_head(st, hid, w_dev, BL, 0, Lt, lambda *a: 0, None, 2.0, max_steps=100, step0=5)
    torch.cuda.synchronize()
    g = st.host()
    assert rc == 0 and steps == Lt - 5 and g["mask"].sum() == 0
    assert (g["commit_step"] == np.arange(Lt)[None, :]).all() and (g["nfe"] == Lt).all()
    with pytest.raises(pkg.ForkError):
        pkg.fork_decode_loop_fused_head(pkg.ForkState(B, Lt), hid, w_dev, BL, 0, Lt, lambda *a: 0, None, 2.0, max_steps=1)
