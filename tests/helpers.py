"""Shared test plumbing: comparing the CUDA path's buffers with the oracle's, and running the oracle's
decode loop on generator inputs while keeping every confidence away from the threshold."""
import copy

import numpy as np

import fork_synth as fs
import oracle

RTOL, ATOL = 1e-4, 1e-5          # |gpu - oracle| <= ATOL + RTOL * |oracle| for conf, entropy, log-prob


def assert_close(name, got, want, where=None, rtol=None, atol=None):
    RTOL, ATOL = (globals()["RTOL"] if rtol is None else rtol), (globals()["ATOL"] if atol is None else atol)
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    if where is not None:
        got, want = got[where], want[where]
    both_nan = np.isnan(got) & np.isnan(want)
    both_inf = np.isinf(want) & (got == want)
    ok = both_nan | both_inf | (np.abs(got - want) <= ATOL + RTOL * np.abs(want))
    if not ok.all():
        i = np.flatnonzero(~ok.ravel())[:5]
        raise AssertionError("%s: %d of %d outside tolerance; first got=%s want=%s" %
                             (name, (~ok).sum(), ok.size, got.ravel()[i], want.ravel()[i]))


def assert_equal(name, got, want, where=None):
    got = np.asarray(got)
    want = np.asarray(want)
    if where is not None:
        got, want = got[where], want[where]
    if not (got.astype(np.int64) == want.astype(np.int64)).all():
        bad = np.flatnonzero((got.astype(np.int64) != want.astype(np.int64)).ravel())[:8]
        raise AssertionError("%s differs at %s: got=%s want=%s" % (name, bad, got.ravel()[bad], want.ravel()[bad]))


def compare_step_state(g: dict, o: "oracle.StepState", nseq=None, last_step_outputs=True, rtol=None, atol=None):
    """Bit-exact integers, floats within tolerance.  `g` is ForkState.host(); compares the first
    `nseq` sequences (all by default).  Positions never written keep their initial fill on both
    sides (-1 / 255 / NaN), so whole arrays can be compared."""
    n = o.B if nseq is None else nseq
    for name in ("tokens", "mask", "cand", "commit_step", "commit_fallback", "row_status"):
        assert_equal(name, g[name][:n], getattr(o, name)[:n])
    per_seq = ("nfe", "n_fallback")
    if last_step_outputs:        # describe the LAST step only: comparable when both sides ran the same steps
        per_seq += ("n_unmasked", "is_fallback", "fallback_pos")
    for name in per_seq:
        assert_equal(name, g[name][:n], getattr(o, name)[:n])
    for name in ("conf", "entropy", "logp", "commit_logp"):
        assert_close(name, g[name][:n], getattr(o, name)[:n], rtol=rtol, atol=atol)


def live_mask(mask, lo, hi):
    B, Lt = mask.shape
    k = np.arange(Lt)[None, :]
    return (mask != 0) & (k >= np.asarray(lo)[:, None]) & (k < np.asarray(hi)[:, None])


FALLBACK_MARGIN = {0: 0.0, 1: 5e-4, 2: 5e-4, 3: 5e-3, 4: 0.0}   # per fallback order: keys are confidences (<=1) or entropies (<=12 nats)
SAMPLE_MARGIN = 2e-6                                             # drawn candidates: distance of U * total from the nearest boundary of the running sum, over the total


def decisions_are_clear(st, live, threshold, margin, fallback_mode=0, temperature=0.0):
    """True when no decision of the step just taken sits within rounding distance of flipping:
    confidences against the threshold, the fallback order's best against its runner-up, and (with
    stochastic candidates) the point of the running sum that the draw hits against the boundaries of the
    drawn token's stretch (fp32 sums in another order could otherwise land on a neighbour)."""
    if not (np.abs(st.conf[live] - np.float64(np.float32(threshold))) >= margin).all():
        return False
    if not (st.fallback_margin >= FALLBACK_MARGIN[fallback_mode]).all():
        return False
    if temperature > 0 and not (st.sample_margin[live] >= SAMPLE_MARGIN).all():
        return False
    return True


def oracle_reference_loop(w: "fs.Workload", nseq: int, threshold: float, margin: float = 1e-4,
                          max_steps: int = 100000, nthreads: int = 0, fallback_mode: int = 0,
                          fallback_rand=None, temperature: float = 0.0, sample_seed: int = 0):
    """The oracle's semi-autoregressive loop on the first `nseq` sequences of workload `w`, with
    host-generated logits.  At every step the nonce is bumped until no decision of the step lies
    within rounding distance of flipping (see decisions_are_clear), so fp32 and fp64 cannot
    disagree on it.
    Returns (final StepState, per-step nonces, steps taken, per-step live-row counts)."""
    cfg = w.cfg(B=nseq)
    st = oracle.StepState(nseq, w.Lt)
    logits = np.empty((nseq, w.Lt, w.V), w.np_dtype)
    fs.canary_host(logits)
    lo, hi = oracle.block_cursors(st.mask, 0, w.Lt, w.block_len)
    nonces, live_counts = [], []
    step = 0
    while (lo < hi).any():
        assert step < max_steps
        live = live_mask(st.mask, lo, hi)
        nonce = 0
        while True:
            fs.fill_host(cfg, step, st.mask, lo, hi, logits, nonce=nonce, nthreads=nthreads)
            trial = copy.deepcopy(st)
            assert oracle.step(trial, logits, lo, hi, threshold, step_id=step, nthreads=nthreads,
                               fallback_mode=fallback_mode, fallback_rand=fallback_rand, temperature=temperature,
                               sample_seed=sample_seed) == 0
            if decisions_are_clear(trial, live, threshold, margin, fallback_mode, temperature):
                break
            nonce += 1
            assert nonce < 64
        st = trial
        nonces.append(nonce)
        live_counts.append(int(live.sum()))
        step += 1
        lo, hi = oracle.block_cursors(st.mask, 0, w.Lt, w.block_len, lo, hi)
    return st, np.asarray(nonces, np.uint32), step, live_counts


def to_torch_logits(arr: np.ndarray, device="cuda"):
    import torch
    if arr.dtype == np.uint16:
        return torch.from_numpy(arr.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(arr).to(device)
