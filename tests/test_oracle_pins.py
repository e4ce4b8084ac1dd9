"""Pins for the fp64 oracle: everything here checks the oracle against something other than itself
(closed forms, brute force from the definition, library routines, hand-worked rows and steps,
invariants and special cases of the loop).  CPU only."""
import math
import os

import mpmath as mp
import numpy as np
import pytest
import scipy.special
import scipy.stats

import fork_synth as fs
import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "closed_forms.txt")
LN = math.log


def f32row(vals):
    return np.asarray(vals, np.float32)


def bf16row(vals):
    return fs.f32_to_bf16_bits(np.asarray(vals, np.float32))


# ---------------------------------------------------------------------------- row statistics ----
def test_hand_worked_rows():
    """Softmax rows small enough to do by hand (Section 2: c = q(x_0 | x_t); entropy in nats)."""
    s = oracle.row_stats(f32row([0, 0, 0, 0]))
    assert s["cand"] == 0 and s["conf"] == pytest.approx(0.25, abs=1e-15)
    assert s["entropy"] == pytest.approx(1.3862943611198906, abs=1e-13)
    assert s["logp"] == pytest.approx(-1.3862943611198906, abs=1e-13)
    # [2,1,0]: s = 1 + e^-1 + e^-2, t = -e^-1 - 2 e^-2
    s = oracle.row_stats(f32row([2, 1, 0]))
    assert s["s"] == pytest.approx(1.5032147244080551, abs=1e-13)
    assert s["t"] == pytest.approx(-0.6385500076, abs=1e-9)
    assert s["conf"] == pytest.approx(0.6652409557748219, abs=1e-13)
    assert s["entropy"] == pytest.approx(0.8323955818, abs=1e-9)
    assert s["logp"] == pytest.approx(-0.4076059644443803, abs=1e-13)
    s = oracle.row_stats(f32row([3, 0]))
    assert s["conf"] == pytest.approx(1 / (1 + math.exp(-3)), abs=1e-15)
    assert s["entropy"] == pytest.approx(0.1908649711, abs=1e-9)
    s = oracle.row_stats(f32row([1, 1, 0]))      # tie: lowest index wins
    assert s["cand"] == 0
    assert s["conf"] == pytest.approx(0.4223187982515182, abs=1e-13)
    assert s["entropy"] == pytest.approx(1.0173572076, abs=1e-9)
    s = oracle.row_stats(f32row([0, 1, 1]))
    assert s["cand"] == 1


def _golden_cases():
    out = []
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            V, k, h, conf, H, lpt, lpb = line.split()
            out.append((int(V), int(k), float(h), float(conf), float(H), float(lpt), float(lpb)))
    return out


@pytest.mark.parametrize("case", _golden_cases(), ids=lambda c: "V%d-k%d-h%g" % c[:3])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_peak_over_flat_closed_form(case, dtype):
    """k equal tops of height h over zeros: conf = 1/(k+(V-k)e^-h), H = ln s + h(V-k)e^-h/s."""
    V, k, h, conf, H, lpt, lpb = case
    rng = np.random.default_rng(V * 7 + k)
    x = np.zeros(V, np.float32)
    tops = np.sort(rng.choice(V, size=k, replace=False))
    x[tops] = h                                   # h is exactly representable in bf16 in every case
    row = f32row(x) if dtype == "f32" else bf16row(x)
    s = oracle.row_stats(row)
    assert s["cand"] == int(tops[0])
    assert s["conf"] == pytest.approx(conf, rel=1e-12)
    assert s["entropy"] == pytest.approx(H, rel=1e-12)
    assert s["logp"] == pytest.approx(lpt, rel=1e-12, abs=1e-15)
    bg = int(np.setdiff1d(np.arange(min(V, 64)), tops)[0])
    lp, st = oracle.row_logp(row, bg)
    assert st == 0 and lp == pytest.approx(lpb, rel=1e-12)
    lp, st = oracle.row_logp(row, int(tops[-1]))
    assert lp == pytest.approx(lpt, rel=1e-12, abs=1e-15)


def test_tie_position_does_not_matter():
    """The arg-max of tied tops is the lowest index wherever the tops sit (first, last, anywhere)."""
    V = 1000
    for tops in ([0, V - 1], [V - 1, V - 2], [500, 3, 998], [1, 0]):
        x = np.zeros(V, np.float32)
        x[tops] = 5.0
        assert oracle.row_stats(x)["cand"] == min(tops)
    x = np.full(V, -2.5, np.float32)                  # uniform row
    s = oracle.row_stats(x)
    assert s["cand"] == 0 and s["conf"] == pytest.approx(1 / V, rel=1e-13)
    assert s["entropy"] == pytest.approx(LN(V), rel=1e-13)
    # signed zeros compare equal: the first of them wins
    assert oracle.row_stats(f32row([-0.0, 0.0, -1.0]))["cand"] == 0
    assert oracle.row_stats(f32row([0.0, -0.0, -1.0]))["cand"] == 0


@pytest.mark.parametrize("seed", range(6))
def test_brute_force_without_max_shift(seed):
    """p_v = e^{x_v} / sum_u e^{x_u} and H = -sum p ln p with no max shift, in 50-digit arithmetic."""
    mp.mp.dps = 50
    rng = np.random.default_rng(seed)
    V = int(rng.integers(2, 17))
    x = (rng.uniform(-20, 20, size=V)).astype(np.float32)
    if seed % 2:
        x = fs.bf16_bits_to_f32(fs.f32_to_bf16_bits(x))
    row = x if seed % 2 == 0 else fs.f32_to_bf16_bits(x)
    ex = [mp.e ** mp.mpf(float(v)) for v in x]
    Z = sum(ex)
    p = [e / Z for e in ex]
    H = -sum(pi * mp.log(pi) for pi in p)
    best = max(range(V), key=lambda i: (float(x[i]), -i))
    s = oracle.row_stats(row)
    assert s["cand"] == best
    assert s["conf"] == pytest.approx(float(p[best]), rel=1e-12)
    assert s["entropy"] == pytest.approx(float(H), rel=1e-11, abs=1e-13)
    for tok in range(V):
        lp, st = oracle.row_logp(row, tok)
        assert st == 0 and lp == pytest.approx(float(mp.log(p[tok])), rel=1e-12, abs=1e-13)
    # probabilities from the per-token log-probabilities sum to one
    assert sum(math.exp(oracle.row_logp(row, t)[0]) for t in range(V)) == pytest.approx(1.0, abs=1e-13)


@pytest.mark.parametrize("V,dtype,sigma", [(1024, "f32", 2.0), (4097, "bf16", 3.0), (126464, "bf16", 3.0),
                                           (3, "f32", 5.0), (50000, "f32", 3.0)])
def test_against_library_softmax(V, dtype, sigma):
    """Gaussian rows have no closed form: compare with scipy's logsumexp / softmax / entropy."""
    rng = np.random.default_rng(V)
    x = (rng.standard_normal(V) * sigma).astype(np.float32)
    x[rng.integers(0, V)] += 9.0
    row = x if dtype == "f32" else fs.f32_to_bf16_bits(x)
    xd = (x if dtype == "f32" else fs.bf16_bits_to_f32(row)).astype(np.float64)
    lse = scipy.special.logsumexp(xd)
    p = scipy.special.softmax(xd)
    s = oracle.row_stats(row)
    assert s["cand"] == int(np.argmax(xd))
    assert s["conf"] == pytest.approx(float(p.max()), rel=1e-11)
    assert s["entropy"] == pytest.approx(float(scipy.stats.entropy(p)), rel=1e-10, abs=1e-12)
    assert s["logp"] == pytest.approx(float(xd.max() - lse), rel=1e-11, abs=1e-13)
    tok = int(rng.integers(0, V))
    assert oracle.row_logp(row, tok)[0] == pytest.approx(float(xd[tok] - lse), rel=1e-11)
    # invariants
    assert 1.0 / V <= s["conf"] <= 1.0
    assert 0.0 <= s["entropy"] <= LN(V) + 1e-12
    assert s["logp"] == pytest.approx(LN(s["conf"]), abs=1e-13)


def test_minus_inf_is_probability_zero_and_bad_rows():
    x = f32row([1.0, -np.inf, 0.5, -np.inf, 1.0])
    s = oracle.row_stats(x)
    ref = oracle.row_stats(f32row([1.0, 0.5, 1.0]))
    assert s["status"] == 0 and s["cand"] == 0
    for key in ("conf", "entropy", "logp"):
        assert s[key] == pytest.approx(ref[key], abs=1e-15)
    assert oracle.row_logp(x, 1)[0] == -np.inf
    for bad in ([1.0, np.nan, 3.0, 2.0], [np.inf, 0.0], [-np.inf, -np.inf], [np.nan, np.nan]):
        s = oracle.row_stats(f32row(bad))
        assert s["status"] & oracle.ROW_BAD and s["conf"] == 0.0 and math.isnan(s["entropy"])
    assert oracle.row_stats(f32row([1.0, np.nan, 3.0, 3.0]))["cand"] == 2   # max over the non-NaN entries
    assert oracle.row_stats(f32row([np.nan, np.nan]))["cand"] == 0
    assert oracle.row_stats(f32row([0.0, np.inf, np.inf]))["cand"] == 1
    lp, st = oracle.row_logp(f32row([0.0, 1.0]), 2)
    assert st & oracle.ROW_BAD_TOKEN and lp == 0.0
    lp, st = oracle.row_logp(f32row([0.0, 1.0]), -1)
    assert st & oracle.ROW_BAD_TOKEN


def test_bf16_bits_are_widened_exactly():
    # 0x4049 = 3.140625, 0xC000 = -2.0 ; a transposed / misread half would change the result
    row = np.array([0x4049, 0xC000, 0x0000], np.uint16)
    s = oracle.row_stats(row)
    ref = oracle.row_stats(f32row([3.140625, -2.0, 0.0]))
    assert s["cand"] == 0 and s["conf"] == ref["conf"] and s["entropy"] == ref["entropy"]


# ------------------------------------------------------------------------------ one step --------
def rows_with_conf(confs, V=2, dtype=np.float32):
    """[n, V] logits whose row i has arg-max 1 and confidence confs[i]: logits (0, ln(c/(1-c)), -inf...)."""
    n = len(confs)
    x = np.full((n, V), -np.inf, dtype)
    x[:, 0] = 0.0
    x[:, 1] = [math.log(c / (1 - c)) for c in confs]
    return x


def test_hand_worked_step_from_algorithm_2():
    """Block of 4, lambda 0.9, confidences (.95,.5,.92,.3): positions 0 and 2 are committed in
    parallel.  Next step (.6,.8) at positions 1,3: nobody clears, so the LEFTMOST masked position
    (1) is committed, not the most confident one (3) as Fast-dLLM (Algorithm 1) would."""
    st = oracle.StepState(1, 4)
    st.tokens[:] = -7
    lo, hi = np.array([0], np.int32), np.array([4], np.int32)
    logits = rows_with_conf([0.95, 0.5001, 0.92, 0.3]).reshape(1, 4, 2)
    logits[0, 3] = [math.log(0.7 / 0.3), 0.0]      # arg-max 0, confidence .7 -> still below lambda
    assert oracle.step(st, logits, lo, hi, 0.9, step_id=0) == 0
    assert st.mask.tolist() == [[0, 1, 0, 1]]
    assert st.tokens.tolist() == [[1, -7, 1, -7]]
    assert st.n_unmasked[0] == 2 and st.is_fallback[0] == 0 and st.fallback_pos[0] == -1
    assert st.commit_step.tolist() == [[0, -1, 0, -1]] and st.commit_fallback.tolist() == [[0, 255, 0, 255]]
    assert st.conf[0, 0] == pytest.approx(0.95, abs=1e-7) and st.conf[0, 3] == pytest.approx(0.7, abs=1e-7)
    assert st.commit_logp[0, 2] == pytest.approx(LN(0.92), abs=1e-7)
    assert st.nfe[0] == 1 and st.n_fallback[0] == 0
    logits = rows_with_conf([0.99, 0.6, 0.99, 0.8]).reshape(1, 4, 2)   # rows 0,2 are no longer masked
    assert oracle.step(st, logits, lo, hi, 0.9, step_id=1) == 0
    assert st.mask.tolist() == [[0, 0, 0, 1]]
    assert st.n_unmasked[0] == 1 and st.is_fallback[0] == 1 and st.fallback_pos[0] == 1
    assert st.commit_step.tolist() == [[0, 1, 0, -1]] and st.commit_fallback.tolist() == [[0, 1, 0, 255]]
    assert st.commit_logp[0, 1] == pytest.approx(LN(0.6), abs=1e-7)
    assert st.nfe[0] == 2 and st.n_fallback[0] == 1
    # confidence exactly AT the threshold is not committed (strict >): 0.5 = 1/(1+e^0) exactly
    st2 = oracle.StepState(1, 2)
    logits = np.zeros((1, 2, 2), np.float32)
    oracle.step(st2, logits, np.array([0], np.int32), np.array([2], np.int32), 0.5)
    assert st2.is_fallback[0] == 1 and st2.mask.tolist() == [[0, 1]]
    st3 = oracle.StepState(1, 2)
    oracle.step(st3, logits, np.array([0], np.int32), np.array([2], np.int32), np.nextafter(np.float32(0.5), 0))
    assert st3.is_fallback[0] == 0 and st3.mask.tolist() == [[0, 0]]


@pytest.mark.parametrize("seed", range(8))
def test_step_invariants_random(seed):
    """Exactly one commit, the leftmost, at a fallback step; otherwise exactly the positions above
    the threshold; nothing outside the block or already unmasked changes; untouched rows may hold
    NaN canaries."""
    rng = np.random.default_rng(seed)
    B, Lt, V = 5, 24, 37
    lam = float(rng.choice([0.3, 0.6, 0.9]))
    mask = (rng.random((B, Lt)) < 0.6).astype(np.uint8)
    lo = rng.integers(0, Lt - 8, size=B).astype(np.int32)
    hi = (lo + rng.integers(0, 9, size=B)).astype(np.int32)
    if seed == 0:
        mask[0, lo[0]:hi[0]] = 0                        # a sequence with nothing to do
    x = (rng.standard_normal((B, Lt, V)) * 2).astype(np.float32)
    peak = rng.random((B, Lt)) < 0.4
    x[peak, 5] += 9.0
    live = np.zeros((B, Lt), bool)
    for b in range(B):
        live[b, lo[b]:hi[b]] = mask[b, lo[b]:hi[b]] == 1
    x[~live] = np.nan                                   # canaries: must never be read
    st = oracle.StepState(B, Lt, tokens=np.full((B, Lt), -3, np.int32), mask=mask)
    assert oracle.step(st, x, lo, hi, lam, step_id=11) == 0
    p = scipy.special.softmax(np.where(live[..., None], x, 0.0).astype(np.float64), axis=-1)
    conf = p.max(-1)
    for b in range(B):
        act = np.flatnonzero(live[b])
        if len(act) == 0:
            assert st.n_unmasked[b] == 0 and st.is_fallback[b] == 0 and st.fallback_pos[b] == -1
            assert st.nfe[b] == 0
            continue
        above = [k for k in act if conf[b, k] > lam]
        want = above if above else [act[0]]
        got = [k for k in range(Lt) if mask[b, k] == 1 and st.mask[b, k] == 0]
        assert got == list(want)
        assert st.is_fallback[b] == (0 if above else 1)
        assert st.fallback_pos[b] == (-1 if above else act[0])
        assert st.n_unmasked[b] == len(want) and st.nfe[b] == 1 and st.n_fallback[b] == (0 if above else 1)
        for k in want:
            assert st.tokens[b, k] == int(np.argmax(x[b, k])) and st.commit_step[b, k] == 11
        np.testing.assert_allclose(st.conf[b, act], conf[b, act], rtol=1e-11)
    untouched = st.mask == mask
    assert (st.tokens[untouched] == -3).all() and (st.commit_step[untouched] == -1).all()
    assert np.isnan(st.conf[~live]).all()


def test_step_window_and_strides():
    """pos0 > 0: the logits buffer only covers a window of positions; row (b,k) is at k - pos0."""
    rng = np.random.default_rng(3)
    B, Lt, V, pos0, Ll = 2, 16, 11, 8, 4
    x = rng.standard_normal((B, Ll, V)).astype(np.float32)
    st = oracle.StepState(B, Lt)
    lo, hi = np.full(B, 8, np.int32), np.full(B, 12, np.int32)
    assert oracle.step(st, x, lo, hi, -1.0, pos0=pos0) == 0      # lambda < 0: everything is committed
    for b in range(B):
        assert st.tokens[b, 8:12].tolist() == np.argmax(x[b], -1).tolist()
        assert st.mask[b].tolist() == [1] * 8 + [0] * 4 + [1] * 4


# ----------------------------------------------------------------------------- the loop ---------
def scripted_provider(conf_of):
    """Rows with V=2: confidence conf_of(step,b,k) and arg-max token 1."""
    def prov(step, tokens, mask, lo, hi, logits):
        B, Ll, V = logits.shape
        logits[...] = np.nan
        for b in range(B):
            for k in range(lo[b], hi[b]):
                if mask[b, k]:
                    c = conf_of(step, b, k)
                    logits[b, k] = [0.0, math.log(c / (1 - c))]
        return 0
    return prov


def test_loop_threshold_above_one_is_left_to_right_decoding():
    """lambda >= 1 can never be exceeded, so every step is a fallback: one token per step, strictly
    left to right, T = number of masked positions (AR decoding, Section 2 'GRPO for masked dLLMs')."""
    B, Lt, BL = 3, 12, 4
    st = oracle.StepState(B, Lt)
    st.mask[1, :5] = 0
    st.mask[2, :] = 0                                    # already complete
    logits = np.zeros((B, Lt, 2), np.float32)
    rc, steps = oracle.decode_loop(st, logits, BL, 0, Lt, scripted_provider(lambda s, b, k: 0.97), 1.0, 100)
    assert rc == 0 and steps == 12
    assert st.nfe.tolist() == [12, 7, 0] and st.n_fallback.tolist() == [12, 7, 0]
    assert st.commit_step[0].tolist() == list(range(12))
    assert st.commit_step[1].tolist() == [-1] * 5 + list(range(7))
    assert (st.mask == 0).all() and (st.commit_fallback[0] == 1).all()


def test_loop_negative_threshold_commits_a_block_per_step():
    B, Lt, BL = 2, 10, 4                                 # blocks [0,4) [4,8) [8,10)
    st = oracle.StepState(B, Lt)
    st.mask[1, 0:4] = 0                                  # first block of sequence 1 is done
    logits = np.zeros((B, Lt, 2), np.float32)
    rc, steps = oracle.decode_loop(st, logits, BL, 0, Lt, scripted_provider(lambda s, b, k: 0.6), -0.5, 100)
    assert rc == 0 and steps == 3 and st.nfe.tolist() == [3, 2] and st.n_fallback.tolist() == [0, 0]
    assert st.commit_step[0].tolist() == [0] * 4 + [1] * 4 + [2] * 2
    assert st.commit_step[1].tolist() == [-1] * 4 + [0] * 4 + [1] * 2


def test_loop_scripted_trajectory_counted_by_hand():
    """One sequence, two blocks of 4, lambda .9.  Position k is 'confident' (0.95) only once every
    position to its left in the block is committed, except position 0 and 2 of each block which are
    confident from the start.  By hand: step 0 commits {0,2}; step 1: 1 is now confident (0 is
    committed) -> commits {1}; step 2: 3 confident -> {3}.  Same for the second block: 6 steps, no
    fallback.  With positions 1 and 5 never confident: block = {0,2}, fallback 1, then {3}."""
    Lt, BL = 8, 4

    def conf_a(step, b, k, mask_holder=[]):
        return 0.95
    st = oracle.StepState(1, Lt)
    logits = np.zeros((1, Lt, 2), np.float32)

    def prov(step, tokens, mask, lo, hi, lg):
        lg[...] = np.nan
        for k in range(lo[0], hi[0]):
            if mask[0, k]:
                j = k % BL
                ok = j in (0, 2) or all(mask[0, lo[0]:k] == 0)
                c = 0.95 if ok else 0.4
                lg[0, k] = [0.0, math.log(c / (1 - c))]
        return 0
    rc, steps = oracle.decode_loop(st, logits, BL, 0, Lt, prov, 0.9, 100)
    assert rc == 0 and steps == 6 and st.n_fallback[0] == 0
    assert st.commit_step[0].tolist() == [0, 1, 0, 2, 3, 4, 3, 5]

    st = oracle.StepState(1, Lt)

    def prov2(step, tokens, mask, lo, hi, lg):
        lg[...] = np.nan
        for k in range(lo[0], hi[0]):
            if mask[0, k]:
                j = k % BL
                ok = j in (0, 2) or (j == 3 and all(mask[0, lo[0]:k] == 0))
                c = 0.95 if ok else 0.4
                lg[0, k] = [0.0, math.log(c / (1 - c))]
        return 0
    rc, steps = oracle.decode_loop(st, logits, BL, 0, Lt, prov2, 0.9, 100)
    assert rc == 0 and steps == 6 and st.n_fallback[0] == 2
    assert st.commit_step[0].tolist() == [0, 1, 0, 2, 3, 4, 3, 5]
    assert st.commit_fallback[0].tolist() == [0, 1, 0, 0, 0, 1, 0, 0]
    # every step commits at least one token, so T <= number of masked positions; totals add up
    assert st.nfe[0] == 6 and (st.mask == 0).all()


def test_loop_max_steps_and_provider_error():
    st = oracle.StepState(1, 8)
    logits = np.zeros((1, 8, 2), np.float32)
    rc, steps = oracle.decode_loop(st, logits, 4, 0, 8, scripted_provider(lambda s, b, k: 0.6), 1.0, 3)
    assert rc == oracle.ERR_MAX_STEPS and steps == 3 and st.mask.sum() == 5
    st = oracle.StepState(1, 8)
    calls = []

    def failing(step, *a):
        calls.append(step)
        return 0 if step < 2 else 9
    prov = scripted_provider(lambda s, b, k: 0.6)
    rc, steps = oracle.decode_loop(st, logits, 4, 0, 8,
                                   lambda s, *a: (prov(s, *a) if s < 2 else 9), 1.0, 100)
    assert rc == oracle.ERR_PROVIDER and steps == 2 and st.mask.sum() == 6


def test_loop_generation_window_inside_a_longer_buffer():
    """Prompt positions (outside [gen_lo, gen_hi)) are never touched even when marked masked."""
    st = oracle.StepState(1, 12)
    logits = np.zeros((1, 12, 2), np.float32)
    rc, steps = oracle.decode_loop(st, logits, 4, 2, 11, scripted_provider(lambda s, b, k: 0.95), 0.9, 100)
    assert rc == 0 and steps == 3                       # blocks [2,6) [6,10) [10,11)
    assert st.mask[0].tolist() == [1, 1] + [0] * 9 + [1]


# --------------------------------------------------------------------------- log-likelihood -----
def test_logprob_matches_step_and_sums_in_order():
    rng = np.random.default_rng(5)
    B, Lt, V = 3, 10, 29
    x = (rng.standard_normal((B, Lt, V)) * 3).astype(np.float32)
    st = oracle.StepState(B, Lt)
    lo, hi = np.zeros(B, np.int32), np.full(B, Lt, np.int32)
    oracle.step(st, x, lo, hi, -1.0)                    # commits the arg-max everywhere
    select = (rng.random((B, Lt)) < 0.5).astype(np.uint8)
    select[2] = 0
    rc, lp, ssum, scnt, status = oracle.logprob(x, st.tokens, select)
    assert rc == 0 and (status == 0).all()
    sel = select.astype(bool)
    np.testing.assert_allclose(lp[sel], st.commit_logp[sel], rtol=1e-13)
    assert (lp[~sel] == 0).all()
    assert scnt.tolist() == select.sum(1).tolist() and ssum[2] == 0.0
    np.testing.assert_allclose(ssum, np.where(sel, lp, 0).sum(1), rtol=1e-13)
    # any token: library log-softmax
    toks = rng.integers(0, V, size=(B, Lt)).astype(np.int32)
    rc, lp, ssum, scnt, status = oracle.logprob(x, toks, np.ones((B, Lt), np.uint8))
    ref = scipy.special.log_softmax(x.astype(np.float64), axis=-1)
    np.testing.assert_allclose(lp, np.take_along_axis(ref, toks[..., None].astype(np.int64), -1)[..., 0], rtol=1e-12)
    toks[1, 4] = V
    rc, lp, ssum, scnt, status = oracle.logprob(x, toks, np.ones((B, Lt), np.uint8))
    assert status[1, 4] & oracle.ROW_BAD_TOKEN and lp[1, 4] == 0.0 and scnt[1] == Lt


def test_head_logits_is_the_plain_product():
    """oracle.head_logits against what fixes it: an identity-like weight returns the hidden states,
    and a small case equals the triple loop in exact rational arithmetic rounded once to fp32."""
    from fractions import Fraction
    rng = np.random.default_rng(5)
    d, V, n = 8, 11, 3
    eye = np.zeros((d, d), np.float32)
    np.fill_diagonal(eye, 1.0)
    h = fs.f32_to_bf16_bits(rng.standard_normal((n, d)).astype(np.float32))
    assert (oracle.head_logits(h, fs.f32_to_bf16_bits(eye)) == fs.bf16_bits_to_f32(h)).all()
    w = fs.f32_to_bf16_bits(rng.standard_normal((V, d)).astype(np.float32))
    got = oracle.head_logits(h, w)
    hf, wf = fs.bf16_bits_to_f32(h), fs.bf16_bits_to_f32(w)
    for i in range(n):
        for v in range(V):
            exact = sum(Fraction(float(hf[i, j])) * Fraction(float(wf[v, j])) for j in range(d))
            assert got[i, v] == np.float32(float(exact))
    assert got.dtype == np.float32 and got.shape == (n, V)
