"""Pins for the oracle's variants of the sampling step and for the ForkGRPO objective (CPU only).

Each part is checked against something other than itself: the grid and a chi-square of the uniform
stream, softmax(x/tau) from scipy for the drawn candidates (one slice and several), the draw
recomputed here by a numpy cumulative sum along the stated order, hand-worked fallback choices
(Algorithm 1 versus Algorithm 2), numpy sorting for the selections, hand-worked advantages and
clipping cases of Eq. 2, and finite differences for both derivatives.
"""
import math

import numpy as np
import pytest
from scipy.special import log_softmax, softmax

import oracle


def two_logit_rows(confs, V=2):
    """fp32 rows whose largest softmax probability is conf (V=2: gap = logit(conf))."""
    rows = np.zeros((len(confs), V), np.float32)
    for i, c in enumerate(confs):
        rows[i, 1] = math.log(c / (1.0 - c))
    return rows


def one_block_state(rows, masked):
    """B=1, one block over len(rows) positions, the given positions masked."""
    n, V = rows.shape
    st = oracle.StepState(1, n, mask=np.array([[1 if k in masked else 0 for k in range(n)]], np.uint8))
    logits = np.ascontiguousarray(rows.reshape(1, n, V))
    return st, logits, np.zeros(1, np.int32), np.full(1, n, np.int32)


# ---- uniform stream -------------------------------------------------------------------------
def test_uniform_stream_grid_uniformity_independence():
    n = 60000
    u = np.array([oracle.noise(1234, 3, k // 256, k % 256) for k in range(n)])     # rows (b, k) of one step
    for col in (0, 1):
        assert u[:, col].min() > 0.0 and u[:, col].max() < 1.0
        grid = u[:, col] * 2.0 ** 23 - 0.5
        assert np.all(grid == np.round(grid))                  # midpoints of the 2^-23 grid
        counts, _ = np.histogram(u[:, col], bins=64, range=(0.0, 1.0))
        chi2 = float(((counts - n / 64) ** 2 / (n / 64)).sum())
        assert chi2 < 130.0                                    # 63 degrees of freedom, p ~ 1e-6
        assert abs(u[:, col].mean() - 0.5) < 0.01 and abs(u[:, col].var() - 1.0 / 12.0) < 0.005
        assert abs(np.corrcoef(u[:-1, col], u[1:, col])[0, 1]) < 0.02      # neighbouring positions
    assert abs(np.corrcoef(u[:, 0], u[:, 1])[0, 1]) < 0.02                # the token's and the slice's uniform
    joint, _, _ = np.histogram2d(u[:, 0], u[:, 1], bins=8, range=((0, 1), (0, 1)))
    assert float(((joint - n / 64) ** 2 / (n / 64)).sum()) < 130.0
    # other steps and seeds are uncorrelated
    base = u[:20000, 0]
    other = np.array([oracle.noise(1234, 4, k // 256, k % 256)[0] for k in range(20000)])
    assert abs(np.corrcoef(base, other)[0, 1]) < 0.03
    other = np.array([oracle.noise(1235, 3, k // 256, k % 256)[0] for k in range(20000)])
    assert abs(np.corrcoef(base, other)[0, 1]) < 0.03


def visiting_order(v0, v1, group):
    """The order in which a slice [v0, v1) is laid out: groups of `group` entries dealt to 256 lanes
    round robin, lane after lane, the left-over entries last (written here independently of the oracle)."""
    n = v1 - v0
    ngroups = n // group
    order = []
    for lane in range(256):
        for j in range(lane, ngroups, 256):
            order.extend(range(v0 + j * group, v0 + (j + 1) * group))
    order.extend(range(v0 + ngroups * group, v1))
    return np.array(order, np.int64)


def draw_by_cumsum(x, tau, u, order):
    w = np.exp((x[order].astype(np.float64) - x.astype(np.float64).max()) / tau)
    c = np.cumsum(w)
    i = int(np.searchsorted(c, u * c[-1], side="left"))
    lo = c[i - 1] if i > 0 else 0.0
    return int(order[i]), min(u * c[-1] - lo, c[i] - u * c[-1]) / c[-1], float(c[-1])


# ---- stochastic candidates --------------------------------------------------------------------
@pytest.mark.parametrize("tau", [0.7, 1.3])
def test_sampled_candidates_follow_tempered_softmax(tau):
    x = np.array([2.0, 1.0, 0.5, 0.0, -1.0, 1.5], np.float32)
    B, Lt, V = 32, 64, x.shape[0]
    logits = np.ascontiguousarray(np.broadcast_to(x, (B, Lt, V))).copy()
    counts = np.zeros(V)
    p_plain = softmax(x.astype(np.float64))
    for step_id in range(4):
        st = oracle.StepState(B, Lt)
        rc = oracle.step(st, logits, np.zeros(B, np.int32), np.full(B, Lt, np.int32), threshold=-1.0,
                         step_id=step_id, temperature=tau, sample_seed=99)
        assert rc == 0
        assert np.all(st.mask == 0)                            # threshold < 0: everything commits
        counts += np.bincount(st.tokens.ravel(), minlength=V)
        # confidence and log-probability are those of the drawn token under the UNtempered softmax
        assert np.allclose(st.conf, p_plain[st.tokens], rtol=1e-12)
        assert np.allclose(st.logp, np.log(p_plain[st.tokens]), atol=1e-12)
        assert np.allclose(st.entropy, -(p_plain * np.log(p_plain)).sum(), atol=1e-12)
    n = counts.sum()
    expect = softmax(x.astype(np.float64) / tau) * n
    chi2 = float(((counts - expect) ** 2 / expect).sum())
    assert chi2 < 30.0                                         # 5 degrees of freedom, p ~ 1e-5
    greedy = np.zeros(V)
    greedy[0] = n
    assert float(((counts - greedy) ** 2).sum()) > 1e5          # and it is not the arg-max sampler


def test_sampling_limits_and_the_draw_recomputed():
    rng = np.random.default_rng(5)
    B, Lt, V = 2, 16, 5003                                     # 625 groups of 8: more than one round of the 256 lanes, 3 left over
    for dtype, group in ((np.float32, 4), (np.uint16, 8)):
        xf = rng.normal(0, 2, (B, Lt, V)).astype(np.float32)
        if dtype is np.uint16:
            u32 = xf.view(np.uint32).astype(np.uint64)
            logits = ((u32 + 0x7FFF + ((u32 >> 16) & 1)) >> 16).astype(np.uint16)
            xf = (logits.astype(np.uint32) << 16).view(np.float32)
        else:
            logits = xf
        lo, hi = np.zeros(B, np.int32), np.full(B, Lt, np.int32)
        cold = oracle.StepState(B, Lt)
        oracle.step(cold, logits, lo, hi, -1.0, temperature=1e-3, sample_seed=1)
        picked = np.take_along_axis(xf, cold.tokens[..., None].astype(np.int64), -1)[..., 0]
        assert np.array_equal(picked, xf.max(-1))                # tau -> 0 draws a maximum (any of them when bf16 values tie)
        zero = oracle.StepState(B, Lt)
        oracle.step(zero, logits, lo, hi, -1.0, temperature=0.0, sample_seed=1)
        assert np.array_equal(zero.tokens, xf.argmax(-1)) and np.all(np.isinf(zero.sample_margin))
        warm = oracle.StepState(B, Lt)
        oracle.step(warm, logits, lo, hi, -1.0, temperature=1.0, sample_seed=1)
        order = visiting_order(0, V, group)
        assert sorted(order.tolist()) == list(range(V))
        for b in range(B):
            for k in range(Lt):
                tok, margin, _ = draw_by_cumsum(xf[b, k], 1.0, oracle.noise(1, 0, b, k)[0], order)
                assert warm.tokens[b, k] == tok
                assert math.isclose(warm.sample_margin[b, k], margin, rel_tol=1e-6, abs_tol=1e-12)
        # a different seed gives different draws
        other = oracle.StepState(B, Lt)
        oracle.step(other, logits, lo, hi, -1.0, temperature=1.0, sample_seed=2)
        assert not np.array_equal(other.tokens, warm.tokens)
        # the vocabulary in three slices: the slice by its own uniform, the token inside it by the other
        cuts = np.array([0, 1672, 3344, V], np.int32)
        cut = oracle.StepState(B, Lt)
        oracle.step(cut, logits, lo, hi, -1.0, temperature=1.0, sample_seed=1, slices=cuts)
        for b in range(B):
            for k in range(Lt):
                u_tok, u_slice = oracle.noise(1, 0, b, k)
                draws = [draw_by_cumsum_slice(xf[b, k], 1.0, u_tok, int(cuts[r]), int(cuts[r + 1]), group) for r in range(3)]
                totals = np.cumsum([d[2] for d in draws])
                r = int(np.searchsorted(totals, u_slice * totals[-1], side="left"))
                assert cut.tokens[b, k] == draws[r][0]


def draw_by_cumsum_slice(x, tau, u, v0, v1, group):
    order = visiting_order(v0, v1, group)
    w = np.exp((x[order].astype(np.float64) - x.astype(np.float64).max()) / tau)
    c = np.cumsum(w)
    i = int(np.searchsorted(c, u * c[-1], side="left"))
    return int(order[i]), 0.0, float(c[-1])


def test_sampled_candidates_in_slices_follow_tempered_softmax():
    x = np.array([2.0, 1.0, 0.5, 0.0, -1.0, 1.5, 0.3, -0.4, 1.1, 0.9, -2.0], np.float32)
    B, Lt, V = 32, 64, x.shape[0]
    logits = np.ascontiguousarray(np.broadcast_to(x, (B, Lt, V))).copy()
    counts = np.zeros(V)
    for step_id in range(4):
        st = oracle.StepState(B, Lt)
        assert oracle.step(st, logits, np.zeros(B, np.int32), np.full(B, Lt, np.int32), threshold=-1.0, step_id=step_id,
                           temperature=0.9, sample_seed=7, slices=np.array([0, 4, 8, V], np.int32)) == 0
        counts += np.bincount(st.tokens.ravel(), minlength=V)
    expect = softmax(x.astype(np.float64) / 0.9) * counts.sum()
    assert float(((counts - expect) ** 2 / expect).sum()) < 40.0   # 10 degrees of freedom, p ~ 1e-5


def test_sampling_skips_minus_inf_and_flags_bad_rows():
    x = np.array([[0.0, -np.inf, 0.0, -np.inf], [np.nan, 1.0, 0.0, 0.0]], np.float32)
    st, logits, lo, hi = one_block_state(x, {0, 1})
    for seed in range(40):
        s2 = oracle.StepState(1, 2)
        oracle.step(s2, logits, lo, hi, -1.0, temperature=5.0, sample_seed=seed)
        assert s2.tokens[0, 0] in (0, 2)                       # never a probability-0 token
        assert s2.row_status[0, 1] & oracle.ROW_BAD and s2.conf[0, 1] == 0.0
        assert s2.tokens[0, 1] == 1                            # bad row: greedy candidate over the non-NaN entries


# ---- fallback orders -----------------------------------------------------------------------------
def test_fallback_orders_hand_worked_step():
    # Algorithm 1 against Algorithm 2 on the same state: positions 1 and 3 masked, c = (0.60, 0.80)
    rows = two_logit_rows([0.95, 0.60, 0.92, 0.80])
    expect = {oracle.FB_LEFTMOST: 1, oracle.FB_MAX_CONF: 3, oracle.FB_MIN_CONF: 1, oracle.FB_MAX_ENTROPY: 1}
    for mode, pos in expect.items():
        st, logits, lo, hi = one_block_state(rows, {1, 3})
        assert oracle.step(st, logits, lo, hi, 0.9, fallback_mode=mode) == 0
        assert st.is_fallback[0] == 1 and st.fallback_pos[0] == pos and st.n_unmasked[0] == 1
        assert st.mask[0].tolist() == [0, 0 if pos == 1 else 1, 0, 0 if pos == 3 else 1]
        assert st.commit_fallback[0, pos] == 1
    # entropy gap of the two rows, from the binary entropy function
    h = lambda c: -(c * math.log(c) + (1 - c) * math.log(1 - c))
    st, logits, lo, hi = one_block_state(rows, {1, 3})
    oracle.step(st, logits, lo, hi, 0.9, fallback_mode=oracle.FB_MAX_ENTROPY)
    assert math.isclose(st.fallback_margin[0], h(0.60) - h(0.80), abs_tol=1e-6)
    st, logits, lo, hi = one_block_state(rows, {1, 3})
    oracle.step(st, logits, lo, hi, 0.9, fallback_mode=oracle.FB_MAX_CONF)
    assert math.isclose(st.fallback_margin[0], 0.20, abs_tol=1e-6)
    for rand, pos in [(4, 1), (5, 3), (0xFFFFFFFF, 3)]:
        st, logits, lo, hi = one_block_state(rows, {1, 3})
        oracle.step(st, logits, lo, hi, 0.9, fallback_mode=oracle.FB_RANDOM, fallback_rand=np.array([rand], np.uint32))
        assert st.fallback_pos[0] == pos
    # a step that is not a fallback is the same under every order
    for mode in range(5):
        st, logits, lo, hi = one_block_state(rows, {0, 1, 2, 3})
        oracle.step(st, logits, lo, hi, 0.9, fallback_mode=mode, fallback_rand=np.array([7], np.uint32))
        assert st.is_fallback[0] == 0 and st.mask[0].tolist() == [0, 1, 0, 1] and np.isinf(st.fallback_margin[0])


def test_lowest_confidence_and_highest_entropy_differ():
    # row A: p = (.5, .5, 0): conf .5, H = ln 2.   row B: p = (.55, .225, .225): conf .55, H = 1.0000
    rows = np.array([[0.0, 0.0, -np.inf], np.log([0.55, 0.225, 0.225])], np.float32)
    st, logits, lo, hi = one_block_state(rows, {0, 1})
    oracle.step(st, logits, lo, hi, 0.9, fallback_mode=oracle.FB_MIN_CONF)
    assert st.fallback_pos[0] == 0
    st, logits, lo, hi = one_block_state(rows, {0, 1})
    oracle.step(st, logits, lo, hi, 0.9, fallback_mode=oracle.FB_MAX_ENTROPY)
    assert st.fallback_pos[0] == 1
    assert math.isclose(st.entropy[0, 0], math.log(2), abs_tol=1e-7)
    # ties go to the lower position; bad rows are passed over; all bad -> leftmost
    rows = two_logit_rows([0.7, 0.7, 0.7])
    for mode in (oracle.FB_MAX_CONF, oracle.FB_MIN_CONF, oracle.FB_MAX_ENTROPY):
        st, logits, lo, hi = one_block_state(rows, {1, 2})
        oracle.step(st, logits, lo, hi, 0.9, fallback_mode=mode)
        assert st.fallback_pos[0] == 1 and st.fallback_margin[0] == 0.0
    rows = two_logit_rows([0.6, 0.7, 0.8])
    rows[0, 0] = np.nan
    st, logits, lo, hi = one_block_state(rows, {0, 1, 2})
    oracle.step(st, logits, lo, hi, 0.9, fallback_mode=oracle.FB_MIN_CONF)
    assert st.fallback_pos[0] == 1
    rows[:, 0] = np.nan
    st, logits, lo, hi = one_block_state(rows, {1, 2})
    oracle.step(st, logits, lo, hi, 0.9, fallback_mode=oracle.FB_MAX_CONF)
    assert st.fallback_pos[0] == 1


def test_fallback_orders_against_numpy_on_random_loops():
    rng = np.random.default_rng(11)
    B, Lt, V, BL = 3, 24, 40, 8
    for mode in range(5):
        st = oracle.StepState(B, Lt)
        ref_mask = np.ones((B, Lt), np.uint8)
        rand = rng.integers(0, 2 ** 32, B, dtype=np.uint64).astype(np.uint32)
        step_logits = []

        def provider(step_id, tokens, mask, lo, hi, logits):
            # a few strong peaks, many flat rows: a mix of parallel and fallback steps
            x = rng.normal(0, 1, (B, Lt, V)).astype(np.float32)
            peak = rng.random((B, Lt)) < 0.4
            x[peak, 0] += 9.0
            logits[...] = x
            # the rule restated with numpy on the oracle's own confidences comes after the step
            step_logits.append((lo.copy(), hi.copy(), x))
            return 0

        logits = np.zeros((B, Lt, V), np.float32)
        rc, steps = oracle.decode_loop(st, logits, BL, 0, Lt, provider, 0.9, 500, fallback_mode=mode,
                                       fallback_rand=rand)
        assert rc == 0 and np.all(st.mask == 0)
        for step_id, (lo, hi, x) in enumerate(step_logits):
            p = softmax(x.astype(np.float64), axis=-1)
            conf = p.max(-1)
            ent = -(p * np.log(p)).sum(-1)
            for b in range(B):
                live = [k for k in range(lo[b], hi[b]) if ref_mask[b, k]]
                if not live:
                    continue
                above = [k for k in live if conf[b, k] > np.float64(np.float32(0.9))]
                if above:
                    chosen = above
                elif mode == oracle.FB_LEFTMOST:
                    chosen = [live[0]]
                elif mode == oracle.FB_RANDOM:
                    chosen = [live[int(rand[b]) % len(live)]]
                else:
                    key = {oracle.FB_MAX_CONF: conf[b, live], oracle.FB_MIN_CONF: -conf[b, live],
                           oracle.FB_MAX_ENTROPY: ent[b, live]}[mode]
                    chosen = [live[int(np.argmax(key))]]           # argmax returns the first maximum
                for k in chosen:
                    ref_mask[b, k] = 0
                    assert st.commit_step[b, k] == step_id, (mode, step_id, b, k)
                    assert st.commit_fallback[b, k] == (0 if above else 1)
        assert np.all(ref_mask == 0)


def test_threshold_one_with_fast_dllm_order_commits_by_confidence():
    confs = [0.55, 0.9, 0.7, 0.6, 0.8]
    rows = two_logit_rows(confs)
    st, logits, lo, hi = one_block_state(rows, set(range(5)))
    order = []
    for step_id in range(5):
        oracle.step(st, logits, lo, hi, 1.0, step_id=step_id, fallback_mode=oracle.FB_MAX_CONF)
        order.append(int(st.fallback_pos[0]))
    assert order == [1, 4, 2, 3, 0]                              # descending confidence


# ---- JustGRPO-Fast selection ---------------------------------------------------------------------
def test_top_entropy_selection_against_numpy():
    rng = np.random.default_rng(3)
    B, Lt = 5, 256
    H = rng.gamma(2.0, 1.0, (B, Lt)).astype(np.float32)
    H[1, 10:20] = H[1, 5]                                       # ties
    H[2, ::7] = np.nan
    elig = (rng.random((B, Lt)) < 0.8).astype(np.uint8)
    elig[3] = 1
    elig[4] = 0
    rc, sel, cnt = oracle.select_top_entropy(H, elig, 0.2)
    assert rc == 0
    for b in range(B):
        idx = np.flatnonzero(elig[b])
        n = len(idx)
        want = int(math.floor(float(np.float32(0.2)) * n))
        if n > 0:
            want = max(want, 1)
        assert cnt[b] == want == sel[b].sum()
        key = np.where(np.isnan(H[b, idx]), -np.inf, H[b, idx].astype(np.float64))
        order = idx[np.lexsort((idx, -key))]                      # entropy descending, then position ascending
        assert sorted(order[:want].tolist()) == np.flatnonzero(sel[b]).tolist()
    assert cnt[3] == 51 and cnt[4] == 0                           # floor(0.2 * 256)
    rc, sel, cnt = oracle.select_top_entropy(H[:1, :10], np.ones((1, 10), np.uint8), 0.2)
    assert cnt[0] == 2
    rc, sel, cnt = oracle.select_top_entropy(H[:1, :3], np.ones((1, 3), np.uint8), 0.2)
    assert cnt[0] == 1                                            # at least one position
    rc, sel, cnt = oracle.select_top_entropy(H[:1], elig[:1], 1.0)
    assert np.array_equal(sel, elig[:1])


# ---- ForkGRPO objective (Eq. 2) --------------------------------------------------------------------
def test_grpo_advantages_and_skipped_groups():
    B, Lt, G = 8, 4, 4
    lp = np.full((B, Lt), -1.0, np.float32)
    sel = np.zeros((B, Lt), np.uint8)
    sel[:, 1] = 1
    reward = np.array([1, 0, 0, 1, 0.5, 0.5, 0.5, 0.5], np.float32)
    r = oracle.grpo_loss(lp, lp, sel, reward, G, 0.2, 0.2)
    assert r["rc"] == 0
    assert np.allclose(r["adv"][:4], [1, -1, -1, 1]) and np.all(r["adv"][4:] == 0)
    assert r["skipped"].tolist() == [0, 1]
    assert np.allclose(r["ratio"][:, 1], 1.0) and np.all(r["ratio"][:, 0] == 0)
    assert np.allclose(r["seq_obj"], r["adv"])                  # rho = 1: the term is the advantage
    assert abs(r["objective"]) < 1e-15
    assert np.allclose(r["dlogp"][:4, 1], np.array([1, -1, -1, 1]) / (B * 1))
    assert np.all(r["dlogp"][4:] == 0)
    # population standard deviation: rewards (3, 1) -> mean 2, std 1
    r = oracle.grpo_loss(lp[:2], lp[:2], sel[:2], np.array([3, 1], np.float32), 2, 0.2, 0.2)
    assert np.allclose(r["adv"], [1, -1])
    # unequal group: (1, 0, 0, 0) -> mean .25, std sqrt(3)/4
    r = oracle.grpo_loss(lp[:4], lp[:4], sel[:4], np.array([1, 0, 0, 0], np.float32), 4, 0.2, 0.2)
    assert np.allclose(r["adv"], np.array([0.75, -0.25, -0.25, -0.25]) / (math.sqrt(3) / 4))


def test_every_position_selected_is_the_justgrpo_objective():
    """Eq. 1 (JustGRPO) is Eq. 2 with F_i = all L positions: the same call with every position selected against the
    formula of Eq. 1 written out with numpy (one group statistic per prompt, a mean over positions, a mean over rollouts)."""
    rng = np.random.default_rng(11)
    P, G, L, eps = 3, 4, 7, float(np.float32(0.2))            # (the clip range is passed in fp32)
    B = P * G
    old = rng.normal(-1.5, 0.5, (B, L)).astype(np.float32)
    new = (old + rng.normal(0, 0.3, (B, L))).astype(np.float32)
    reward = rng.random(B).astype(np.float32)
    r = oracle.grpo_loss(new, old, np.ones((B, L), np.uint8), reward, G, eps, eps)
    rho = np.exp(new.astype(np.float64) - old.astype(np.float64))
    rg = reward.astype(np.float64).reshape(P, G)
    adv = ((rg - rg.mean(1, keepdims=True)) / rg.std(1, keepdims=True)).reshape(B, 1)
    want = np.minimum(rho * adv, np.clip(rho, 1 - eps, 1 + eps) * adv).mean(1).mean()
    assert abs(r["objective"] - want) <= 1e-12 * max(1.0, abs(want))
    assert np.allclose(r["seq_obj"], np.minimum(rho * adv, np.clip(rho, 1 - eps, 1 + eps) * adv).mean(1), rtol=1e-12, atol=1e-14)


def test_grpo_clipping_cases_and_fallback_count_average():
    B, Lt, G = 2, 3, 2
    old = np.zeros((B, Lt), np.float32)
    new = np.zeros((B, Lt), np.float32)
    new[:, 0] = math.log(1.5)      # above 1 + eps
    new[:, 1] = math.log(0.5)      # below 1 - eps
    new[:, 2] = math.log(1.1)      # inside
    sel = np.ones((B, Lt), np.uint8)
    sel[1, 2] = 0                   # rollout 1 has two fallback steps, rollout 0 three
    r = oracle.grpo_loss(new, old, sel, np.array([1, 0], np.float32), G, 0.2, 0.2)
    # rollout 0, A = +1: min(1.5, 1.2) = 1.2 ; min(0.5, 0.8) = 0.5 ; 1.1
    assert math.isclose(r["seq_obj"][0], (1.2 + 0.5 + 1.1) / 3, rel_tol=1e-6)
    # rollout 1, A = -1: min(-1.5, -1.2) = -1.5 ; min(-0.5, -0.8) = -0.8
    assert math.isclose(r["seq_obj"][1], (-1.5 - 0.8) / 2, rel_tol=1e-6)
    assert math.isclose(r["objective"], (r["seq_obj"][0] + r["seq_obj"][1]) / 2, rel_tol=1e-12)
    d = r["dlogp"]
    assert d[0, 0] == 0.0 and math.isclose(d[0, 1], 0.5 / (2 * 3), rel_tol=1e-6) and math.isclose(d[0, 2], 1.1 / 6, rel_tol=1e-6)
    assert math.isclose(d[1, 0], -1.5 / (2 * 2), rel_tol=1e-6) and d[1, 1] == 0.0 and d[1, 2] == 0.0
    # a rollout without fallback steps contributes nothing and divides by nothing
    sel[1] = 0
    r = oracle.grpo_loss(new, old, sel, np.array([1, 0], np.float32), G, 0.2, 0.2)
    assert r["seq_obj"][1] == 0.0 and np.all(r["dlogp"][1] == 0) and np.isfinite(r["objective"])


def test_grpo_derivative_by_finite_differences():
    rng = np.random.default_rng(8)
    B, Lt, G = 6, 5, 3
    old = rng.normal(-2, 0.5, (B, Lt)).astype(np.float32)
    new = (old + rng.normal(0, 0.15, (B, Lt))).astype(np.float32)
    sel = (rng.random((B, Lt)) < 0.6).astype(np.uint8)
    reward = rng.random(B).astype(np.float32)
    base = oracle.grpo_loss(new, old, sel, reward, G, 0.2, 0.2)
    h = 2.0 ** -7                                                # exactly representable fp32 steps
    for i in range(B):
        for k in range(Lt):
            up, dn = new.copy(), new.copy()
            up[i, k] += h
            dn[i, k] -= h
            num = (oracle.grpo_loss(up, old, sel, reward, G, 0.2, 0.2)["objective"] -
                   oracle.grpo_loss(dn, old, sel, reward, G, 0.2, 0.2)["objective"]) / (float(up[i, k]) - float(dn[i, k]))
            rho = base["ratio"][i, k]
            near_kink = sel[i, k] and min(abs(rho - 0.8), abs(rho - 1.2)) < 0.02
            if not near_kink:
                assert math.isclose(num, base["dlogp"][i, k], rel_tol=2e-4, abs_tol=1e-7), (i, k)


def test_row_logp_gradient():
    rng = np.random.default_rng(2)
    V = 12
    x = rng.normal(0, 2, V).astype(np.float32)
    tok, w = 5, -0.37
    g = oracle.row_logp_grad(x, tok, w)
    p = softmax(x.astype(np.float64))
    onehot = np.eye(V)[tok]
    assert np.allclose(g, w * (onehot - p), atol=1e-14)
    assert abs(g.sum()) < 1e-14                                  # shifts of the logits change nothing
    h = 2.0 ** -6
    for v in range(V):
        up, dn = x.copy(), x.copy()
        up[v] += h
        dn[v] -= h
        num = w * (oracle.row_logp(up, tok)[0] - oracle.row_logp(dn, tok)[0]) / (float(up[v]) - float(dn[v]))
        assert math.isclose(num, g[v], rel_tol=1e-3, abs_tol=1e-5)
    # uniform row: 1[v = tok] - 1/V ; bf16 rows ; -inf entries get no gradient
    g = oracle.row_logp_grad(np.zeros(8, np.float32), 3, 2.0)
    assert np.allclose(g, 2.0 * (np.eye(8)[3] - 0.125))
    bits = (np.array([1.0, 2.0, -np.inf, 0.5], np.float32).view(np.uint32) >> 16).astype(np.uint16)
    g = oracle.row_logp_grad(bits, 1, 1.0)
    assert g[2] == 0.0 and abs(g.sum()) < 1e-14
    assert math.isclose(oracle.row_lse(x), float(np.log(np.exp(x.astype(np.float64)).sum())), rel_tol=1e-13)
    assert math.isclose(oracle.row_lse(x), float(x[tok]) - float(log_softmax(x.astype(np.float64))[tok]), rel_tol=1e-12)
