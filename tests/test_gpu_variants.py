"""The variants of the sampling step on the GPU against the oracle, through the C ABI: the
fallback orders the paper compares Fork-dLLM with (Algorithm 1 and the ablations of Section 4.1).
Inputs are re-drawn until every decision has a clear margin in the oracle (threshold, fallback
ranking), so that fp32 and fp64 take the same one."""
import numpy as np
import pytest
import torch

import fork_synth as fs
import oracle
from helpers import (assert_close, assert_equal, FALLBACK_MARGIN, compare_step_state, decisions_are_clear, live_mask,
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


# ---- stochastic candidates (temperature > 0) -----------------------------------------------------
def sample_both(x, mask, lo, hi, lam, tau, seed, step=3, pos0=0, logits_t=None):
    """One step with drawn candidates on both sides; None for the GPU side when some decision of
    the oracle (threshold, winning perturbed key) has no clear margin."""
    pkg = F()
    B, Ll, V = x.shape
    Lt = mask.shape[1]
    o = oracle.StepState(B, Lt, mask=mask)
    assert oracle.step(o, x, lo, hi, lam, step_id=step, pos0=pos0, temperature=tau, sample_seed=seed) == 0
    if not decisions_are_clear(o, live_mask(mask, lo, hi), lam, 1e-4, 0, tau):
        return None, o
    g = pkg.ForkState(B, Lt, mask=mask)
    keep = [torch.from_numpy(np.asarray(a)).cuda() for a in (lo, hi)]
    lg = to_torch_logits(x) if logits_t is None else logits_t
    pkg.fork_step(g, lg, keep[0], keep[1], lam, step=step, pos0=pos0, temperature=tau, sample_seed=seed)
    torch.cuda.synchronize()
    return g.host(), o


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("V", [2, 7, 8, 1023, 1024, 2049, 4104, 6151, 40000])
def test_sampled_step_small_vocabularies(V, dtype):
    """Aligned V takes the bulk-copy ring, unaligned V the scalar path; several chunks, ragged tails."""
    done = 0
    for seed in range(20):
        rng = np.random.default_rng(V * 7 + seed)
        B, Lt = 4, 24
        mask = (rng.random((B, Lt)) < 0.7).astype(np.uint8)
        lo = rng.integers(0, 10, size=B).astype(np.int32)
        hi = (lo + rng.integers(0, 14, size=B)).astype(np.int32)
        x = make_rows(rng, (B, Lt), V, dtype, peak=6.0)
        g, o = sample_both(x, mask, lo, hi, 0.9 if V > 8 else 0.45, tau=[0.8, 1.3][seed % 2], seed=1000 + seed)
        if g is None:
            continue
        compare_step_state(g, o)
        done += 1
        if done == 3:
            return
    raise AssertionError("too few inputs with clear margins")


def test_sampled_step_full_vocabulary_rows_span_many_ctas():
    """V = 126464 bf16: every row is cut into parts over several CTAs; the drawn token must come out
    of their lane sums taken together."""
    w = fs.workload("b8")
    B, Lt, V = 2, 8, w.V
    cfg = w.cfg(B=B)
    mask = np.ones((B, Lt), np.uint8)
    lo, hi = np.zeros(B, np.int32), np.full(B, Lt, np.int32)
    for nonce in range(8):
        x = np.empty((B, Lt, V), np.uint16)
        for b in range(B):
            for l in range(Lt):
                x[b, l] = fs.row_host(cfg, 0, b, l, nonce=nonce)
        g, o = sample_both(x, mask, lo, hi, w.threshold, tau=0.8, seed=77)
        if g is None:
            continue
        compare_step_state(g, o)
        return
    raise AssertionError("no input with clear margins found")


def test_sampled_step_with_banned_token_ranges():
    """-inf logits (banned tokens) can never be drawn; threads that meet them take their clamped path.
    The rows are flat enough for most draws to land on a low-probability token, where fp32 and fp64
    running sums may pick neighbours: every position commits (threshold below 0), positions whose draw
    has a clear margin are compared with the oracle, all of them with the ban."""
    pkg = F()
    from helpers import SAMPLE_MARGIN
    checked = 0
    for seed in range(4):
        rng = np.random.default_rng(50 + seed)
        B, Lt, V = 2, 6, 8200
        mask = np.ones((B, Lt), np.uint8)
        lo, hi = np.zeros(B, np.int32), np.full(B, Lt, np.int32)
        x = make_rows(rng, (B, Lt), V, "f32", peak=3.0)
        x[:, :, 100:3000] = -np.inf
        x[0, 2, :] = -np.inf
        x[0, 2, 4097] = 1.0                                     # a single allowed token
        o = oracle.StepState(B, Lt, mask=mask)
        assert oracle.step(o, x, lo, hi, -1.0, step_id=3, temperature=1.5, sample_seed=seed) == 0
        st = pkg.ForkState(B, Lt, mask=mask)
        pkg.fork_step(st, to_torch_logits(x), torch.from_numpy(lo).cuda(), torch.from_numpy(hi).cuda(), -1.0, step=3,
                      temperature=1.5, sample_seed=seed)
        torch.cuda.synchronize()
        g = st.host()
        assert (g["mask"] == 0).all()
        assert g["cand"][0, 2] == 4097 and not ((g["cand"] >= 100) & (g["cand"] < 3000)).any()
        clear = o.sample_margin >= SAMPLE_MARGIN
        assert_equal("cand", g["cand"], o.cand, where=clear)
        assert_equal("tokens", g["tokens"], o.tokens, where=clear)
        for name in ("conf", "logp", "entropy"):
            assert_close(name, g[name], getattr(o, name), where=clear)
        assert_close("entropy", g["entropy"], o.entropy)         # (does not depend on the draw)
        checked += int(clear.sum())
    assert checked >= 12


@pytest.mark.parametrize("V,dtype", [(6, "f32"), (8, "f32"), (16, "bf16")])
def test_sampled_candidates_follow_tempered_softmax_on_the_gpu(V, dtype):
    """Distribution pin of the CUDA sampler on its own: frequencies against scipy's softmax(x/tau)."""
    from scipy.special import softmax
    pkg = F()
    rng = np.random.default_rng(V)
    xrow = rng.normal(0, 1.5, V).astype(np.float32)
    if dtype == "bf16":
        xrow = fs.bf16_bits_to_f32(fs.f32_to_bf16_bits(xrow))
    B, Lt, tau = 64, 128, 0.9
    x = np.ascontiguousarray(np.broadcast_to(xrow, (B, Lt, V))).copy()
    xt = to_torch_logits(x if dtype == "f32" else fs.f32_to_bf16_bits(x))
    lo = torch.zeros(B, dtype=torch.int32, device="cuda")
    hi = torch.full((B,), Lt, dtype=torch.int32, device="cuda")
    counts = np.zeros(V)
    for step in range(3):
        st = pkg.ForkState(B, Lt)
        pkg.fork_step(st, xt, lo, hi, -1.0, step=step, temperature=tau, sample_seed=4242)
        torch.cuda.synchronize()
        h = st.host()
        assert (h["mask"] == 0).all()
        counts += np.bincount(h["tokens"].ravel(), minlength=V)
        p_plain = softmax(xrow.astype(np.float64))
        assert np.allclose(h["conf"], p_plain[h["tokens"]], rtol=1e-4, atol=1e-6)
    n = counts.sum()
    expect = softmax(xrow.astype(np.float64) / tau) * n
    chi2 = float(((counts - expect) ** 2 / expect).sum())
    assert chi2 < 3.0 * V + 25.0, (chi2, counts, expect)


def test_tiny_decode_loop_with_sampled_candidates():
    w = fs.workload("tiny")
    B, tau, seed = 4, 0.8, 2024
    ost, nonces, osteps, _ = oracle_reference_loop(w, B, w.threshold, temperature=tau, sample_seed=seed)
    pkg = F()
    cfg = w.cfg(B=B)
    logits = torch.empty((B, w.Lt, w.V), dtype=torch.float32, device="cuda")
    st = pkg.ForkState(B, w.Lt)
    prov = fs.Provider(cfg, w.Lt * w.V, w.V, 0, w.Lt, nonce=nonces)
    rc, steps = pkg.fork_decode_loop(st, logits, w.block_len, 0, w.Lt, prov.address, prov.ctx, w.threshold, 10000,
                                     temperature=tau, sample_seed=seed)
    torch.cuda.synchronize()
    prov.close()
    assert rc == 0 and steps == osteps
    h = st.host()
    compare_step_state(h, ost)
    assert (h["tokens"] == h["cand"]).all()
    greedy, _, _, _ = oracle_reference_loop(w, B, w.threshold)
    assert (greedy.tokens != ost.tokens).any()                 # the draws are not the arg-max everywhere


# ---- vocabulary-parallel slices (ranks emulated one after the other on one GPU) -------------------
def shard_offsets(V, n_ranks, elem_size):
    shards = F().vocab_shards(V, n_ranks, elem_size)
    return np.array([off for off, _ in shards] + [V], np.int32)


def vp_both(x, mask, lo, hi, lam, n_ranks, **variant):
    """fork_vp_reduce on every slice in turn, then fork_vp_select, against the oracle on the whole
    vocabulary."""
    pkg = F()
    B, Ll, V = x.shape
    Lt = mask.shape[1]
    o = oracle.StepState(B, Lt, mask=mask)
    ov = dict(variant)
    if "fallback_rand" in ov:
        ov["fallback_rand"] = ov["fallback_rand"].cpu().numpy().view(np.uint32)
    if variant.get("temperature", 0.0) > 0:                     # how the vocabulary is cut fixes the order the draw visits it in
        ov["slices"] = shard_offsets(V, n_ranks, 2 if x.dtype == np.uint16 else 4)
    assert oracle.step(o, x, lo, hi, lam, step_id=4, **ov) == 0
    if not decisions_are_clear(o, live_mask(mask, lo, hi), lam, 1e-4, variant.get("fallback_mode", 0),
                               variant.get("temperature", 0.0)):
        return None, o
    g = pkg.ForkState(B, Lt, mask=mask)
    xt = to_torch_logits(x)
    lo_d, hi_d = torch.from_numpy(np.asarray(lo)).cuda(), torch.from_numpy(np.asarray(hi)).cuda()
    parts, keys = [], []
    for off, n in pkg.vocab_shards(V, n_ranks, xt.element_size()):
        p_, k_ = pkg.fork_vp_reduce(g, xt[:, :, off:off + n], lo_d, hi_d, lam, off, step=4, **variant)
        parts.append(p_)
        keys.append(k_)
    torch.cuda.synchronize()
    assert (g.mask.cpu().numpy() == mask).all()                 # the local phase commits nothing
    keys_t = torch.stack(keys, 0) if keys[0] is not None else None
    pkg.fork_vp_select(g, torch.stack(parts, 0), keys_t, lo_d, hi_d, lam, step=4, Ll=Ll, **variant)
    torch.cuda.synchronize()
    return g.host(), o


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("V,n_ranks", [(4096, 2), (6151, 4), (40000, 8), (1000, 3)])
def test_vocab_parallel_step_equals_the_full_vocabulary_oracle(V, n_ranks, dtype):
    for seed in range(6):
        rng = np.random.default_rng(V + n_ranks + seed)
        B, Lt = 4, 40
        mask = (rng.random((B, Lt)) < 0.7).astype(np.uint8)
        lo = rng.integers(0, 10, size=B).astype(np.int32)
        hi = (lo + rng.integers(0, 36, size=B)).astype(np.int32)
        mask[2, lo[2]:hi[2]] = 0
        x = make_rows(rng, (B, Lt), V, dtype, peak=6.0)
        g, o = vp_both(x, mask, lo, hi, 0.9, n_ranks)
        if g is None:
            continue
        compare_step_state(g, o)
        return
    raise AssertionError("no input with clear margins found")


def test_vocab_parallel_special_rows():
    """Slices holding nothing but -inf, NaN / +inf in one slice, a row that is -inf everywhere, ties
    across slices (lowest global index), more than 32 live rows."""
    rng = np.random.default_rng(9)
    B, Lt, V, n_ranks = 2, 48, 4096, 4
    mask = np.ones((B, Lt), np.uint8)
    lo, hi = np.zeros(B, np.int32), np.full(B, Lt, np.int32)
    x = make_rows(rng, (B, Lt), V, "f32", peak=6.0)
    x[0, 0, :1024] = -np.inf                                  # first slice empty
    x[0, 1, 1024:] = -np.inf                                  # only the first slice holds anything
    x[0, 2, 2000] = np.nan
    x[0, 3, 3000] = np.inf
    x[0, 4, :] = -np.inf
    x[0, 5, :] = 0.0                                          # ties everywhere: index 0 wins
    top = x[0, 6].max() + 1.0
    x[0, 6, 1500] = top
    x[0, 6, 3500] = top                                       # tie across slices
    g, o = vp_both(x, mask, lo, hi, 0.9, n_ranks)
    assert g is not None
    compare_step_state(g, o)
    assert g["cand"][0, 5] == 0 and g["cand"][0, 6] == 1500 and g["row_status"][0, 4] == 1


@pytest.mark.parametrize("n_ranks", [2, 4])
def test_vocab_parallel_with_drawn_candidates_and_other_fallback_orders(n_ranks):
    done = 0
    for seed in range(12):
        rng = np.random.default_rng(300 + seed)
        B, Lt, V = 3, 20, 8192
        mask = np.ones((B, Lt), np.uint8)
        lo, hi = np.zeros(B, np.int32), np.full(B, Lt, np.int32)
        x = make_rows(rng, (B, Lt), V, "bf16", peak=4.0, peak_frac=0.3)
        rand = torch.from_numpy(rng.integers(0, 2 ** 31, B).astype(np.int32)).cuda()
        variant = [dict(temperature=0.8, sample_seed=5 + seed), dict(fallback_mode=1),
                   dict(temperature=1.2, sample_seed=seed, fallback_mode=3), dict(fallback_mode=4, fallback_rand=rand)][seed % 4]
        g, o = vp_both(x, mask, lo, hi, 0.9, n_ranks, **variant)
        if g is None:
            continue
        compare_step_state(g, o)
        done += 1
    assert done >= 6


@pytest.mark.parametrize("n_ranks,variant", [(2, {}), (4, dict(temperature=0.9, sample_seed=11)), (8, dict(fallback_mode=1))])
def test_vocab_parallel_with_the_exchange_fused_into_the_reduction(n_ranks, variant):
    """fork_vp_reduce_peers: every (emulated) rank's reduction kernel stores its slice results into
    slot `rank` of every rank's gather buffer; afterwards all gather buffers are identical and the
    select phase on each rank's own buffer reproduces the full-vocabulary oracle.  The ranks run one
    after the other on one GPU, each with its own replica of the state; the "peer" buffers are
    ordinary tensors of the same device."""
    pkg = F()
    done = 0
    for seed in range(8):
        rng = np.random.default_rng(500 + 10 * n_ranks + seed)
        B, Lt, V = 3, 40, 6151
        mask = (rng.random((B, Lt)) < 0.8).astype(np.uint8)
        lo = rng.integers(0, 6, size=B).astype(np.int32)
        hi = (lo + rng.integers(0, 34, size=B)).astype(np.int32)
        x = make_rows(rng, (B, Lt), V, "bf16", peak=6.0)
        o = oracle.StepState(B, Lt, mask=mask)
        ov = dict(variant, slices=shard_offsets(V, n_ranks, 2)) if variant.get("temperature", 0.0) > 0 else variant
        assert oracle.step(o, x, lo, hi, 0.9, step_id=4, **ov) == 0
        if not decisions_are_clear(o, live_mask(mask, lo, hi), 0.9, 1e-4, variant.get("fallback_mode", 0),
                                   variant.get("temperature", 0.0)):
            continue
        xt = to_torch_logits(x)
        lo_d, hi_d = torch.from_numpy(lo).cuda(), torch.from_numpy(hi).cuda()
        sampled = variant.get("temperature", 0.0) > 0
        gp = [torch.full((n_ranks, B, Lt, 4), float("nan"), device="cuda") for _ in range(n_ranks)]
        gk = [torch.full((n_ranks, B, Lt, 4), float("nan"), device="cuda") for _ in range(n_ranks)] if sampled else None
        states = [pkg.ForkState(B, Lt, mask=mask) for _ in range(n_ranks)]
        for r, (off, n) in enumerate(pkg.vocab_shards(V, n_ranks, xt.element_size())):
            pkg.fork_vp_reduce_peers(states[r], xt[:, :, off:off + n], lo_d, hi_d, 0.9, off, r, gp, gk, step=4, **variant)
        torch.cuda.synchronize()                                # stands for the barrier among real ranks
        for j in range(1, n_ranks):
            assert gp[j].cpu().numpy().tobytes() == gp[0].cpu().numpy().tobytes()
        for j in range(n_ranks):
            assert (states[j].mask.cpu().numpy() == mask).all()  # the local phase commits nothing
            pkg.fork_vp_select(states[j], gp[j], gk[j] if sampled else None, lo_d, hi_d, 0.9, step=4, Ll=Lt, **variant)
        torch.cuda.synchronize()
        for j in range(n_ranks):
            compare_step_state(states[j].host(), o)
        done += 1
        if done == 2:
            return
    raise AssertionError("no input with clear margins found")


def test_fused_exchange_rejects_bad_arguments():
    pkg = F()
    st = pkg.ForkState(1, 8)
    x = torch.zeros((1, 8, 64), dtype=torch.float32, device="cuda")
    lo, hi = torch.zeros(1, dtype=torch.int32).cuda(), torch.full((1,), 8, dtype=torch.int32).cuda()
    buf = [torch.zeros((2, 1, 8, 4), device="cuda") for _ in range(2)]
    with pytest.raises(pkg.ForkError):                         # rank outside the group
        pkg.fork_vp_reduce_peers(st, x, lo, hi, 0.9, 0, 2, buf)
    with pytest.raises(pkg.ForkError):                         # drawn candidates need key buffers
        pkg.fork_vp_reduce_peers(st, x, lo, hi, 0.9, 0, 0, buf, None, temperature=0.7, sample_seed=1)
    with pytest.raises(pkg.ForkError):                         # a null peer address
        pkg.fork_vp_reduce_peers(st, x, lo, hi, 0.9, 0, 0, [buf[0], 0])
