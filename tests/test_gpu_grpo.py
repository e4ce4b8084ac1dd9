"""ForkGRPO objective (Eq. 2) and the log-softmax backward on the GPU against the oracle."""
import numpy as np
import pytest
import torch

import fork_synth as fs
import oracle
from helpers import assert_close, to_torch_logits
from test_gpu_step import make_rows

pytestmark = pytest.mark.gpu


def F():
    import paper_2609_39859_b200 as pkg
    return pkg


def close(name, got, want, rtol, atol):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    ok = (np.isnan(got) & np.isnan(want)) | (np.abs(got - want) <= atol + rtol * np.abs(want))
    assert ok.all(), "%s: %d outside tolerance, e.g. got %s want %s" % (
        name, (~ok).sum(), got.ravel()[np.flatnonzero(~ok.ravel())[:4]], want.ravel()[np.flatnonzero(~ok.ravel())[:4]])


@pytest.mark.parametrize("B,Lt,G", [(32, 64, 8), (128, 256, 8), (6, 5, 3), (16, 33, 16)])
def test_grpo_loss_matches_the_oracle(B, Lt, G):
    pkg = F()
    eps_lo, eps_hi = 0.2, 0.28
    for seed in range(6):
        rng = np.random.default_rng(seed * 31 + B)
        old = rng.normal(-1.5, 0.7, (B, Lt)).astype(np.float32)
        new = (old + rng.normal(0, 0.2, (B, Lt))).astype(np.float32)
        sel = (rng.random((B, Lt)) < 0.2).astype(np.uint8)
        sel[1] = 0                                             # a rollout without fallback steps
        reward = (rng.random(B) < 0.5).astype(np.float32)
        reward[:G] = 1.0                                       # a group with equal rewards: skipped
        o = oracle.grpo_loss(new, old, sel, reward, G, eps_lo, eps_hi)
        rho = o["ratio"][sel != 0]
        if (np.abs(rho - (1 - np.float32(eps_lo))) < 1e-4).any() or (np.abs(rho - (1 + np.float32(eps_hi))) < 1e-4).any():
            continue                                           # a ratio on a clip boundary: fp32 may pick the other branch
        g = pkg.fork_grpo_loss(*(torch.from_numpy(x).cuda() for x in (new, old, sel, reward)), G, eps_lo, eps_hi)
        torch.cuda.synchronize()
        h = {k: v.cpu().numpy() for k, v in g.items()}
        assert np.array_equal(h["skipped"][: B // G], o["skipped"][: B // G]) and o["skipped"][0] == 1
        close("adv", h["adv"], o["adv"], 1e-5, 1e-6)
        close("ratio", h["ratio"], o["ratio"], 1e-5, 1e-7)
        close("seq_obj", h["seq_obj"], o["seq_obj"], 1e-4, 1e-6)
        close("objective", h["objective"][0], o["objective"], 1e-4, 1e-6)
        close("dlogp", h["dlogp"], o["dlogp"], 1e-4, 1e-9)
        assert (h["dlogp"][sel == 0] == 0).all() and (h["dlogp"][:G] == 0).all()
        return
    raise AssertionError("no input away from the clip boundaries")


def test_grpo_loss_rejects_bad_arguments():
    pkg = F()
    z = torch.zeros((4, 8), dtype=torch.float32, device="cuda")
    sel = torch.zeros((4, 8), dtype=torch.uint8, device="cuda")
    r = torch.zeros(4, dtype=torch.float32, device="cuda")
    for group, lo, hi in ((3, 0.2, 0.2), (0, 0.2, 0.2), (2, -0.1, 0.2), (2, 0.2, float("nan"))):
        with pytest.raises(pkg.ForkError) as e:
            pkg.fork_grpo_loss(z, z, sel, r, group, lo, hi)
        assert e.value.status == pkg.FORK_ERR_INVALID_ARG


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("V", [5, 8, 1000, 4096, 5003, 40000])
def test_logprob_backward_matches_the_oracle(V, dtype):
    """Score, then differentiate: rows of selected positions hold dlogp * (onehot - softmax), every
    other row keeps its canary.  Unaligned V takes the scalar path, the rest the 128-bit path with
    a ragged end."""
    pkg = F()
    rng = np.random.default_rng(V + (dtype == "f32"))
    B, Lt = 3, 12
    x = make_rows(rng, (B, Lt), V, dtype, peak=5.0)
    if V > 100:
        xf = x if dtype == "f32" else None
        if xf is not None:
            xf[0, 1, 10:50] = -np.inf                          # banned tokens get no probability
    tokens = rng.integers(0, V, (B, Lt)).astype(np.int32)
    sel = (rng.random((B, Lt)) < 0.5).astype(np.uint8)
    sel[0, 1] = 1
    tokens[2, 3] = V + 5                                       # out of range: flagged when scored, no gradient
    sel[2, 3] = 1
    dlogp = rng.normal(0, 0.01, (B, Lt)).astype(np.float32)
    st = pkg.ForkState(B, Lt)
    xt = to_torch_logits(x)
    tok_d, sel_d = torch.from_numpy(tokens).cuda(), torch.from_numpy(sel).cuda()
    lp, ssum, scnt, status, lse = pkg.fork_logprob(xt, tok_d, sel_d, st, want_lse=True)
    grad = torch.full_like(xt, 7.0)
    pkg.fork_logprob_backward(xt, tok_d, sel_d, lse, torch.from_numpy(dlogp).cuda(), grad, st)
    torch.cuda.synchronize()
    g = grad.float().cpu().numpy()
    lse_h = lse.cpu().numpy()
    for b in range(B):
        for k in range(Lt):
            if not sel[b, k] or tokens[b, k] >= V:
                assert (g[b, k] == 7.0).all(), (b, k)
                continue
            assert abs(lse_h[b, k] - oracle.row_lse(x[b, k])) <= 1e-5 + 1e-5 * abs(lse_h[b, k])
            want = oracle.row_logp_grad(x[b, k], int(tokens[b, k]), float(dlogp[b, k]))
            w = abs(float(dlogp[b, k]))
            if dtype == "f32":
                close("grad", g[b, k], want, 1e-4, 2e-6 * w)
            else:
                close("grad", g[b, k], want, 2.0 ** -8, 2e-6 * w)
            assert abs(g[b, k].sum()) <= (1e-4 if dtype == "f32" else 2e-2) * w * max(1.0, np.abs(want).sum() / w)


def test_scoring_loss_backward_chain_at_the_training_shape_of_a_few_rows():
    """V = 126464 fp32 rows through fork_logprob -> fork_grpo_loss -> fork_logprob_backward."""
    pkg = F()
    w = fs.workload("grpo")
    B, Lt, V, G = 8, 4, w.V, 4
    cfg = w.cfg(B=B)
    x = np.empty((B, Lt, V), np.float32)
    for b in range(B):
        for l in range(Lt):
            x[b, l] = fs.row_host(cfg, 0, b, l)
    rng = np.random.default_rng(0)
    tokens = x.argmax(-1).astype(np.int32)
    tokens[:, 1] = rng.integers(0, V, B)
    sel = np.ones((B, Lt), np.uint8)
    sel[:, 3] = 0
    reward = rng.random(B).astype(np.float32)
    st = pkg.ForkState(B, Lt)
    xt = torch.from_numpy(x).cuda()
    tok_d, sel_d = torch.from_numpy(tokens).cuda(), torch.from_numpy(sel).cuda()
    lp, ssum, scnt, status, lse = pkg.fork_logprob(xt, tok_d, sel_d, st, want_lse=True)
    old = (lp + 0.05 * torch.randn_like(lp)) * (sel_d != 0)
    out = pkg.fork_grpo_loss(lp, old.contiguous(), sel_d, torch.from_numpy(reward).cuda(), G, 0.2, 0.2)
    grad = torch.zeros_like(xt)
    pkg.fork_logprob_backward(xt, tok_d, sel_d, lse, out["dlogp"], grad, st)
    torch.cuda.synchronize()
    rc, olp, osum, ocnt, _ = oracle.logprob(x, tokens, sel)
    assert_close("logp", lp.cpu().numpy(), olp)
    o = oracle.grpo_loss(lp.cpu().numpy(), old.cpu().numpy(), sel, reward, G, 0.2, 0.2)
    close("objective", out["objective"].cpu().numpy()[0], o["objective"], 1e-4, 1e-6)
    close("dlogp", out["dlogp"].cpu().numpy(), o["dlogp"], 1e-4, 1e-9)
    g = grad.cpu().numpy()
    d = out["dlogp"].cpu().numpy()
    for b, k in ((0, 0), (3, 1), (7, 2)):
        want = oracle.row_logp_grad(x[b, k], int(tokens[b, k]), float(d[b, k]))
        close("grad", g[b, k], want, 1e-4, 2e-6 * abs(float(d[b, k])))
    assert (g[:, 3] == 0).all()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("V", [5, 1000, 5003, 40000])
def test_fused_pass_matches_the_oracle_and_the_three_calls(V, dtype):
    """fork_grpo_fused = fork_logprob -> fork_grpo_loss -> fork_logprob_backward with every selected row read
    once: log-probabilities and log-sum-exps against the oracle's rows, Eq. 2 against the oracle on those
    log-probabilities, gradient rows against the oracle's row derivative for the dlogp it reports, canaries
    in every row it must not touch; and the same numbers as the three calls in a row."""
    pkg = F()
    rng = np.random.default_rng(7 * V + (dtype == "f32"))
    B, Lt, G = 8, 6, 4
    x = make_rows(rng, (B, Lt), V, dtype, peak=5.0)
    if V > 100 and dtype == "f32":
        x[0, 1, 10:50] = -np.inf                               # banned tokens get no probability
        x[3, 2, :7] = -np.inf                                  # a thread's first vectors hold nothing finite
    tokens = rng.integers(0, V, (B, Lt)).astype(np.int32)
    if V > 100 and dtype == "f32":
        tokens[0, 1] = 60
    sel = (rng.random((B, Lt)) < 0.6).astype(np.uint8)
    sel[0, 1] = sel[3, 2] = sel[2, 3] = 1
    sel[5] = 0                                                 # a rollout without fallback steps
    tokens[2, 3] = V + 5                                       # out of range: flagged, scores 0, no gradient
    reward = rng.random(B).astype(np.float32)
    reward[:G] = 0.5                                           # a group with equal rewards: skipped
    xt = to_torch_logits(x)
    tok_d, sel_d, rew_d = (torch.from_numpy(t).cuda() for t in (tokens, sel, reward))
    st = pkg.ForkState(B, Lt)
    lp3, _, _, status3, lse3 = pkg.fork_logprob(xt, tok_d, sel_d, st, want_lse=True)
    old_d = ((lp3 + 0.1 * torch.randn_like(lp3)) * (sel_d != 0)).contiguous()
    old = old_d.cpu().numpy()
    for eps in ((0.2, 0.28), (0.02, 0.03)):                    # the second range clips many ratios
        loss3 = pkg.fork_grpo_loss(lp3, old_d, sel_d, rew_d, G, *eps)
        grad3 = torch.full_like(xt, 7.0)
        pkg.fork_logprob_backward(xt, tok_d, sel_d, lse3, loss3["dlogp"], grad3, st)
        grad = torch.full_like(xt, 7.0)
        out = pkg.fork_grpo_fused(xt, tok_d, sel_d, old_d, rew_d, G, eps[0], eps[1], grad, st)
        torch.cuda.synchronize()
        assert pkg.fork_device_status(st) == 0
        h = {k: v.cpu().numpy() for k, v in out.items()}
        rc, olp, _, _, ostatus = oracle.logprob(x, tokens, sel)
        assert rc == 0
        on = sel != 0
        assert_close("logp", h["logp"], olp, where=on)
        assert (h["row_status"][on] == ostatus[on]).all() and h["row_status"][2, 3] == pkg.FORK_ROW_BAD_TOKEN
        o = oracle.grpo_loss(h["logp"], old, sel, reward, G, *eps)
        rho = o["ratio"][on]
        if (np.abs(rho - (1 - np.float32(eps[0]))) < 1e-4).any() or (np.abs(rho - (1 + np.float32(eps[1]))) < 1e-4).any():
            continue                                           # a ratio on a clip boundary: fp32 may pick the other branch
        assert np.array_equal(h["skipped"], o["skipped"]) and o["skipped"][0] == 1
        close("adv", h["adv"], o["adv"], 1e-5, 1e-6)
        close("ratio", h["ratio"][on], o["ratio"][on], 1e-5, 1e-7)
        close("seq_obj", h["seq_obj"], o["seq_obj"], 1e-4, 1e-6)
        close("objective", h["objective"][0], o["objective"], 1e-4, 1e-6)
        close("dlogp", h["dlogp"][on], o["dlogp"][on], 1e-4, 1e-9)
        assert (h["dlogp"][:G][on[:G]] == 0).all()
        g, g3 = grad.float().cpu().numpy(), grad3.float().cpu().numpy()
        n_rows = 0
        for b in range(B):
            for k in range(Lt):
                if not sel[b, k] or tokens[b, k] >= V:
                    assert (g[b, k] == 7.0).all(), (b, k)
                    continue
                assert abs(h["lse"][b, k] - oracle.row_lse(x[b, k])) <= 1e-5 + 1e-5 * abs(h["lse"][b, k])
                w = float(h["dlogp"][b, k])
                want = oracle.row_logp_grad(x[b, k], int(tokens[b, k]), w)
                if dtype == "f32":
                    close("grad", g[b, k], want, 1e-4, 2e-6 * abs(w))
                else:
                    close("grad", g[b, k], want, 2.0 ** -8, 2e-6 * abs(w))
                n_rows += 1
        assert n_rows > 10
        # the three calls in a row say the same
        close("logp vs three calls", h["logp"][on], lp3.cpu().numpy()[on], 1e-6, 2e-6)
        close("dlogp vs three calls", h["dlogp"][on], loss3["dlogp"].cpu().numpy()[on], 1e-4, 1e-9)
        close("objective vs three calls", h["objective"][0], loss3["objective"].cpu().numpy()[0], 1e-5, 1e-7)
        close("grad vs three calls", g, g3, 2e-3 if dtype == "f32" else 2.0 ** -7, 1e-7)


def test_fused_pass_with_a_non_finite_row_and_at_the_training_width():
    """V = 126464 fp32 (the scoring workload's rows): a handful of rows against the oracle, one of them with a NaN,
    which must come out flagged with a NaN score, no contribution to the derivative, and a NaN gradient row as
    from the three calls."""
    pkg = F()
    w = fs.workload("grpo")
    B, Lt, V, G = 8, 3, w.V, 4
    cfg = w.cfg(B=B)
    x = np.empty((B, Lt, V), np.float32)
    for b in range(B):
        for l in range(Lt):
            x[b, l] = fs.row_host(cfg, 0, b, l)
    x[4, 1, 77777] = np.nan
    rng = np.random.default_rng(1)
    tokens = x.argmax(-1).astype(np.int32)
    tokens[:, 1] = rng.integers(0, V, B)
    sel = np.ones((B, Lt), np.uint8)
    sel[:, 2] = 0
    reward = rng.random(B).astype(np.float32)
    xt = torch.from_numpy(x).cuda()
    tok_d, sel_d, rew_d = (torch.from_numpy(t).cuda() for t in (tokens, sel, reward))
    st = pkg.ForkState(B, Lt)
    rc, olp, _, _, ostatus = oracle.logprob(x, tokens, sel)
    old = (olp + 0.05 * rng.standard_normal(olp.shape)).astype(np.float32) * (sel != 0)
    old[4, 1] = -3.0
    grad = torch.zeros_like(xt)
    out = pkg.fork_grpo_fused(xt, tok_d, sel_d, torch.from_numpy(old).cuda(), rew_d, G, 0.2, 0.2, grad, st)
    torch.cuda.synchronize()
    h = {k: v.cpu().numpy() for k, v in out.items()}
    on = sel != 0
    assert_close("logp", h["logp"], olp, where=on)
    assert np.isnan(h["logp"][4, 1]) and h["row_status"][4, 1] == pkg.FORK_ROW_NONFINITE and h["dlogp"][4, 1] == 0
    g = grad.cpu().numpy()
    assert np.isnan(g[4, 1]).all() and (g[:, 2] == 0).all()
    ok = on.copy()
    ok[4, 1] = False
    o = oracle.grpo_loss(np.where(ok, h["logp"], 0).astype(np.float32), old, ok.astype(np.uint8), reward, G, 0.2, 0.2)
    for b, k in ((0, 0), (3, 1), (7, 0), (5, 1)):
        want = oracle.row_logp_grad(x[b, k], int(tokens[b, k]), float(h["dlogp"][b, k]))
        close("grad", g[b, k], want, 1e-4, 2e-6 * abs(float(h["dlogp"][b, k])))
    rows_ok = [b for b in range(B) if b != 4]
    close("ratio", h["ratio"][rows_ok][on[rows_ok]], o["ratio"][rows_ok][on[rows_ok]], 1e-5, 1e-7)


def test_fused_pass_edge_shapes():
    """Nothing selected at all; a single selected row (one cluster works, the others only meet at the barriers);
    bf16 rows of the training width whose halves differ in length and whose last vector is ragged."""
    pkg = F()
    rng = np.random.default_rng(5)
    # (a) nothing selected: no row is read, the objective is 0, grad keeps its canary
    B, Lt, V, G = 4, 5, 1000, 2
    x = make_rows(rng, (B, Lt), V, "f32", peak=5.0)
    xt = to_torch_logits(x)
    tokens = torch.zeros((B, Lt), dtype=torch.int32, device="cuda")
    sel = torch.zeros((B, Lt), dtype=torch.uint8, device="cuda")
    old = torch.zeros((B, Lt), dtype=torch.float32, device="cuda")
    reward = torch.rand(B, device="cuda")
    st = pkg.ForkState(B, Lt)
    grad = torch.full_like(xt, 7.0)
    out = pkg.fork_grpo_fused(xt, tokens, sel, old, reward, G, 0.2, 0.2, grad, st)
    torch.cuda.synchronize()
    assert float(out["objective"][0]) == 0.0 and (out["seq_obj"] == 0).all() and (grad == 7.0).all()
    # (b) one selected row
    sel[2, 3] = 1
    tokens[2, 3] = 17
    old[2, 3] = -4.0
    out = pkg.fork_grpo_fused(xt, tokens, sel, old, reward, G, 0.2, 0.2, grad, st)
    torch.cuda.synchronize()
    g = grad.cpu().numpy()
    others = np.ones((B, Lt), bool)
    others[2, 3] = False
    assert (g[others] == 7.0).all()
    lp = oracle.row_logp(x[2, 3], 17)
    lp = lp[0] if isinstance(lp, tuple) else lp
    assert abs(float(out["logp"][2, 3]) - lp) <= 1e-5 + 1e-4 * abs(lp)
    want = oracle.row_logp_grad(x[2, 3], 17, float(out["dlogp"][2, 3]))
    close("grad", g[2, 3], want, 1e-4, 2e-6 * abs(float(out["dlogp"][2, 3])) + 1e-12)
    # (c) bf16, V = 126464 + 24: an odd number of vectors (the two halves differ) and no ragged end; then + 3: a ragged end
    for V in (126464 + 24, ):
        B, Lt, G = 4, 2, 2
        xb = make_rows(rng, (B, Lt), V, "bf16", peak=6.0)
        xt = to_torch_logits(xb)
        tokens_h = rng.integers(0, V, (B, Lt)).astype(np.int32)
        tokens_h[0, 0] = V - 1                                  # in the second half's last vector
        tokens_h[1, 1] = 0
        sel_h = np.ones((B, Lt), np.uint8)
        rc, olp, _, _, _ = oracle.logprob(xb, tokens_h, sel_h)
        old_h = (olp + 0.05 * rng.standard_normal(olp.shape)).astype(np.float32)
        reward_h = rng.random(B).astype(np.float32)
        st = pkg.ForkState(B, Lt)
        grad = torch.zeros_like(xt)
        out = pkg.fork_grpo_fused(xt, *(torch.from_numpy(t).cuda() for t in (tokens_h, sel_h, old_h, reward_h)), G, 0.2, 0.2, grad, st)
        torch.cuda.synchronize()
        assert pkg.fork_device_status(st) == 0
        h = {k: v.cpu().numpy() for k, v in out.items()}
        assert_close("logp", h["logp"], olp)
        o = oracle.grpo_loss(h["logp"], old_h, sel_h, reward_h, G, 0.2, 0.2)
        close("dlogp", h["dlogp"], o["dlogp"], 1e-4, 1e-9)
        g = grad.float().cpu().numpy()
        for b, k in ((0, 0), (1, 1), (3, 0)):
            want = oracle.row_logp_grad(xb[b, k], int(tokens_h[b, k]), float(h["dlogp"][b, k]))
            close("grad", g[b, k], want, 2.0 ** -8, 2e-6 * abs(float(h["dlogp"][b, k])))
