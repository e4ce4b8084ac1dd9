"""Host side of the synthetic-logit generator: determinism, dtype conversion, distribution,
planting rules and the statistics the workload recipes promise (checked with the oracle)."""
import math

import numpy as np
import pytest
import scipy.stats
import torch

import fork_synth as fs
import oracle


def test_bf16_conversion_matches_round_to_nearest_even():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000).astype(np.float32) * 7,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38, -65504.0], np.float32)])
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (fs.f32_to_bf16_bits(x) == ref).all()
    assert (fs.bf16_bits_to_f32(ref) == torch.from_numpy(x).to(torch.bfloat16).float().numpy()).all()


def test_rows_are_pure_functions_of_their_coordinates():
    w = fs.workload("tiny")
    c = w.cfg()
    a = fs.row_host(c, 3, 0, 5)
    assert (a == fs.row_host(c, 3, 0, 5)).all()
    assert not (a == fs.row_host(c, 4, 0, 5)).all()
    assert not (a == fs.row_host(c, 3, 0, 6)).all()
    assert not (a == fs.row_host(c, 3, 0, 5, nonce=1)).all()
    c2 = w.cfg()
    c2.seed += 1
    assert not (a == fs.row_host(c2, 3, 0, 5)).all()


def test_background_is_standard_normal_times_sigma():
    w = fs.workload("grpo")
    c = w.cfg()
    c.peak_prob = 0.0
    z = np.concatenate([fs.row_host(c, 0, 0, l) for l in range(6)]) / np.float32(3.0)
    assert abs(z.mean()) < 5e-3 and abs(z.std() - 1) < 5e-3
    assert abs(scipy.stats.kurtosis(z)) < 0.03 and abs(scipy.stats.skew(z)) < 0.02
    assert scipy.stats.kstest(z, "norm").pvalue > 1e-3
    assert 4.3 < np.abs(z).max() < 6.6              # tails are refined beyond the 2^-17 quantile


def test_fill_touches_only_live_rows():
    w = fs.workload("tiny")
    c = w.cfg(B=2)
    Lt, V = c.Lt, c.V
    mask = np.ones((2, Lt), np.uint8)
    mask[0, 3] = 0
    lo, hi = np.array([0, 8], np.int32), np.array([8, 16], np.int32)
    logits = np.empty((2, Lt, V), np.float32)
    fs.canary_host(logits)
    n = fs.fill_host(c, 7, mask, lo, hi, logits, nonce=2)
    assert n == 15
    for b in range(2):
        for k in range(Lt):
            live = lo[b] <= k < hi[b] and mask[b, k]
            if live:
                assert (logits[b, k] == fs.row_host(c, 7, b, k, nonce=2)).all()
            else:
                assert np.isnan(logits[b, k]).all()
    # a block-window buffer (pos0 > 0)
    win = np.empty((2, 8, V), np.float32)
    fs.canary_host(win)
    n = fs.fill_host(c, 7, mask, np.array([8, 8], np.int32), np.array([16, 16], np.int32), win, pos0=8, nonce=2)
    assert n == 16 and (win[1] == logits[1, 8:16]).all()


def test_planting_rules():
    w = fs.workload("passk")
    c = w.cfg()
    kinds = {"fork": 0, "peak": 0, "none": 0}
    for b in range(4):
        for l in range(256):
            p = fs.plan_host(c, b, l)
            if p["is_fork"]:
                kinds["fork"] += 1
                assert 2 <= p["n_planted"] <= 4 and len(set(p["tok"])) == p["n_planted"]
                top = p["val"][0]
                assert all(0 <= top - v < w.fork_gap for v in p["val"])
            elif p["n_planted"] == 1:
                kinds["peak"] += 1
                assert p["val"][0] == pytest.approx(w.peak_base() + 10.0, abs=1e-5)
            else:
                kinds["none"] += 1
    assert 0.06 < kinds["fork"] / 1024 < 0.14 and kinds["none"] == 0
    # planted values land in the row; a fork row's tops are exact ties or one bf16 step apart
    for l in range(256):
        p = fs.plan_host(c, 0, l)
        if p["is_fork"]:
            row = fs.bf16_bits_to_f32(fs.row_host(c, 0, 0, l))
            got = row[p["tok"]]
            assert (got == fs.bf16_bits_to_f32(fs.f32_to_bf16_bits(np.array(p["val"], np.float32)))).all()
            assert got.max() - got.min() <= 0.125
            assert oracle.row_stats(fs.row_host(c, 0, 0, l))["conf"] < 0.56
            break


@pytest.mark.parametrize("name,lo_frac,hi_frac", [("b8", 0.22, 0.40), ("tiny", 0.60, 0.92), ("sweep", 0.17, 0.36)])
def test_calibrated_fallback_prone_fraction(name, lo_frac, hi_frac):
    """Share of positions whose confidence stays at or below the threshold (fallback-prone)."""
    w = fs.workload(name)
    c = w.cfg()
    n, below = 0, 0
    for b in range(min(c.B, 2)):
        for l in range(0, c.Lt, max(1, c.Lt // 48)):
            s = oracle.row_stats(fs.row_host(c, 0, b, l))
            n += 1
            below += s["conf"] <= w.threshold
            p = fs.plan_host(c, b, l)
            if p["n_planted"] == 1 and p["val"][0] - w.peak_base() > 3.0:
                assert s["cand"] == p["tok"][0]
    assert lo_frac <= below / n <= hi_frac, below / n


def test_literal_variant_almost_never_clears_the_threshold():
    w = fs.workload("b8").literal()
    c = w.cfg()
    confs = [oracle.row_stats(fs.row_host(c, 0, 0, l))["conf"] for l in range(24)]
    assert max(confs) < 0.9


def test_scoring_inputs():
    w = fs.workload("grpo")
    c = w.cfg(B=4)
    tokens, select = fs.scoring_inputs(w, c)
    assert tokens.shape == (4, 256) and 0.12 < select.mean() < 0.28
    on_peak = np.mean([tokens[b, l] == fs.plan_host(c, b, l)["tok"][0] for b in range(4) for l in range(256)])
    assert 0.7 < on_peak < 0.9 and tokens.min() >= 0 and tokens.max() < c.V
