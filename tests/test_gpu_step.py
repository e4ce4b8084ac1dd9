"""CUDA fork_step / fork_logprob against the fp64 oracle on small and edge-case inputs, called through
the C ABI.  Integers bit-exact, floats within |g-o| <= 1e-5 + 1e-4 |o|."""
import math

import numpy as np
import pytest
import torch

import fork_synth as fs
import oracle
from helpers import assert_close, assert_equal, compare_step_state, live_mask, to_torch_logits

pytestmark = pytest.mark.gpu


def F():
    import paper_2609_39859_b200 as pkg
    return pkg


def make_rows(rng, shape, V, dtype, sigma=3.0, peak=9.0, peak_frac=0.5):
    x = (rng.standard_normal(shape + (V,)) * sigma).astype(np.float32)
    flat = x.reshape(-1, V)
    for i in range(flat.shape[0]):
        if rng.random() < peak_frac:
            flat[i, rng.integers(0, V)] += rng.uniform(0, peak) + math.log(V)
    return x if dtype == "f32" else fs.f32_to_bf16_bits(x)


def run_both(x_np, mask, lo, hi, lam, pos0=0, step=5, tokens=None, logits_t=None, keep_margin=True):
    """One step on both sides from the same host inputs; returns (gpu host dict, oracle state)."""
    pkg = F()
    B, Ll, V = x_np.shape
    Lt = mask.shape[1]
    tokens = np.full((B, Lt), -3, np.int32) if tokens is None else tokens
    o = oracle.StepState(B, Lt, tokens=tokens, mask=mask)
    assert oracle.step(o, x_np, lo, hi, lam, step_id=step, pos0=pos0) == 0
    if keep_margin:     # inputs must not put a confidence within 1e-4 of the threshold
        live = live_mask(mask, lo, hi)
        assert (np.abs(o.conf[live] - np.float64(np.float32(lam))) >= 1e-4).all(), "test input too close to lambda"
    g = pkg.ForkState(B, Lt, tokens=tokens, mask=mask)
    lg = to_torch_logits(x_np) if logits_t is None else logits_t
    pkg.fork_step(g, lg, torch.from_numpy(np.asarray(lo, np.int32)).cuda(),
                  torch.from_numpy(np.asarray(hi, np.int32)).cuda(), lam, step=step, pos0=pos0)
    torch.cuda.synchronize()
    return g.host(), o


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("V", [1, 2, 7, 8, 9, 255, 1023, 1024, 1025, 2047, 2048, 2049, 4104, 6151, 40000])
def test_step_small_vocabularies(V, dtype):
    """Aligned and unaligned V (the latter takes the scalar path), several chunks and a ragged tail."""
    rng = np.random.default_rng(V * 3 + (dtype == "f32"))
    B, Lt = 5, 40
    mask = (rng.random((B, Lt)) < 0.7).astype(np.uint8)
    lo = rng.integers(0, 20, size=B).astype(np.int32)
    hi = (lo + rng.integers(0, 20, size=B)).astype(np.int32)
    mask[1, lo[1]:hi[1]] = 0                                        # a sequence with no live row
    x = make_rows(rng, (B, Lt), V, dtype)
    live = live_mask(mask, lo, hi)
    if dtype == "f32":
        x[~live] = np.nan                                           # canaries: rows that must not be read
    else:
        x[~live] = 0x7FC0
    g, o = run_both(x, mask, lo, hi, 0.9 if V > 2 else 0.45)
    compare_step_state(g, o)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_step_padded_rows_take_the_vector_path_with_a_ragged_tail(dtype):
    """V is odd but the row pitch is a multiple of 16 bytes: vector loads plus a scalar tail."""
    rng = np.random.default_rng(11)
    B, Lt, V, pitch = 3, 16, 5003, 5008
    mask = np.ones((B, Lt), np.uint8)
    lo, hi = np.zeros(B, np.int32), np.full(B, Lt, np.int32)
    x = make_rows(rng, (B, Lt), V, dtype)
    buf = np.full((B, Lt, pitch), 0x7FC0 if dtype == "bf16" else np.nan, x.dtype)
    buf[..., :V] = x
    lt = to_torch_logits(buf)[..., :V]
    assert lt.stride(1) == pitch
    g, o = run_both(x, mask, lo, hi, 0.9, logits_t=lt)
    compare_step_state(g, o)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_ties_resolve_to_the_lowest_index_across_every_boundary(dtype):
    """Equal tops placed at vector, thread-stride, chunk and CTA-split boundaries, first/last element."""
    V = 126464
    vec = 8 if dtype == "bf16" else 4
    spots = [[0, V - 1], [V - 1, V - 2], [vec - 1, vec], [2047, 2048], [2048 * 31 - 1, 2048 * 31],
             [256 * vec - 1, 256 * vec, 512 * vec], [70000, 5], [V - 1, 0, 63232], [4095, 4096, 4097, 100000],
             [V // 2, V // 2 + 1], [1, 126463], [12345, 12344]]
    n = len(spots)
    x = np.zeros((1, n, V), np.float32)
    for i, s in enumerate(spots):
        x[0, i, s] = 16.0
    xs = x if dtype == "f32" else fs.f32_to_bf16_bits(x)
    mask = np.ones((1, n), np.uint8)
    g, o = run_both(xs, mask, [0], [n], 0.9)
    assert g["cand"][0].tolist() == [min(s) for s in spots]
    compare_step_state(g, o)
    # few rows: every row is split over many CTAs; also a single row
    for rows in (1, 2, 3):
        g, o = run_both(xs[:, :rows], mask[:, :rows], [0], [rows], 0.9)
        compare_step_state(g, o)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_closed_form_rows_on_the_gpu(dtype):
    """One peak of height h over zeros (closed forms in tests/golden/closed_forms.txt)."""
    cases = [(126464, 1, 14.0, 0.90484830865468718, 1.4321116429117138),
             (126464, 1, 16.0, 0.98596815884916369, 0.23864067657074723),
             (152064, 1, 14.0, 0.88774882085252779, 1.69058294346715),
             (126464, 2, 14.0, 0.47502400162525053, 1.4437179009796957),
             (126464, 4, 20.0, 0.24998371021855374, 1.3876627048843249)]
    pkg = F()
    for V, k, h, conf, H in cases:
        x = np.zeros((1, 1, V), np.float32)
        x[0, 0, np.arange(k) * 1000 + 17] = h
        xs = x if dtype == "f32" else fs.f32_to_bf16_bits(x)
        g = pkg.ForkState(1, 1)
        pkg.fork_step(g, to_torch_logits(xs), torch.zeros(1, dtype=torch.int32).cuda(),
                      torch.ones(1, dtype=torch.int32).cuda(), 0.5)
        r = g.host()
        assert r["cand"][0, 0] == 17
        assert_close("conf", r["conf"][0, 0], conf)
        assert_close("entropy", r["entropy"][0, 0], H)
        assert_close("logp", r["logp"][0, 0], math.log(conf))


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_nonfinite_rows(dtype):
    """-inf has probability zero (fast path); NaN / +inf / all -inf rows are flagged and never clear
    a threshold, but can still be the leftmost fallback."""
    rng = np.random.default_rng(2)
    V, n = 9000, 10
    x = (rng.standard_normal((1, n, V)) * 2).astype(np.float32)
    x[0, :, 77] += 14.0
    x[0, 0, 100:5000] = -np.inf                      # banned range: still an ordinary row
    x[0, 1, :] = -np.inf; x[0, 1, 4000] = 1.0        # a single finite entry: conf 1
    x[0, 2, 5] = np.nan
    x[0, 3, 8999] = np.inf
    x[0, 4, :] = -np.inf
    x[0, 5, :] = np.nan
    x[0, 6, :3] = -np.inf                            # leading -inf before the first finite value
    x[0, 7, 3] = np.inf; x[0, 7, 2] = np.inf
    x[0, 8, 0] = np.nan; x[0, 8, 1:] = -np.inf
    xs = x if dtype == "f32" else fs.f32_to_bf16_bits(x)
    mask = np.ones((1, n), np.uint8)
    g, o = run_both(xs, mask, [0], [n], 0.9, keep_margin=False)
    compare_step_state(g, o)
    assert g["row_status"][0].tolist() == [0, 0, 1, 1, 1, 1, 0, 1, 1, 0]
    # bad row as the leftmost fallback
    g, o = run_both(xs[:, 2:6], mask[:, :4], [0], [4], 0.9, keep_margin=False)
    compare_step_state(g, o)
    assert g["is_fallback"][0] == 1 and g["fallback_pos"][0] == 0 and g["mask"][0].tolist() == [0, 1, 1, 1]


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_banned_token_ranges_of_minus_inf_at_full_vocabulary(dtype):
    """Many rows with ranges of -inf logits (banned tokens) at V=126464+3 on a padded pitch: the
    streaming path first runs unclamped, the threads that met -inf redo their vectors clamped and
    stay clamped for later rows; several stages, a partly filled last stage and a scalar tail."""
    rng = np.random.default_rng(21)
    B, Lt, V, pitch = 3, 24, 126467, 126472
    x = (rng.standard_normal((B, Lt, V)) * 3).astype(np.float32)
    x[np.arange(B)[:, None], np.arange(Lt)[None, :], rng.integers(0, V, size=(B, Lt))] += 25.0
    for b in range(B):
        for l in range(Lt):
            kind = (b * Lt + l) % 4
            if kind == 0:
                x[b, l, :2000] = -np.inf                       # reserved ids at the start
            elif kind == 1:
                a = int(rng.integers(0, V - 30000))
                x[b, l, a:a + 30000] = -np.inf                 # a long range in the middle
            elif kind == 2:
                x[b, l, V - 300:] = -np.inf                    # padding ids at the end, incl. the scalar tail
    xs = x if dtype == "f32" else fs.f32_to_bf16_bits(x)
    buf = np.full((B, Lt, pitch), np.nan if dtype == "f32" else 0x7FC0, xs.dtype)
    buf[..., :V] = xs
    lt = to_torch_logits(buf)[..., :V]
    mask = np.ones((B, Lt), np.uint8)
    g, o = run_both(xs, mask, np.zeros(B, np.int32), np.full(B, Lt, np.int32), 0.9, logits_t=lt)
    compare_step_state(g, o)
    assert (g["row_status"] == 0).all()


def test_threshold_extremes_and_strictness():
    rng = np.random.default_rng(4)
    x = make_rows(rng, (3, 12), 300, "f32")
    mask = np.ones((3, 12), np.uint8)
    lo, hi = np.array([0, 4, 12], np.int32), np.array([12, 8, 12], np.int32)
    for lam in (-1.0, 1.0, 2.0, 0.0):
        g, o = run_both(x, mask, lo, hi, lam, keep_margin=False)
        compare_step_state(g, o)
    # confidence exactly at the threshold is not committed: two equal logits, conf = 0.5 exactly
    z = np.zeros((1, 2, 2), np.float32)
    g, o = run_both(z, np.ones((1, 2), np.uint8), [0], [2], 0.5, keep_margin=False)
    compare_step_state(g, o)
    assert g["is_fallback"][0] == 1 and g["mask"][0].tolist() == [0, 1]


def test_window_buffer_and_clamping():
    pkg = F()
    rng = np.random.default_rng(6)
    B, Lt, V, pos0, Ll = 3, 64, 1000, 32, 16
    x = make_rows(rng, (B, Ll), V, "bf16")
    mask = (rng.random((B, Lt)) < 0.8).astype(np.uint8)
    lo, hi = np.full(B, 32, np.int32), np.full(B, 48, np.int32)
    g, o = run_both(x, mask, lo, hi, 0.9, pos0=pos0)
    compare_step_state(g, o)
    # a block that reaches outside the window is clipped and reported
    lo2, hi2 = np.array([30, 32, 40], np.int32), np.array([48, 50, 44], np.int32)
    o = oracle.StepState(B, Lt, mask=mask)
    oracle.step(o, x, lo2, hi2, 0.9, pos0=pos0)
    st = pkg.ForkState(B, Lt, mask=mask)
    pkg.fork_step(st, to_torch_logits(x), torch.from_numpy(lo2).cuda(), torch.from_numpy(hi2).cuda(), 0.9, pos0=pos0)
    assert pkg.fork_device_status(st) & pkg.FORK_DEV_WINDOW_CLAMPED
    compare_step_state(st.host(), o)
    pkg.fork_step(st, to_torch_logits(x), torch.from_numpy(lo).cuda(), torch.from_numpy(hi).cuda(), 0.9, pos0=pos0)
    assert pkg.fork_device_status(st) == 0


def test_large_block_more_rows_than_threads_per_cta():
    rng = np.random.default_rng(8)
    B, Lt, V = 2, 700, 520
    x = make_rows(rng, (B, Lt), V, "bf16", peak_frac=0.3)
    mask = (rng.random((B, Lt)) < 0.9).astype(np.uint8)
    g, o = run_both(x, mask, [0, 10], [700, 650], 0.9)
    compare_step_state(g, o)
    g, o = run_both(x, mask, [0, 10], [700, 650], 1.5)
    compare_step_state(g, o)


def test_same_inputs_twice_give_identical_bytes():
    pkg = F()
    rng = np.random.default_rng(9)
    B, Lt, V = 4, 8, 126464
    x = to_torch_logits(make_rows(rng, (B, Lt), V, "bf16"))
    lo, hi = torch.zeros(B, dtype=torch.int32).cuda(), torch.full((B,), Lt, dtype=torch.int32).cuda()
    outs = []
    for _ in range(3):
        st = pkg.ForkState(B, Lt)
        pkg.fork_step(st, x, lo, hi, 0.9)
        outs.append(st.host())
    for name in outs[0]:
        for other in outs[1:]:
            assert outs[0][name].tobytes() == other[name].tobytes(), name


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_logprob_small(dtype):
    pkg = F()
    rng = np.random.default_rng(12)
    for V in (5, 1000, 2049, 30000):
        B, Lt = 4, 24
        x = make_rows(rng, (B, Lt), V, dtype)
        tokens = rng.integers(0, V, size=(B, Lt)).astype(np.int32)
        select = (rng.random((B, Lt)) < 0.4).astype(np.uint8)
        select[2] = 0
        tokens[0, 3] = V                               # out of range where selected
        select[0, 3] = 1
        if dtype == "f32":
            x[1, 5, 0] = -np.inf
            tokens[1, 5] = 0
            select[1, 5] = 1
            x[3, 7, V // 2] = np.nan
            select[3, 7] = 1
            x[~select.astype(bool)] = np.nan           # unselected rows are never read
        rc, lp, ssum, scnt, status = oracle.logprob(x, tokens, select)
        st = pkg.ForkState(B, Lt)
        glp, gsum, gcnt, gst = pkg.fork_logprob(to_torch_logits(x), torch.from_numpy(tokens).cuda(),
                                                torch.from_numpy(select).cuda(), st)
        torch.cuda.synchronize()
        assert_equal("seq_cnt", gcnt.cpu().numpy(), scnt)
        assert_equal("status", gst.cpu().numpy(), status)
        assert_close("logp", glp.cpu().numpy(), lp)
        assert_close("seq_sum", gsum.cpu().numpy(), ssum)


def test_step_host_entry_point_matches_device_entry_point():
    import ctypes as C
    pkg = F()
    rng = np.random.default_rng(13)
    B, Lt, V = 3, 16, 3000
    x = make_rows(rng, (B, Lt), V, "bf16")
    mask = (rng.random((B, Lt)) < 0.8).astype(np.uint8)
    lo, hi = np.zeros(B, np.int32), np.full(B, Lt, np.int32)
    g, o = run_both(x, mask, lo, hi, 0.9)
    h = oracle.StepState(B, Lt, tokens=np.full((B, Lt), -3, np.int32), mask=mask)   # only used as host buffers
    conf32, ent32, lp32, clp32 = (np.full((B, Lt), np.nan, np.float32) for _ in range(4))
    a = pkg.fork_step_args()
    a.logits = x.ctypes.data
    a.stride_b, a.stride_l, a.pos0 = Lt * V, V, 0
    a.B, a.Lt, a.Ll, a.V, a.dtype = B, Lt, Lt, V, pkg.FORK_BF16
    a.tokens, a.mask, a.blk_lo, a.blk_hi = h.tokens.ctypes.data, h.mask.ctypes.data, lo.ctypes.data, hi.ctypes.data
    a.threshold, a.step = 0.9, 5
    a.conf, a.cand, a.entropy, a.logp = conf32.ctypes.data, h.cand.ctypes.data, ent32.ctypes.data, lp32.ctypes.data
    a.row_status = h.row_status.ctypes.data
    a.commit_step, a.commit_fallback, a.commit_logp = h.commit_step.ctypes.data, h.commit_fallback.ctypes.data, clp32.ctypes.data
    a.n_unmasked, a.is_fallback, a.fallback_pos = h.n_unmasked.ctypes.data, h.is_fallback.ctypes.data, h.fallback_pos.ctypes.data
    a.nfe, a.n_fallback = h.nfe.ctypes.data, h.n_fallback.ctypes.data
    L = pkg.lib()
    nbytes = L.fork_staging_bytes(C.byref(a))
    staging = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    sp = staging.data_ptr() + (-staging.data_ptr()) % 256
    st = pkg.ForkState(B, Lt)
    rc = L.fork_step_host(C.byref(a), C.c_void_p(sp), nbytes, C.c_void_p(st.ws_ptr), st.ws_bytes, None)
    assert rc == 0
    got = dict(tokens=h.tokens, mask=h.mask, cand=h.cand, commit_step=h.commit_step, commit_fallback=h.commit_fallback,
               row_status=h.row_status, n_unmasked=h.n_unmasked, is_fallback=h.is_fallback, fallback_pos=h.fallback_pos,
               nfe=h.nfe, n_fallback=h.n_fallback, conf=conf32, entropy=ent32, logp=lp32, commit_logp=clp32)
    for name in got:
        assert got[name].tobytes() == g[name].tobytes(), name


def test_read_probe_runs_and_rejects_bad_arguments():
    import ctypes as C
    pkg = F()
    L = pkg.lib()
    buf = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    sink = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert L.fork_read_probe(C.c_void_p(buf.data_ptr()), buf.numel(), C.c_void_p(sink.data_ptr()), None) == 0
    assert L.fork_read_probe(C.c_void_p(buf.data_ptr()), 1000, C.c_void_p(sink.data_ptr()), None) == 0      # ragged size
    torch.cuda.synchronize()
    assert int(sink.cpu()[0]) == 0
    assert L.fork_read_probe(None, 16, C.c_void_p(sink.data_ptr()), None) == pkg.FORK_ERR_INVALID_ARG
    assert L.fork_read_probe(C.c_void_p(buf.data_ptr() + 4), 16, C.c_void_p(sink.data_ptr()), None) == pkg.FORK_ERR_INVALID_ARG
