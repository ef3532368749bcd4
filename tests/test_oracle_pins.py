"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these re-type the oracle's own formula: they use a dense numpy fp64
restatement built from library matmuls, closed forms, exact invariants and
integer counts.  All run on the tiny configuration (h=128, f=448, E=8, T=256).
"""
import itertools
from math import comb

import numpy as np
import pytest
import torch

from oracle import moe_oracle as O
from paper_2402_14800_b200 import synth
from tests import dense_ref as D

H, F, E, T = 128, 448, 8, 256
FULL = (1 << E) - 1


@pytest.fixture(scope="module")
def cfg0():
    W = synth.make_layer_weights(H, F, E, seed=0)
    x = synth.make_tokens(T, H, seed=0)
    b = synth.bf16_bits
    return dict(x=b(x), Wg=b(W.W_gate), W1=b(W.W1), W3=b(W.W3), W2=b(W.W2))


@pytest.fixture(scope="module")
def dense(cfg0):
    return dict(l=D.logits(cfg0["x"], cfg0["Wg"]),
                Y=D.all_experts(cfg0["x"], cfg0["W1"], cfg0["W3"], cfg0["W2"]))


def fwd(c, kept=FULL, beta=0.0, **kw):
    return O.moe_forward(c["x"], c["Wg"], c["W1"], c["W3"], c["W2"], kept, beta, **kw)


# ---------------------------------------------------------------- bf16 helpers

def test_bf16_rounding_matches_library():
    rng = np.random.default_rng(0)
    v = np.concatenate([
        rng.standard_normal(2000).astype(np.float32) * 10.0 ** rng.integers(-6, 6, 2000),
        # exact halfway cases between two bf16 values: ties go to even
        np.array([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -1.0 - 2 ** -8, 2 ** -130, 0.0, -0.0,
                  3.3895314e38, np.inf, -np.inf], np.float32),
    ]).astype(np.float32)
    want = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([O.f32_to_bf16(float(a)) for a in v], np.uint16)
    assert (got == want).all()
    back = np.array([O.bf16_to_f32(int(b)) for b in want], np.float32)
    ref = torch.from_numpy(want.view(np.int16)).view(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(back, ref)


# ---------------------------------------------------------------------- router

@pytest.mark.parametrize("kept", [FULL, 0b10110111, 0b01011010, 0b00100100])
def test_router_closed_form(cfg0, dense, kept):
    """Softmax -> top-2 -> renormalise collapses to w~_e0 = 1/(1+exp(l_e1-l_e0));
    the ratio w_e1/w_e0 = exp(l_e1-l_e0); Sec. 3.1 / Eq. 1 with any kept subset."""
    r = O.route(cfg0["x"], cfg0["Wg"], kept, 0.0)
    l = dense["l"]
    e0, e1, gap01, gap12 = D.top2(l, kept)
    clear = (gap01 > 1e-3) & (gap12 > 1e-3)
    assert clear.sum() > 0.9 * T
    assert (r["idx"][clear, 0] == e0[clear]).all() and (r["idx"][clear, 1] == e1[clear]).all()
    d = l[np.arange(T), e1] - l[np.arange(T), e0]
    np.testing.assert_allclose(r["wn"][clear, 0], (1 / (1 + np.exp(d)))[clear], rtol=2e-5)
    np.testing.assert_allclose(r["wn"][clear, 1], (1 / (1 + np.exp(-d)))[clear], rtol=2e-5)
    np.testing.assert_allclose(r["ratio"][clear], np.exp(d)[clear], rtol=2e-5)
    np.testing.assert_allclose(r["wn"].sum(1), 1.0, rtol=1e-6)
    # softmax over the kept experts only (Sec. 3.2): w_e0 = exp(l_e0) / sum_kept exp(l)
    keptv = np.array([(kept >> e) & 1 for e in range(E)], bool)
    sm = np.exp(l - l.max(1, keepdims=True)) * keptv
    sm /= sm.sum(1, keepdims=True)
    np.testing.assert_allclose(r["w"][clear, 0], sm[np.arange(T), e0][clear], rtol=2e-5)
    np.testing.assert_allclose(r["w"][clear, 1], sm[np.arange(T), e1][clear], rtol=2e-5)
    # logits are reported for all E experts
    np.testing.assert_allclose(r["logits"], l, rtol=0, atol=1e-5)


def test_router_rejects_fewer_than_two_kept(cfg0):
    with pytest.raises(ValueError):
        O.route(cfg0["x"], cfg0["Wg"], 0b100, 0.0)


def test_topk_tie_goes_to_lower_index():
    # two identical router rows -> exactly equal logits
    x = synth.bf16_bits(synth.make_tokens(16, 64, seed=3))
    wg = synth.make_layer_weights(64, 64, 4, seed=3).W_gate
    wg[3] = wg[1]
    wg[0] = -wg[1]
    r = O.route(x, synth.bf16_bits(wg), 0b1111, 0.0)
    l = r["logits"]
    assert np.array_equal(l[:, 1], l[:, 3])
    top_is_tied = l[:, 1] >= np.maximum(l[:, 0], l[:, 2])
    assert top_is_tied.any()
    assert (r["idx"][top_is_tied, 0] == 1).all() and (r["idx"][top_is_tied, 1] == 3).all()
    np.testing.assert_array_equal(r["ratio"][top_is_tied], 1.0)
    # beta = 1 with an exact tie: strict '<' does not skip
    r1 = O.route(x, synth.bf16_bits(wg), 0b1111, 1.0)
    assert (r1["skipped"][top_is_tied] == 0).all()
    assert (r1["skipped"][~top_is_tied] == 1).all()


# --------------------------------------------------------------------- forward

def test_beta0_all_kept_is_textbook_top2(cfg0, dense):
    """beta = 0, all experts kept: Eq. 2 equals dense all-experts-then-mask."""
    out = fwd(cfg0)
    assert out["skipped"].sum() == 0
    l, Y = dense["l"], dense["Y"]
    e0, e1, gap01, gap12 = D.top2(l, FULL)
    ok = gap12 > 1e-3
    assert (out["idx"][ok, 0] == e0[ok]).all() and (out["idx"][ok, 1] == e1[ok]).all()
    sm = np.exp(l - l.max(1, keepdims=True))
    sm /= sm.sum(1, keepdims=True)
    mask = np.zeros_like(sm)
    mask[np.arange(T), e0] = 1
    mask[np.arange(T), e1] = 1
    wt = sm * mask
    wt /= wt.sum(1, keepdims=True)
    z = np.einsum("te,teh->th", wt, Y)
    scale = np.abs(z).max()
    assert np.abs(out["z"][ok] - z[ok]).max() < 2e-6 * scale
    # R2: y is z rounded to bf16; allow a different rounding only where z sits on a boundary
    ulp_off = np.abs(out["y"][ok].astype(np.int32) - D.to_bf16_bits(z[ok]).astype(np.int32))
    assert ulp_off.max() <= 1 and (ulp_off != 0).mean() < 1e-3


def test_dense_mask_catches_swapped_projections(cfg0, dense):
    """The dense pin is sensitive to the operand roles: silu(W3 x) * W1 x differs."""
    Yswap = D.all_experts(cfg0["x"][:8], cfg0["W3"], cfg0["W1"], cfg0["W2"])
    assert np.abs(Yswap - dense["Y"][:8]).max() > 1e-2 * np.abs(dense["Y"][:8]).max()


def test_beta_above_one_is_top1(cfg0, dense):
    """beta > 1 always skips e_1 and the output is E_e0(x) with weight exactly 1."""
    out = fwd(cfg0, beta=1.5)
    assert out["skipped"].all()
    assert (out["wn"][:, 0] == 1.0).all() and (out["wn"][:, 1] == 0.0).all()
    e0 = np.argmax(dense["l"], 1)
    gap = np.sort(dense["l"], 1)
    ok = gap[:, -1] - gap[:, -2] > 1e-3
    z = dense["Y"][np.arange(T), e0]
    assert np.abs(out["z"][ok] - z[ok]).max() < 1e-9 * np.abs(z).max()


def test_skip_output_difference_closed_form(cfg0, dense):
    """App. A.2 with i=1, k=2 is an equality: z^ - z = w~_e1 (f_e0 - f_e1)."""
    a = fwd(cfg0, beta=0.0)
    b = fwd(cfg0, beta=2.0)
    Y = dense["Y"]
    t = np.arange(T)
    f0, f1 = Y[t, a["idx"][:, 0]], Y[t, a["idx"][:, 1]]
    want = a["wn"][:, 1:2].astype(np.float64) * (f0 - f1)
    got = b["z"] - a["z"]
    # the two fp32 weights sum to 1 only up to one rounding (2^-24), hence the bound
    assert np.abs(got - want).max() < 3e-7 * np.abs(Y).max()


def test_median_beta_skips_exactly_half(cfg0):
    """Sec. 3.3 / appendix: beta = median of w_e1/w_e0 skips half of the batch."""
    ratio = fwd(cfg0)["ratio"]
    assert len(np.unique(ratio)) == T  # no ties in this batch
    beta = O.beta_median(ratio)
    srt = np.sort(ratio)
    assert srt[T // 2 - 1] < beta < srt[T // 2]
    out = fwd(cfg0, beta=beta)
    assert int(out["skipped"].sum()) == T // 2
    np.testing.assert_array_equal(out["skipped"], (ratio < np.float32(beta)).astype(np.uint8))
    # odd count: the middle element itself, and strict '<' keeps that token
    beta_odd = O.beta_median(ratio[:-1])
    assert beta_odd == np.sort(ratio[:-1])[(T - 1) // 2]
    out_odd = O.route(cfg0["x"][:-1], cfg0["Wg"], FULL, beta_odd)
    assert int(out_odd["skipped"].sum()) == (T - 1) // 2
    # the synthetic router gives a beta of the magnitude the paper prints (0.33 .. 0.62)
    vals = [float(v) for line in open("tests/golden/paper_beta_values.txt")
            if not line.startswith("#") for v in line.split(":")[1].split(",")]
    assert len(vals) == 64
    assert 0.5 * min(vals) < beta < 1.5 * max(vals)


def test_beta_median_matches_numpy():
    rng = np.random.default_rng(1)
    for n in (1, 2, 7, 100, 101):
        r = rng.random(n).astype(np.float32)
        assert O.beta_median(r) == np.float32(np.median(r.astype(np.float64)))


# --------------------------------------------------------------------- pruning

@pytest.mark.parametrize("kept", [0b11011101, 0b01100110])
def test_pruned_layer_keeps_tokens_whose_top2_survive(cfg0, kept):
    """Sec. 3.2: removing experts and their router rows leaves a token untouched
    (bit for bit) when both of its experts are kept, and re-routes it otherwise."""
    full = fwd(cfg0)
    pr = fwd(cfg0, kept=kept)
    inside = np.array([((kept >> a) & 1) and ((kept >> b) & 1) for a, b in full["idx"]], bool)
    assert 0 < inside.sum() < T
    assert np.array_equal(pr["y"][inside], full["y"][inside])
    assert np.array_equal(pr["z"][inside], full["z"][inside])
    assert np.array_equal(pr["idx"][inside], full["idx"][inside])
    assert np.array_equal(pr["wn"][inside], full["wn"][inside])
    assert all(((kept >> e) & 1) for e in pr["idx"].ravel())
    assert (np.abs(pr["z"][~inside] - full["z"][~inside]).max(1) > 0).all()


def test_pruned_router_equals_compacted_layer(cfg0):
    """A pruned layer is the same as a smaller layer built from the kept experts only."""
    kept = 0b10110110
    ids = [e for e in range(E) if (kept >> e) & 1]
    pr = fwd(cfg0, kept=kept)
    small = O.moe_forward(cfg0["x"], cfg0["Wg"][ids], cfg0["W1"][ids], cfg0["W3"][ids],
                          cfg0["W2"][ids], (1 << len(ids)) - 1, 0.0)
    assert np.array_equal(np.array(ids)[small["idx"]], pr["idx"])
    assert np.array_equal(small["y"], pr["y"])


def test_relabelling_experts_permutes_routing_only(cfg0):
    perm = np.array([3, 7, 0, 5, 1, 6, 2, 4])
    a = fwd(cfg0, beta=0.4)
    b = O.moe_forward(cfg0["x"], cfg0["Wg"][perm], cfg0["W1"][perm], cfg0["W3"][perm],
                      cfg0["W2"][perm], FULL, 0.4)
    assert np.array_equal(perm[b["idx"]], a["idx"])
    assert np.array_equal(a["y"], b["y"]) and np.array_equal(a["skipped"], b["skipped"])


def test_residual_is_added_before_the_output_rounding(cfg0):
    res = synth.bf16_bits(synth.make_tokens(T, H, seed=9))
    a = fwd(cfg0, beta=0.3)
    b = fwd(cfg0, beta=0.3, residual=res)
    want = D.to_bf16_bits(D.bits_to_f64(res) + a["z"])
    assert np.array_equal(b["y"], want)


# ---------------------------------------------------------------------- search

def test_subset_enumeration_is_lexicographic():
    for r in (8, 6, 4, 2):
        m = O.enumerate_subsets(E, r)
        want = [sum(1 << i for i in c) for c in itertools.combinations(range(E), r)]
        assert m.tolist() == want and len(m) == comb(E, r)
    assert len(O.enumerate_subsets(8, 6)) == 28 and len(O.enumerate_subsets(8, 4)) == 70


def search(c, r, fast=True, sl=slice(None)):
    fn = O.prune_search_allexperts if fast else O.prune_search_bruteforce
    return fn(c["x"][sl], c["Wg"], c["W1"], c["W3"], c["W2"], r)


def test_full_subset_has_zero_loss(cfg0):
    for fast in (True, False):
        s = search(cfg0, E, fast, slice(0, 32))
        assert s["losses"].tolist() == [0.0] and s["best_subset"] == FULL


@pytest.mark.parametrize("r", [6, 4])
def test_search_forms_agree_and_count_disturbed_tokens(cfg0, r):
    """Eq. 3 evaluated per subset equals all-experts-once + gather; the number of
    tokens with a non-zero error is the number whose top-2 is not inside C."""
    fast = search(cfg0, r, True)
    brute = search(cfg0, r, False)
    np.testing.assert_allclose(fast["losses"], brute["losses"], rtol=1e-12)
    assert np.array_equal(fast["n_changed"], brute["n_changed"])
    assert fast["best_subset"] == brute["best_subset"]
    idx = O.route(cfg0["x"], cfg0["Wg"], FULL, 0.0)["idx"]
    pair = (1 << idx[:, 0]) | (1 << idx[:, 1])
    for C, n in zip(fast["subsets"], fast["n_changed"]):
        assert n == int(((pair & ~C) != 0).sum())
    assert (fast["losses"] >= 0).all()
    assert fast["best_subset"] == fast["subsets"][int(np.argmin(fast["losses"]))]
    np.testing.assert_allclose(fast["loss_sq"], fast["losses"] ** 2, rtol=1e-12)


def test_search_loss_matches_dense_restatement(cfg0, dense):
    """Reconstruction loss of a few subsets from the dense numpy pieces: route in
    fp64 among kept logits, gather bf16-rounded expert outputs, Frobenius norm."""
    s = search(cfg0, 6, True)
    l, Y = dense["l"], D.round_bf16(dense["Y"])
    t = np.arange(T)

    def layer(kept):
        e0, e1, _, _ = D.top2(l, kept)
        d = l[t, e1] - l[t, e0]
        return (1 / (1 + np.exp(d)))[:, None] * Y[t, e0] + (1 / (1 + np.exp(-d)))[:, None] * Y[t, e1]

    Fref = layer(FULL)
    for ci in (0, 5, 13, 27):
        want = np.linalg.norm(layer(int(s["subsets"][ci])) - Fref)
        assert abs(s["losses"][ci] - want) < 1e-5 * want


def test_loss_squares_add_over_token_chunks(cfg0):
    whole = search(cfg0, 6, True)
    a = search(cfg0, 6, True, slice(0, 100))
    b = search(cfg0, 6, True, slice(100, T))
    np.testing.assert_allclose(a["loss_sq"] + b["loss_sq"], whole["loss_sq"], rtol=1e-12)
    assert np.array_equal(a["n_changed"] + b["n_changed"], whole["n_changed"])


def test_loss_is_zero_iff_no_token_is_disturbed(cfg0):
    # keep only tokens routed inside {0,...,5}: the subset {0..5} must then cost nothing
    idx = O.route(cfg0["x"], cfg0["Wg"], FULL, 0.0)["idx"]
    sel = np.where((idx < 6).all(1))[0]
    assert len(sel) > 8
    c = dict(cfg0, x=cfg0["x"][sel])
    s = search(c, 6, True)
    assert s["losses"][0] == 0.0 and s["subsets"][0] == 0b111111 and s["best_subset"] == 0b111111
    assert (s["losses"][1:] > 0).all()


# ----------------------------------------------------------------------- stack

def test_rmsnorm_matches_numpy(cfg0):
    x = D.bits_to_f64(cfg0["x"])
    want = D.to_bf16_bits(x / np.sqrt((x * x).mean(1, keepdims=True) + 1e-5))
    assert np.array_equal(O.rmsnorm(cfg0["x"], 1e-5), want)


# ------------------------------------------------------------------- baselines

def test_coselection_counts_and_frequency_subset(cfg0, dense):
    """App. A.1 co-selection map and the activation-frequency baseline of Sec. 4.1."""
    counts = O.coselection(cfg0["x"], cfg0["Wg"])
    assert counts.sum() == T and np.trace(counts) == 0
    e0, e1, gap01, gap12 = D.top2(dense["l"], FULL)
    want = np.zeros((E, E), np.int64)
    np.add.at(want, (e0, e1), 1)
    n_tie = int(((gap01 <= 1e-3) | (gap12 <= 1e-3)).sum())
    assert np.abs(counts - want).sum() <= 2 * n_tie
    freq = counts.sum(0) + counts.sum(1)
    assert freq.sum() == 2 * T
    for r in (6, 4, 2):
        mask = O.frequency_subset(counts, r)
        order = sorted(range(E), key=lambda e: (-freq[e], e))[:r]
        assert mask == sum(1 << e for e in order)
    # a tie in frequency keeps the lower index
    c = np.zeros((4, 4), np.int64)
    c[0, 1] = c[2, 3] = 5
    assert O.frequency_subset(c, 2) == 0b0011


# ----------------------------------------------------------- progressive search

def _unpruned_output(c, Y_rounded):
    r = O.route(c["x"], c["Wg"], FULL, 0.0)
    t = np.arange(len(c["x"]))
    return (r["wn"][:, 0:1].astype(np.float64) * Y_rounded[t, r["idx"][:, 0]]
            + r["wn"][:, 1:2].astype(np.float64) * Y_rounded[t, r["idx"][:, 1]])


def test_progressive_search_reduces_to_layerwise_on_identical_inputs(cfg0):
    """With x_p = x and F_ref = F(x) the progressive loss is the layer-wise loss of Eq. 3."""
    Y = O.all_experts(cfg0["x"], cfg0["W1"], cfg0["W3"], cfg0["W2"], round_bf16=True)
    F = _unpruned_output(cfg0, Y)
    lw = search(cfg0, 6, True)
    pg = O.prune_search_progressive(cfg0["x"], cfg0["Wg"], cfg0["W1"], cfg0["W3"], cfg0["W2"],
                                    F.astype(np.float32), 6)
    # F_ref is stored in fp32: one rounding of relative size 2^-24 on every element
    tol = 2e-7 * np.linalg.norm(F)
    assert np.abs(pg["losses"] - lw["losses"]).max() <= tol + 1e-6 * lw["losses"].max()
    assert pg["best_subset"] == lw["best_subset"]


def test_progressive_search_matches_dense_restatement(cfg0, dense):
    """Different inputs on the two sides: pruned layer on x_p (dense numpy), target from x."""
    Yx = D.round_bf16(dense["Y"])
    F_ref = _unpruned_output(cfg0, Yx).astype(np.float32)
    xp = synth.bf16_bits(synth.make_tokens(T, H, seed=5))
    lp = D.logits(xp, cfg0["Wg"])
    Yp = D.round_bf16(D.all_experts(xp, cfg0["W1"], cfg0["W3"], cfg0["W2"]))
    pg = O.prune_search_progressive(xp, cfg0["Wg"], cfg0["W1"], cfg0["W3"], cfg0["W2"], F_ref, 6)
    t = np.arange(T)
    for ci in (0, 9, 27):
        e0, e1, _, _ = D.top2(lp, int(pg["subsets"][ci]))
        d = lp[t, e1] - lp[t, e0]
        Fp = (1 / (1 + np.exp(d)))[:, None] * Yp[t, e0] + (1 / (1 + np.exp(-d)))[:, None] * Yp[t, e1]
        want = np.linalg.norm(Fp - F_ref.astype(np.float64))
        assert abs(pg["losses"][ci] - want) < 1e-5 * want
    # additive over token chunks, and a zero target gives the norm of the pruned output itself
    a = O.prune_search_progressive(xp[:90], cfg0["Wg"], cfg0["W1"], cfg0["W3"], cfg0["W2"], F_ref[:90], 6)
    b = O.prune_search_progressive(xp[90:], cfg0["Wg"], cfg0["W1"], cfg0["W3"], cfg0["W2"], F_ref[90:], 6)
    np.testing.assert_allclose(a["loss_sq"] + b["loss_sq"], pg["loss_sq"], rtol=1e-12)
    z = O.prune_search_progressive(xp, cfg0["Wg"], cfg0["W1"], cfg0["W3"], cfg0["W2"],
                                   np.zeros((T, H), np.float32), 8)
    e0, e1, _, _ = D.top2(lp, FULL)
    d = lp[t, e1] - lp[t, e0]
    Ffull = (1 / (1 + np.exp(d)))[:, None] * Yp[t, e0] + (1 / (1 + np.exp(-d)))[:, None] * Yp[t, e1]
    assert abs(z["losses"][0] - np.linalg.norm(Ffull)) < 1e-5 * np.linalg.norm(Ffull)


# ------------------------------------------------------- generalised top-k skipping

@pytest.fixture(scope="module")
def cfg16():
    h, f, E_, T_ = 64, 128, 16, 200
    W = synth.make_layer_weights(h, f, E_, seed=7)
    x = synth.make_tokens(T_, h, seed=8)
    b = synth.bf16_bits
    c = dict(x=b(x), Wg=b(W.W_gate), W1=b(W.W1), W3=b(W.W3), W2=b(W.W2))
    return c, D.logits(c["x"], c["Wg"]), D.all_experts(c["x"], c["W1"], c["W3"], c["W2"])


def fwdk(c, kept, k, beta):
    return O.moe_forward_topk(c["x"], c["Wg"], c["W1"], c["W3"], c["W2"], kept, k, beta)


@pytest.mark.parametrize("k", [1, 2, 4])
def test_topk_without_skipping_is_textbook_topk(cfg16, k):
    """beta = 0: App. A.2's z = sum_{m<=k} w_m f_m / sum_{m<=k} w_m, as dense then mask."""
    c, l, Y = cfg16
    kept = 0xFFFF
    out = fwdk(c, kept, k, 0.0)
    Tn = l.shape[0]
    order = np.argsort(-l, axis=1, kind="stable")
    srt = np.take_along_axis(l, order, 1)
    ok = (np.diff(-srt[:, :k + 1], axis=1) > 1e-3).all(1)
    assert ok.sum() > 0.8 * Tn
    assert np.array_equal(out["idx"][ok], order[ok, :k])
    assert (out["n_active"] == k).all()
    sm = np.exp(l - l.max(1, keepdims=True))
    mask = np.zeros_like(sm)
    np.put_along_axis(mask, order[:, :k], 1.0, axis=1)
    wt = sm * mask
    wt /= wt.sum(1, keepdims=True)
    z = np.einsum("te,teh->th", wt, Y)
    assert np.abs(out["z"][ok] - z[ok]).max() < 3e-6 * np.abs(z).max()
    np.testing.assert_allclose(out["wn"].sum(1), 1.0, rtol=1e-6)


def test_topk_skipping_rule_bound_and_monotonicity(cfg16):
    """i* is the smallest i whose skipped mass is <= beta of the selected mass; the output
    error obeys the appendix' bound L <= (skipped mass / selected mass) * max ||f_m - f_n||."""
    c, l, Y = cfg16
    kept, k = 0xFFFF, 4
    base = fwdk(c, kept, k, 0.0)
    t = np.arange(l.shape[0])
    prev = np.full(l.shape[0], k)
    for beta in (0.05, 0.2, 0.5, 0.9, 1.0):
        out = fwdk(c, kept, k, beta)
        na = out["n_active"]
        assert (na <= prev).all() and (na >= 1).all()
        prev = na
        assert np.array_equal(out["idx"], base["idx"])
        # the rule, re-evaluated in fp64 from the dense logits (away from the threshold)
        sel = np.take_along_axis(l, base["idx"].astype(np.int64), 1)
        p = np.exp(sel - sel[:, :1])
        tot = p.sum(1)
        tails = np.stack([p[:, i:].sum(1) for i in range(1, k + 1)], 1)  # i = 1..k
        want = 1 + (tails > beta * tot[:, None]).sum(1)
        clear = (np.abs(tails / tot[:, None] - beta) > 1e-5).all(1)
        assert np.array_equal(na[clear], want[clear])
        np.testing.assert_allclose(out["tail_frac"], tails[t, na - 1] / tot, rtol=1e-5, atol=1e-7)
        assert (out["tail_frac"] <= beta + 1e-6).all()
        # weights renormalised over the survivors, zero for the skipped ones
        assert (out["wn"][t[:, None], np.arange(k)[None, :]] * (np.arange(k)[None, :] >= na[:, None]) == 0).all()
        np.testing.assert_allclose(out["wn"].sum(1), 1.0, rtol=1e-6)
        # the paper's bound on the reconstruction error
        f_sel = Y[t[:, None], base["idx"]]                         # [T, k, h]
        dmax = np.max(np.linalg.norm(f_sel[:, :, None, :] - f_sel[:, None, :, :], axis=3), axis=(1, 2))
        err = np.linalg.norm(out["z"] - base["z"], axis=1)
        assert (err <= out["tail_frac"] * dmax * (1 + 1e-6) + 1e-12).all()
    assert (fwdk(c, kept, k, 1.0)["n_active"] == 1).all()          # beta >= 1 degenerates to top-1


def test_top2_generalised_rule_is_the_pairwise_rule_with_rescaled_beta(cfg0):
    """For k = 2, w_2 <= b (w_1 + w_2) is w_2 <= b/(1-b) w_1: the two forms of the paper agree."""
    bg = 0.3
    g = O.moe_forward_topk(cfg0["x"], cfg0["Wg"], cfg0["W1"], cfg0["W3"], cfg0["W2"], FULL, 2, bg)
    pw = fwd(cfg0, beta=bg / (1 - bg))
    away = np.abs(pw["ratio"] - bg / (1 - bg)) > 1e-5
    assert np.array_equal((g["n_active"] == 1)[away], pw["skipped"].astype(bool)[away])
    assert np.array_equal(g["idx"], pw["idx"])
    same = (g["n_active"] == 1) == pw["skipped"].astype(bool)
    np.testing.assert_allclose(g["z"][same], pw["z"][same], rtol=1e-6, atol=1e-9)


def test_topk_pruned_experts_are_never_selected(cfg16):
    c, l, Y = cfg16
    kept = 0b1010110011110101
    out = fwdk(c, kept, 4, 0.3)
    assert all((kept >> int(e)) & 1 for e in out["idx"].ravel())
    with pytest.raises(ValueError):
        fwdk(c, 0b111, 4, 0.0)


# ----------------------------------------------------- expert-output distance (App. A.2)

@pytest.mark.parametrize("kept", [FULL, 0b10110110])
def test_top2_distance_and_exact_skip_error(cfg0, dense, kept):
    """D_t = ||f_e0 - f_e1|| against the dense numpy outputs; for k = 2 the appendix' bound is an
    equality: ||z^ - z|| = w~_e1 D_t."""
    d = O.top2_distance(cfg0["x"], cfg0["Wg"], cfg0["W1"], cfg0["W3"], cfg0["W2"], kept)
    a = fwd(cfg0, kept=kept, beta=0.0)
    t = np.arange(T)
    want = np.linalg.norm(dense["Y"][t, a["idx"][:, 0]] - dense["Y"][t, a["idx"][:, 1]], axis=1)
    np.testing.assert_allclose(d, want, rtol=1e-9)
    b = fwd(cfg0, kept=kept, beta=2.0)
    err = np.linalg.norm(b["z"] - a["z"], axis=1)
    # the two fp32 weights sum to 1 only up to one rounding, hence the absolute term
    np.testing.assert_allclose(err, a["wn"][:, 1] * d, rtol=2e-6,
                               atol=3e-7 * np.linalg.norm(dense["Y"], axis=2).max())
