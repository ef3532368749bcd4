"""Comparison rules between the CUDA path and the oracle (shared by the GPU tests).

Routing indices, skip flags and the search argmin must agree exactly except on
counted near-ties: top-2 logit gap < 1e-3, |w1/w0 - beta| < 1e-4, subset losses
within 1e-3 relative.  Outputs: per-token relative L2 error <= 1e-2.
"""
import numpy as np
import torch

Y_REL_L2_TOL = 1e-2
LOGIT_GAP_TOL = 1e-3
RATIO_TOL = 1e-4
LOSS_REL_TOL = 1e-3


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.to(torch.float64).numpy()


def near_tie_tokens(logits: np.ndarray, kept_mask: int) -> np.ndarray:
    """Tokens whose kept logits ranked 1-3 have an adjacent gap below the tolerance."""
    T, E = logits.shape
    kept = np.array([(kept_mask >> e) & 1 for e in range(E)], bool)
    lm = np.where(kept[None, :], logits.astype(np.float64), -np.inf)
    srt = -np.sort(-lm, axis=1)
    tie = (srt[:, 0] - srt[:, 1]) < LOGIT_GAP_TOL
    if kept.sum() > 2:
        tie |= (srt[:, 1] - srt[:, 2]) < LOGIT_GAP_TOL
    return tie


def check_routing(gpu_idx, gpu_skipped, gpu_wn, gpu_ratio, ora, kept_mask, beta):
    """Returns the number of near-tie tokens that were excluded."""
    tie = near_tie_tokens(ora["logits"], kept_mask)
    ok = ~tie
    assert np.array_equal(gpu_idx[ok], ora["idx"][ok]), "top-2 indices differ outside near-ties"
    same_idx = (gpu_idx == ora["idx"]).all(1)
    close_beta = np.abs(ora["ratio"].astype(np.float64) - beta) < RATIO_TOL
    chk = ok & ~close_beta
    assert np.array_equal(gpu_skipped[chk], ora["skipped"][chk]), "skip flags differ outside near-ties"
    both = same_idx & (gpu_skipped == ora["skipped"])
    np.testing.assert_allclose(gpu_wn[both], ora["wn"][both], rtol=1e-5, atol=1e-7)
    np.testing.assert_allclose(gpu_ratio[same_idx], ora["ratio"][same_idx], rtol=1e-5, atol=1e-9)
    return int(tie.sum()), int((ok & close_beta).sum())


def check_outputs(gpu_y_bits, ora_y_bits, comparable: np.ndarray):
    """Per-token relative L2 error of y over the tokens whose routing agreed."""
    g = bf16_bits_to_f64(gpu_y_bits)
    o = bf16_bits_to_f64(ora_y_bits)
    err = np.linalg.norm(g - o, axis=1) / np.maximum(np.linalg.norm(o, axis=1), 1e-30)
    assert comparable.any()
    worst = float(err[comparable].max())
    assert worst <= Y_REL_L2_TOL, "per-token relative L2 error %.3e > %.1e" % (worst, Y_REL_L2_TOL)
    return worst


def check_search(gpu_losses, gpu_best, ora):
    gl = np.asarray(gpu_losses, np.float64)
    ol = ora["losses"]
    scale = max(float(ol.max()), 1e-30)
    assert np.all(np.abs(gl - ol) <= LOSS_REL_TOL * np.maximum(ol, 1e-6 * scale)), (gl, ol)
    if gpu_best != ora["best_subset"]:
        i = list(ora["subsets"]).index(gpu_best)
        j = int(np.argmin(ol))
        assert abs(ol[i] - ol[j]) <= LOSS_REL_TOL * ol[j], "argmin differs and is not a near-tie"
        return 1
    return 0


def edge_tokens(idx, skipped, E, tile=128, band=16):
    """Tokens that sit where a tiled grouped GEMM goes wrong first, from a routing record.

    The permutation is a stable counting sort, so the group of expert e holds, in ascending token
    order, the tokens with e in a slot that runs.  Per expert: the first, middle and last row of
    its group, both sides of the first tile boundary, the last row of the last full row tile, rows
    of the partly filled last tile, and both sides of the start of the last band of row tiles."""
    picks = []
    for e in range(E):
        toks = np.nonzero((idx[:, 0] == e) | ((idx[:, 1] == e) & (skipped == 0)))[0]
        n = len(toks)
        if n == 0:
            continue
        last_tile = (n - 1) // tile * tile
        ntiles = (n + tile - 1) // tile
        last_band = (ntiles - 1) // band * band * tile
        rows = {0, n // 2, n - 1, min(n - 1, tile - 1), min(n - 1, tile), last_tile, max(0, last_tile - 1),
                min(n - 1, last_tile + 1), (last_tile + n - 1) // 2, last_band, max(0, last_band - 1)}
        picks.extend(int(toks[r]) for r in rows)
    return np.unique(np.asarray(picks, np.int64))


def sample_tokens(idx, skipped, E, T, n_total, seed):
    """The edge tokens of the batch plus a seeded random remainder, n_total tokens at most
    (all tokens when the batch is smaller)."""
    if T <= n_total:
        return np.arange(T)
    edge = edge_tokens(idx, skipped, E)
    rest = np.setdiff1d(np.arange(T), edge)
    rng = np.random.default_rng(seed)
    extra = rng.choice(rest, size=max(0, n_total - len(edge)), replace=False)
    return np.sort(np.concatenate([edge, extra]))


class StackParity:
    """x_{l+1} = x_l + MoE_l(RMSNorm(x_l)) walked layer by layer on both sides.

    The GPU walks the layers through moe_rmsnorm + moe_forward_residual with a routing record (the
    kernel sequence moe_stack_forward runs), the oracle follows the same recurrence on its own
    states.  Per layer, a token whose GPU routing differs from the oracle's must be explained by a
    near-tie of the ORACLE's logits: an adjacent gap among its three largest kept logits below
    1e-3 + 2 d, or |w1/w0 - beta| below 1e-4 + ratio (exp(2 d) - 1), where d bounds how far any
    logit can have moved because the two sides' layer inputs differ (Cauchy-Schwarz:
    max_e ||Wg_e|| * ||xn_gpu - xn_oracle||).  Every token whose routing agreed in every layer must
    meet the output tolerance at the end; nothing is thrown away unexamined."""

    def __init__(self, T, E, dev, n_oracle=None):
        # the GPU walks all T tokens; the oracle follows the first n_oracle of them (tokens are
        # independent of each other in every step of the recurrence)
        self.T, self.E, self.dev = T, E, dev
        self.n = T if n_oracle is None else n_oracle
        self.agree = np.ones(self.n, bool)
        self.unexplained = []

    def layer(self, layer, host, kept, beta, cur_o, cur_g, eps=1e-5):
        from oracle import moe_oracle as O
        from paper_2402_14800_b200 import binding, synth
        xn_o = O.rmsnorm(cur_o, eps)
        ro = O.route(xn_o, host["Wg"], kept, beta)
        nxt_o = O.moe_forward(xn_o, host["Wg"], host["W1"], host["W3"], host["W2"], kept, beta,
                              residual=cur_o)["y"]
        xn_g = binding.rmsnorm(cur_g, eps)
        stats = binding.RoutingStats(self.T, self.E, self.dev)
        nxt_g = layer.forward(xn_g, beta, residual=cur_g, stats=stats)
        torch.cuda.synchronize()
        gi, gs = stats.idx.cpu().numpy()[:self.n], stats.skipped.cpu().numpy()[:self.n]
        dx = np.linalg.norm(bf16_bits_to_f64(synth.bf16_bits(xn_g)[:self.n]) - bf16_bits_to_f64(xn_o), axis=1)
        d = dx * np.linalg.norm(bf16_bits_to_f64(host["Wg"]), axis=1).max()
        keptv = np.array([(kept >> e) & 1 for e in range(self.E)], bool)
        srt = -np.sort(-np.where(keptv[None, :], ro["logits"].astype(np.float64), -np.inf), axis=1)
        gap = srt[:, 0] - srt[:, 1]
        if keptv.sum() > 2:
            gap = np.minimum(gap, srt[:, 1] - srt[:, 2])
        ratio = ro["ratio"].astype(np.float64)
        idx_same = (gi == ro["idx"]).all(1)
        skip_same = gs == ro["skipped"]
        idx_explained = gap < LOGIT_GAP_TOL + 2 * d
        skip_explained = np.abs(ratio - beta) < RATIO_TOL + ratio * np.expm1(2 * d)
        bad = (~idx_same & ~idx_explained) | (idx_same & ~skip_same & ~skip_explained)
        self.unexplained.extend(int(t) for t in np.nonzero(bad)[0])
        self.agree &= idx_same & skip_same
        return nxt_o, nxt_g

    def finish(self, y_g_bits, y_o_bits, max_rerouted):
        assert not self.unexplained, "routing differs from the oracle without a near-tie: %s" % self.unexplained
        assert (~self.agree).sum() <= max_rerouted, "%d tokens were re-routed" % (~self.agree).sum()
        return check_outputs(y_g_bits[:self.n], y_o_bits, self.agree)
