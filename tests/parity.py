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
