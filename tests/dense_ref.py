"""Textbook dense restatement of the MoE layer in numpy fp64, used to pin the
oracle: every expert is applied to every token with library matmuls, then the
routing mask is applied.  Independent of ``oracle/`` and of the CUDA path."""
import numpy as np
import torch


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.to(torch.float64).numpy()


def round_bf16(a: np.ndarray) -> np.ndarray:
    """fp64 -> fp32 -> bf16 (torch's round-to-nearest-even) -> fp64."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float64)).to(torch.float32)
    return t.to(torch.bfloat16).to(torch.float64).numpy()


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float64)).to(torch.float32).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def logits(x_bits, Wg_bits) -> np.ndarray:
    return bits_to_f64(x_bits) @ bits_to_f64(Wg_bits).T


def all_experts(x_bits, W1_bits, W3_bits, W2_bits) -> np.ndarray:
    """Y[T,E,h]: W2 (silu(W1 x) * W3 x) with the activation rounded to bf16."""
    x = bits_to_f64(x_bits)
    W1, W3, W2 = bits_to_f64(W1_bits), bits_to_f64(W3_bits), bits_to_f64(W2_bits)
    g = np.einsum("th,efh->tef", x, W1)
    u = np.einsum("th,efh->tef", x, W3)
    a = round_bf16(g / (1.0 + np.exp(-g)) * u)
    return np.einsum("tef,ehf->teh", a, W2)


def top2(l: np.ndarray, kept_mask: int):
    """Indices of the two largest kept logits per row (ties -> lower index),
    and the gap between rank 2 and 3 / rank 1 and 2 for near-tie filtering."""
    T, E = l.shape
    kept = np.array([(kept_mask >> e) & 1 for e in range(E)], bool)
    lm = np.where(kept[None, :], l, -np.inf)
    order = np.argsort(-lm, axis=1, kind="stable")
    e0, e1 = order[:, 0], order[:, 1]
    srt = np.take_along_axis(lm, order, axis=1)
    gap01 = srt[:, 0] - srt[:, 1]
    gap12 = srt[:, 1] - srt[:, 2] if kept.sum() > 2 else np.full(T, np.inf)
    return e0, e1, gap01, gap12
