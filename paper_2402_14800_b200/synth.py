"""Seeded synthetic inputs for a Mixtral-style MoE layer.

This module only draws random numbers and rounds them to bf16.  It holds none
of the method's arithmetic (no routing, no expert math), so both the CUDA path
and the CPU oracle can be fed from it without sharing code between them.

Recipe (stands in for Mixtral 8x7B weights and C4/MATH hidden states, which
are not available offline):

* ``x[T, h]``      N(0, 1); ``max(1, round(0.01*h))`` outlier channels, chosen
                    by a seeded permutation, are multiplied by 20.
* ``W1, W3[E,f,h]`` N(0, std 0.02)   (gate and up projections, h contiguous)
* ``W2[E, h, f]``   N(0, std 0.02)   (down projection, f contiguous)
* ``W_gate[E, h]``  N(0, variance 1/h); row e is scaled by exp(N(0, std 0.5))
                    so expert usage is unequal.

Everything is generated in fp32 by ``torch.Generator(device).manual_seed(seed)``
and rounded to bf16 (round-to-nearest-even).  The bits depend on the device
type of the generator, so a parity test draws once and hands the same bits to
both sides.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

OUTLIER_FRACTION = 0.01
OUTLIER_SCALE = 20.0
WEIGHT_STD = 0.02
ROUTER_ROW_LOG_STD = 0.5


@dataclass
class LayerWeights:
    """bf16 tensors of one MoE layer (all on the same device)."""

    W_gate: torch.Tensor  # [E, h]
    W1: torch.Tensor      # [E, f, h]
    W3: torch.Tensor      # [E, f, h]
    W2: torch.Tensor      # [E, h, f]

    @property
    def E(self) -> int:
        return self.W_gate.shape[0]

    @property
    def h(self) -> int:
        return self.W_gate.shape[1]

    @property
    def f(self) -> int:
        return self.W1.shape[1]

    def cpu(self) -> "LayerWeights":
        return LayerWeights(self.W_gate.cpu(), self.W1.cpu(), self.W3.cpu(), self.W2.cpu())


def _generator(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _normal_bf16(shape, std: float, g: torch.Generator, device, chunk_rows: int = 0) -> torch.Tensor:
    """N(0, std) in fp32, rounded to bf16; drawn slab by slab along dim 0 so the
    fp32 staging buffer stays small for multi-GB tensors."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    n0 = shape[0]
    for i in range(n0):
        slab = torch.randn(shape[1:], generator=g, dtype=torch.float32, device=device)
        out[i].copy_(slab.mul_(std))
    return out


def make_layer_weights(h: int, f: int, E: int, seed: int, device="cpu") -> LayerWeights:
    """Draw W_gate, W1, W3, W2 in this fixed order from one seeded generator."""
    g = _generator(seed, device)
    wg = torch.randn((E, h), generator=g, dtype=torch.float32, device=device) * (float(h) ** -0.5)
    row_scale = torch.exp(torch.randn((E,), generator=g, dtype=torch.float32, device=device) * ROUTER_ROW_LOG_STD)
    wg = (wg * row_scale[:, None]).to(torch.bfloat16)
    W1 = _normal_bf16((E, f, h), WEIGHT_STD, g, device)
    W3 = _normal_bf16((E, f, h), WEIGHT_STD, g, device)
    W2 = _normal_bf16((E, h, f), WEIGHT_STD, g, device)
    return LayerWeights(wg, W1, W3, W2)


def make_tokens(T: int, h: int, seed: int, device="cpu") -> torch.Tensor:
    """Hidden states x[T, h] in bf16 with a few large-magnitude channels."""
    g = _generator(seed, device)
    perm = torch.randperm(h, generator=g, device=device)
    n_out = max(1, int(round(OUTLIER_FRACTION * h)))
    scale = torch.ones((h,), dtype=torch.float32, device=device)
    scale[perm[:n_out]] = OUTLIER_SCALE
    x = torch.randn((T, h), generator=g, dtype=torch.float32, device=device)
    return (x * scale[None, :]).to(torch.bfloat16)


def bf16_bits(t: torch.Tensor):
    """Contiguous host ``numpy.uint16`` view of a bf16 tensor's bit patterns."""
    return t.detach().cpu().contiguous().view(torch.uint16).numpy()


# The paper's workload shapes (hidden size, FFN width, experts).
TINY = dict(h=128, f=448, E=8)
MIXTRAL = dict(h=4096, f=14336, E=8)
