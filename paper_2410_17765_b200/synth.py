"""Seeded synthetic inputs for the CP-head log-likelihood.

This module only draws random numbers and casts them; it contains none of the
method's arithmetic, so both the CUDA path and the CPU oracle may be fed from
it.  Everything is drawn on the CPU with one ``torch.Generator`` so that the
same bit patterns reach both sides.

Shapes and distributions follow the workloads the method is used on: hidden
states of a transformer trunk (unit normal after the final norm), small-normal
weights, and either uniform or Zipf-distributed target tokens (natural-language
token frequencies are roughly Zipfian).
"""
from __future__ import annotations

from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class Shape:
    """Problem sizes: N positions, d embedding size, V vocabulary, n predicted
    tokens, r CP rank (number of experts)."""

    N: int
    d: int
    V: int
    n: int
    r: int

    @property
    def K(self) -> int:
        return self.n * self.r


# Named workloads (sizes only).
CONFIGS = {
    "tiny": Shape(N=64, d=256, V=1024, n=3, r=4),
    "train_fwd": Shape(N=4096, d=2048, V=32000, n=2, r=8),
    "train_fwd_bwd": Shape(N=8192, d=4096, V=32000, n=4, r=8),
    "decode_1": Shape(N=1, d=4096, V=128256, n=4, r=8),
    "decode_8": Shape(N=8, d=4096, V=128256, n=4, r=8),
    "decode_64": Shape(N=64, d=4096, V=128256, n=4, r=8),
    "bigvocab_fwd_bwd": Shape(N=8192, d=4096, V=128256, n=4, r=16),
    # train_fwd_bwd at 1/16 of the positions: same kernels and tile shapes, small enough to profile
    "train_fwd_bwd_small": Shape(N=512, d=4096, V=32000, n=4, r=8),
    # bigvocab at 1/4 of the positions (forward only): same schedule regime, profilable
    # full-head variant (Eq. 6 as printed): W_full is n*r*V*d = 1 GB here
    "full_head_train": Shape(N=4096, d=2048, V=32000, n=2, r=4),
    "bigvocab_fwd_small": Shape(N=2048, d=4096, V=128256, n=4, r=16),
}


@dataclass
class Inputs:
    """bf16 operands and int32 targets, all on the CPU.

    h       [N, d]        hidden state per position
    W_head  [n*r, d, d]   head projections, index k = s*r + alpha, [out][in]
    E       [V, d]        shared unembedding
    W_g     [r, d]        gate weights
    x       [N, n]        target tokens x_{t+1..t+n}
    """

    shape: Shape
    h: torch.Tensor
    W_head: torch.Tensor
    E: torch.Tensor
    W_g: torch.Tensor
    x: torch.Tensor


def _randn_bf16(gen: torch.Generator, shape, std: float) -> torch.Tensor:
    """Normal(0, std) drawn in fp32 in slabs along dim 0, cast once to bf16."""
    out = torch.empty(shape, dtype=torch.bfloat16)
    flat = out.view(shape[0], -1)
    per_row = flat.shape[1]
    rows_per_slab = max(1, (1 << 24) // max(1, per_row))
    for r0 in range(0, shape[0], rows_per_slab):
        r1 = min(shape[0], r0 + rows_per_slab)
        slab = torch.randn((r1 - r0, per_row), generator=gen, dtype=torch.float32)
        if std != 1.0:
            slab.mul_(std)
        flat[r0:r1] = slab.to(torch.bfloat16)
    return out


def zipf_targets(gen: torch.Generator, N: int, n: int, V: int, exponent: float = 1.1) -> torch.Tensor:
    """Targets with p(v) proportional to (v+1)^(-exponent); token id = rank."""
    p = torch.arange(1, V + 1, dtype=torch.float64).pow(-exponent)
    cdf = torch.cumsum(p / p.sum(), 0)
    u = torch.rand((N, n), generator=gen, dtype=torch.float64)
    idx = torch.searchsorted(cdf, u).clamp_(max=V - 1)
    return idx.to(torch.int32)


def make_inputs(
    shape: Shape,
    seed: int = 0,
    *,
    weight_std: float = 0.02,
    h_std: float = 1.0,
    targets: str = "uniform",
    weight_scale: float = 1.0,
) -> Inputs:
    """Draw (h, W_head, E, W_g, x) in that order from one seeded generator.

    ``targets`` is "uniform" or "zipf" (exponent 1.1).  ``weight_scale``
    multiplies every weight after the draw (a stress knob: 8 gives logits with
    a standard deviation above 10 at d=4096).
    """
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    s = shape
    std = weight_std * weight_scale
    h = _randn_bf16(gen, (s.N, s.d), h_std)
    W_head = _randn_bf16(gen, (s.K, s.d, s.d), std)
    E = _randn_bf16(gen, (s.V, s.d), std)
    W_g = _randn_bf16(gen, (s.r, s.d), std)
    if targets == "uniform":
        x = torch.randint(0, s.V, (s.N, s.n), generator=gen, dtype=torch.int64).to(torch.int32)
    elif targets == "zipf":
        x = zipf_targets(gen, s.N, s.n, s.V)
    else:
        raise ValueError(f"unknown target distribution {targets!r}")
    return Inputs(shape=s, h=h, W_head=W_head, E=E, W_g=W_g, x=x)


def make_full_head(shape: Shape, seed: int = 0, *, weight_std: float = 0.02, weight_scale: float = 1.0) -> torch.Tensor:
    """W_full [n*r, V, d] bf16 for the full-head variant: one N(0, std) unembedding per (token, expert)."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed + 7919)
    return _randn_bf16(gen, (shape.K, shape.V, shape.d), weight_std * weight_scale)


def subsample_positions(inp: Inputs, idx: torch.Tensor) -> Inputs:
    """The same problem restricted to the positions ``idx`` (weights shared)."""
    idx = idx.to(torch.int64)
    s = inp.shape
    sub = Shape(N=int(idx.numel()), d=s.d, V=s.V, n=s.n, r=s.r)
    return Inputs(shape=sub, h=inp.h[idx].contiguous(), W_head=inp.W_head, E=inp.E,
                  W_g=inp.W_g, x=inp.x[idx].contiguous())


def make_teacher_logits(shape: Shape, x: torch.Tensor, seed: int = 0, *, std: float = 2.0,
                        target_bump: float = 4.0) -> torch.Tensor:
    """Teacher logits [N, n, V] bf16 for the distillation objective: N(0, std) noise with the
    sequence's own token raised by ``target_bump`` (a frozen base model mostly agrees with its
    training data).  Drawn in slabs of positions from a generator of its own."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed + 104729)
    s = shape
    T = _randn_bf16(gen, (s.N, s.n, s.V), std)
    if target_bump != 0.0:
        idx = x.to(torch.int64).unsqueeze(-1)
        T.scatter_(2, idx, (T.gather(2, idx).float() + target_bump).to(torch.bfloat16))
    return T
