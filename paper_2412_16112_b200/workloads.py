"""Seeded synthetic workloads shaped like the paper's FLUX runs.

This module only names the configurations and draws their inputs.  It holds
none of the attention arithmetic and is the one module both the CUDA tests and
the CPU oracle's tests use, so that both sides see identical bits.

The paper's measurements use FLUX-1.dev activations (24 heads of 128 channels,
512 text tokens, a latent token grid of resolution/16).  Those activations are
not available here; Gaussian tensors of the same shapes stand in, with Q and K
RMS-normalised per token and head as FLUX's QK-norm leaves them.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Tuple

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    head_dim: int
    grid_h: int
    grid_w: int
    n_text: int
    radius: float
    dtype: str          # "bf16" or "f32"
    qk_norm: bool       # RMS-normalise Q and K per (token, head)
    seed: int

    @property
    def n_tokens(self) -> int:
        return self.n_text + self.grid_h * self.grid_w

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32


def _w(name, H, d, gh, gw, T, r, dtype, qk_norm, seed) -> Workload:
    return Workload(name, 1, H, d, gh, gw, T, float(r), dtype, qk_norm, seed)


WORKLOADS: Dict[str, Workload] = {w.name: w for w in [
    _w("c0_tiny_f32", 2, 64, 16, 16, 16, 4, "f32", False, 1000),
    _w("c1_1024px_r8", 24, 128, 64, 64, 512, 8, "bf16", True, 1001),
    _w("c2_2048px_r16", 24, 128, 128, 128, 512, 16, "bf16", True, 1002),
    _w("c3_4096px_r8", 24, 128, 256, 256, 512, 8, "bf16", True, 1003),
    _w("c3_4096px_r16", 24, 128, 256, 256, 512, 16, "bf16", True, 1003),
    _w("c3_4096px_r32", 24, 128, 256, 256, 512, 32, "bf16", True, 1003),
    _w("c3_192x320_r16", 24, 128, 192, 320, 512, 16, "bf16", True, 1013),
    _w("c4_8k_r16", 24, 128, 512, 512, 512, 16, "bf16", True, 1004),
]}


def _draw(gen: torch.Generator, n_bh: int, n_tok: int, d: int, norm: bool,
          dtype: torch.dtype) -> torch.Tensor:
    """One tensor, head by head (bounded peak memory; the order of draws is part of the recipe)."""
    out = torch.empty(n_bh, n_tok, d, dtype=dtype)
    for i in range(n_bh):
        x = torch.randn(n_tok, d, generator=gen, dtype=torch.float32)
        if norm:
            x = x / torch.sqrt(x.pow(2).mean(dim=-1, keepdim=True) + 1e-6)
        out[i] = x.to(dtype)
    return out


def make_inputs(w: Workload, heads: int | None = None) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """CPU tensors q, k, v of shape [B, H, N, d] in the workload's dtype.

    Draw order: all of Q (head by head), then K, then V, from one CPU generator
    seeded with ``w.seed``.  ``heads`` overrides H (a cheaper variant of the
    same distribution for tests; it is a different stream, not a slice).
    """
    H = w.H if heads is None else heads
    gen = torch.Generator(device="cpu").manual_seed(w.seed)
    shape = (w.B, H, w.n_tokens, w.head_dim)
    q = _draw(gen, w.B * H, w.n_tokens, w.head_dim, w.qk_norm, w.torch_dtype).view(shape)
    k = _draw(gen, w.B * H, w.n_tokens, w.head_dim, w.qk_norm, w.torch_dtype).view(shape)
    v = _draw(gen, w.B * H, w.n_tokens, w.head_dim, False, w.torch_dtype).view(shape)
    return q, k, v


def make_custom(B, H, grid_h, grid_w, n_text, head_dim, dtype="bf16", qk_norm=True, seed=0):
    """Inputs for an ad-hoc shape with the same value distribution."""
    w = Workload("custom", B, H, head_dim, grid_h, grid_w, n_text, 1.0, dtype, qk_norm, seed)
    return make_inputs(w)


def make_gains(head_dim: int, seed: int = 0) -> Tuple[torch.Tensor, torch.Tensor]:
    """Gain vectors of a Q and a K normalisation layer, fp32 [head_dim]: 1 + 0.1 N(0, 1) (learned gains stay
    near their initial value of one)."""
    gen = torch.Generator(device="cpu").manual_seed(7000 + seed)
    gq = 1.0 + 0.1 * torch.randn(head_dim, generator=gen, dtype=torch.float32)
    gk = 1.0 + 0.1 * torch.randn(head_dim, generator=gen, dtype=torch.float32)
    return gq, gk
