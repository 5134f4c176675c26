"""fp64 CPU oracle of what happens to Q and K between the projection and the attention call in the model
the paper linearises (Sec. 3.1: rotary position embedding on the two axes of the feature map; Sec. 4.3's
high-resolution recipe: a larger NTK factor for the rotary embedding and a log-scale attention factor).

TEST INFRASTRUCTURE ONLY: only the tests use it.  It imports nothing from the CUDA package and shares no code
with it.  Plain numpy in fp64, one definition per function, no fusion:

  rms_norm          x / sqrt(mean(x^2) + eps) * gain over the head's channels (the model's QK normalisation)
  rope_frequencies  w_k = base'^(-2k/dim), k < dim/2, with the NTK-aware base' = base * ntk^(dim/(dim-2))
                    (ntk = 1 leaves the base alone; the paper raises ntk from 1 to 10 beyond the training size)
  token_positions   text tokens sit at (0, 0, 0); image token p = y * grid_w + x at (0, y, x)
  rope              channels split into three axis groups (group a has axes_dim[a] channels); inside a group
                    the pair (2k, 2k+1) turns by the angle position[a] * w_k
  log_scale_factor  sqrt(log n / log n_train): the factor on the logits that keeps the attention entropy of a
                    sequence of n tokens where it was at the training length
  qk_prep           rope(rms_norm(q)) * q_factor and rope(rms_norm(k)): what the attention call consumes

The paper gives none of these formulas itself; they are the published definitions of the parts it names
(rotary embedding, NTK-aware base, entropy-keeping log factor, RMS normalisation), with the model's
conventions for the axis split and the pair layout.
"""
from __future__ import annotations

import numpy as np


def rms_norm(x: np.ndarray, gain: np.ndarray | None, eps: float) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    mean_sq = np.mean(x * x, axis=-1, keepdims=True)
    y = x / np.sqrt(mean_sq + float(eps))
    if gain is not None:
        y = y * np.asarray(gain, dtype=np.float64)
    return y


def rope_frequencies(dim: int, theta: float, ntk: float) -> np.ndarray:
    if dim <= 0 or dim % 2:
        raise ValueError("an axis group holds a positive even number of channels")
    base = float(theta)
    if dim > 2:
        base = base * float(ntk) ** (dim / (dim - 2.0))
    k = np.arange(dim // 2, dtype=np.float64)
    return base ** (-2.0 * k / dim)


def token_positions(grid_h: int, grid_w: int, n_text: int) -> np.ndarray:
    pos = np.zeros((n_text + grid_h * grid_w, 3), dtype=np.int64)
    p = np.arange(grid_h * grid_w)
    pos[n_text:, 1] = p // grid_w
    pos[n_text:, 2] = p % grid_w
    return pos


def rope(x: np.ndarray, positions: np.ndarray, axes_dim, theta: float, ntk: float) -> np.ndarray:
    """x: [..., N, d]; positions: [N, 3]."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    if sum(axes_dim) != d:
        raise ValueError("the axis groups must cover the head's channels")
    out = np.empty_like(x)
    c0 = 0
    for a, dim in enumerate(axes_dim):
        if dim == 0:
            continue
        w = rope_frequencies(dim, theta, ntk)                                  # [dim/2]
        ang = positions[:, a].astype(np.float64)[:, None] * w[None, :]       # [N, dim/2]
        cos, sin = np.cos(ang), np.sin(ang)
        even = x[..., c0:c0 + dim:2]
        odd = x[..., c0 + 1:c0 + dim:2]
        out[..., c0:c0 + dim:2] = even * cos - odd * sin
        out[..., c0 + 1:c0 + dim:2] = even * sin + odd * cos
        c0 += dim
    return out


def log_scale_factor(n_tokens: int, n_train_tokens: int) -> float:
    return float(np.sqrt(np.log(float(n_tokens)) / np.log(float(n_train_tokens))))


def qk_prep(q, k, gain_q, gain_k, grid_h, grid_w, n_text, axes_dim, theta=10000.0, ntk=1.0, eps=1e-6, q_factor=1.0):
    """q, k: [B, H, N, d] (any float dtype; widened to fp64).  Returns fp64 (q', k')."""
    pos = token_positions(grid_h, grid_w, n_text)
    q2 = rope(rms_norm(q, gain_q, eps), pos, axes_dim, theta, ntk) * float(q_factor)
    k2 = rope(rms_norm(k, gain_k, eps), pos, axes_dim, theta, ntk)
    return q2, k2


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest bf16 value (8 significant bits, ties to even) of every element, returned as fp64.  Normal range
    only: the values this is used on are of order one."""
    m, e = np.frexp(np.asarray(x, dtype=np.float64))   # x = m * 2^e, 0.5 <= |m| < 1
    return np.ldexp(np.rint(np.ldexp(m, 8)), e - 8)
