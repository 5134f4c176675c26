"""fp64 CPU oracle of the row-band (patch-wise) parallel form of the operator (Sec. 3.4).

TEST INFRASTRUCTURE ONLY: only the tests use it.  It imports nothing from the CUDA package and shares no code
with it.  Plain numpy in fp64.

Sec. 3.4 cuts the H x W feature map into N bands of rows, one per GPU.  Image queries need the keys of at most
`reach` rows above and below their band (what adjacent GPUs exchange); the exact result for every token is the
single-GPU result, so the oracle of the exact band-parallel form is the plain attention oracle and is not repeated
here.  What is defined here:

  band_rows                rows [y0, y1) of band p when grid_h rows are cut into n_bands bands as evenly as possible
                           (the first grid_h % n_bands bands are one row taller)
  reach                    the largest row offset at which Eq. 3 lets an image query see a key: max dy, dy^2 < ceil(r^2)
  text_rows_patch_average  Eq. 7: for the text queries, the average over the bands of
                           softmax(Q_text K_p^T * scale) V_p, K_p and V_p being the keys and values GPU p holds: the
                           text tokens and the image tokens of band p (every GPU holds the text tokens; the paper
                           does not say so in so many words: this is the reading taken)
"""
from __future__ import annotations

import math

import numpy as np


def band_rows(grid_h: int, n_bands: int, p: int) -> tuple[int, int]:
    if not (0 < n_bands <= grid_h and 0 <= p < n_bands):
        raise ValueError("1 <= n_bands <= grid_h, 0 <= p < n_bands")
    base, extra = divmod(grid_h, n_bands)
    y0 = p * base + min(p, extra)
    return y0, y0 + base + (1 if p < extra else 0)


def reach(radius: float) -> int:
    thr = math.ceil(float(radius) * float(radius))
    dy = 0
    while (dy + 1) * (dy + 1) < thr:
        dy += 1
    return dy


def text_rows_patch_average(q, k, v, grid_h: int, grid_w: int, n_text: int, scale: float, n_bands: int) -> np.ndarray:
    """q, k, v: [B, H, N, d].  Returns the [B, H, n_text, d] fp64 outputs of the text queries under Eq. 7."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    B, H, N, d = q.shape
    if N != n_text + grid_h * grid_w:
        raise ValueError("token axis does not match n_text + grid_h*grid_w")
    out = np.zeros((B, H, n_text, d), dtype=np.float64)
    for p in range(n_bands):
        y0, y1 = band_rows(grid_h, n_bands, p)
        keys = np.concatenate([np.arange(n_text), n_text + np.arange(y0 * grid_w, y1 * grid_w)])
        s = np.einsum("bhid,bhjd->bhij", q[:, :, :n_text], k[:, :, keys]) * float(scale)
        s = s - s.max(axis=-1, keepdims=True)
        w = np.exp(s)
        w = w / w.sum(axis=-1, keepdims=True)
        out += np.einsum("bhij,bhjd->bhid", w, v[:, :, keys])
    return out / n_bands
