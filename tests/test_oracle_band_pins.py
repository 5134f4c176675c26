"""Pins of the row-band oracle (Sec. 3.4, Eq. 7): the band split, the reach of the window, and the patch-wise
average of the text rows against closed forms, special cases that reduce to the exact operator, and brute force."""
import math

import numpy as np
import pytest
import torch

from oracle import clear_oracle as oracle
from oracle import clear_oracle_bands as OB


def test_band_rows_partition_the_grid_evenly():
    for gh, n in ((128, 8), (13, 4), (7, 7), (512, 8), (10, 3), (5, 1)):
        rows = [OB.band_rows(gh, n, p) for p in range(n)]
        assert rows[0][0] == 0 and rows[-1][1] == gh
        assert all(rows[i][1] == rows[i + 1][0] for i in range(n - 1))
        sizes = [b - a for a, b in rows]
        assert max(sizes) - min(sizes) <= 1 and sorted(sizes, reverse=True) == sizes
    assert OB.band_rows(512, 8, 3) == (192, 256)   # H/N rows per GPU when N divides H (Sec. 3.4)
    with pytest.raises(ValueError):
        OB.band_rows(4, 5, 0)


def test_reach_is_the_largest_row_offset_the_mask_allows():
    # straight from the mask rows of the attention oracle: the farthest row with an allowed key in column x
    for r in (1.0, 2.0, 2.5, math.sqrt(2.0), 4.0, 8.0, 16.0):
        gh = gw = 40
        i = (gh // 2) * gw + gw // 2
        row = oracle.mask_row(i, gh, gw, 0, r).reshape(gh, gw)
        ys = np.nonzero(row.any(axis=1))[0]
        assert OB.reach(r) == ys.max() - gh // 2 == gh // 2 - ys.min()
    assert OB.reach(16.0) == 15 and OB.reach(8.0) == 7 and OB.reach(32.0) == 31


def _rand(B, H, gh, gw, T, d, seed):
    rng = np.random.default_rng(seed)
    N = T + gh * gw
    return (rng.normal(size=(B, H, N, d)), rng.normal(size=(B, H, N, d)), rng.normal(size=(B, H, N, d)))


def test_one_band_is_the_exact_operator():
    gh, gw, T, d = 6, 5, 4, 16
    q, k, v = _rand(1, 2, gh, gw, T, d, 1)
    want = oracle.attn(torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), gh, gw, T, 3.0, 0.25)[:, :, :T]
    got = OB.text_rows_patch_average(q, k, v, gh, gw, T, 0.25, 1)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


def test_patch_average_against_brute_force():
    gh, gw, T, d, G = 7, 3, 2, 8, 3
    q, k, v = _rand(1, 1, gh, gw, T, d, 2)
    got = OB.text_rows_patch_average(q, k, v, gh, gw, T, 0.3, G)
    bands = [(0, 3), (3, 5), (5, 7)]   # 7 rows in 3 bands: 3, 2, 2
    for i in range(T):
        acc = np.zeros(d)
        for y0, y1 in bands:
            js = list(range(T)) + [T + y * gw + x for y in range(y0, y1) for x in range(gw)]
            w = np.array([math.exp(0.3 * float(q[0, 0, i] @ k[0, 0, j])) for j in js])
            acc += sum(wj * v[0, 0, j] for wj, j in zip(w, js)) / w.sum()
        np.testing.assert_allclose(got[0, 0, i], acc / G, rtol=1e-12)


def test_closed_forms_at_zero_queries():
    # Q = 0: every band's softmax is uniform over its keys, so the output is the mean over bands of the mean of V
    gh, gw, T, d, G = 8, 4, 3, 5, 4
    q, k, v = _rand(1, 1, gh, gw, T, d, 3)
    q[:] = 0.0
    got = OB.text_rows_patch_average(q, k, v, gh, gw, T, 1.0, G)
    vt, vi = v[0, 0, :T], v[0, 0, T:].reshape(gh, gw, d)
    means = [(vt.sum(0) + vi[2 * p:2 * p + 2].sum((0, 1))) / (T + 2 * gw) for p in range(G)]
    np.testing.assert_allclose(got[0, 0], np.tile(np.mean(means, axis=0), (T, 1)), rtol=1e-12)
    # without text and with equal bands that is the mean over all image tokens: the exact result
    q2, k2, v2 = _rand(1, 1, gh, gw, 0, d, 4)
    assert OB.text_rows_patch_average(q2, k2, v2, gh, gw, 0, 1.0, G).shape == (1, 1, 0, d)


def test_constant_values_and_identical_bands():
    gh, gw, T, d, G = 6, 4, 2, 8, 3
    q, k, v = _rand(1, 2, gh, gw, T, d, 5)
    v[:] = 2.5
    np.testing.assert_allclose(OB.text_rows_patch_average(q, k, v, gh, gw, T, 0.4, G), 2.5, rtol=1e-13)
    # bands holding the same keys and values give the same softmax each: the average is any one of them
    q, k, v = _rand(1, 1, gh, gw, T, d, 6)
    for p in range(1, G):
        k[:, :, T + 2 * p * gw:T + 2 * (p + 1) * gw] = k[:, :, T:T + 2 * gw]
        v[:, :, T + 2 * p * gw:T + 2 * (p + 1) * gw] = v[:, :, T:T + 2 * gw]
    one = OB.text_rows_patch_average(q[:, :, :T + 2 * gw], k[:, :, :T + 2 * gw], v[:, :, :T + 2 * gw], 2, gw, T, 0.4, 1)
    np.testing.assert_allclose(OB.text_rows_patch_average(q, k, v, gh, gw, T, 0.4, G), one, rtol=1e-12)


def test_patch_average_is_an_approximation_not_the_exact_rows():
    gh, gw, T, d = 8, 8, 4, 16
    q, k, v = _rand(1, 1, gh, gw, T, d, 7)
    exact = oracle.attn(torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), gh, gw, T, 3.0, 0.5)[:, :, :T]
    approx = OB.text_rows_patch_average(q, k, v, gh, gw, T, 0.5, 4)
    assert np.abs(approx - exact).max() > 1e-3
