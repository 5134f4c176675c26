"""Pins of the window-kind oracle (`oracle/clear_oracle_windows.c`): closed-form counts, the FLOP figures the
paper prints for its windowed baselines, the pi / 4 remark, brute force with explicit mask matrices, and agreement of
its disc with the forward oracle's mask.  All CPU."""
import math

import numpy as np
import pytest
import torch

from oracle import clear_oracle as fwd
from oracle import clear_oracle_windows as win


def grid_xy(gh, gw):
    ys, xs = np.divmod(np.arange(gh * gw), gw)
    return ys, xs


def explicit_mask(kind, a, b, gh, gw, T):
    ys, xs = grid_xy(gh, gw)
    dy, dx = ys[None, :] - ys[:, None], xs[None, :] - xs[:, None]
    if kind == win.DISC:
        img = (dx * dx + dy * dy).astype(np.float64) < a * a
    elif kind == win.SQUARE:
        img = np.maximum(np.abs(dx), np.abs(dy)).astype(np.float64) < a
    elif kind == win.WINDOWS:
        wy, wx = (ys + b) // a, (xs + b) // a
        img = (wy[:, None] == wy[None, :]) & (wx[:, None] == wx[None, :])
    else:
        img = (np.mod(dx, a) == b % a) & (np.mod(dy, a) == (b // a) % a)
    M = np.ones((T + gh * gw, T + gh * gw), dtype=bool)
    M[T:, T:] = img
    return M


@pytest.mark.parametrize("kind,a,b", [(win.DISC, 2.5, 0), (win.SQUARE, 3.0, 0), (win.SQUARE, 2.5, 0), (win.WINDOWS, 4, 0),
                                      (win.WINDOWS, 4, 2), (win.STRIDED, 3, 0), (win.STRIDED, 3, 5)])
def test_mask_rows_and_counts_equal_the_explicit_matrix(kind, a, b):
    gh, gw, T = 9, 11, 3
    M = explicit_mask(kind, a, b, gh, gw, T)
    total, counts = win.mask_counts(kind, a, b, gh, gw, T)
    assert total == int(M.sum()) and np.array_equal(counts, M.sum(axis=1))
    for i in (0, T - 1, T, T + 5, T + gw + 3, T + gh * gw - 1):
        assert np.array_equal(win.mask_row(kind, a, b, i, gh, gw, T).astype(bool), M[i])


def test_the_disc_is_the_forward_oracles_mask():
    gh, gw, T = 13, 19, 7
    for r in (1.0, math.sqrt(2.0), 2.5, 4.0, 100.0):
        total, counts = win.mask_counts(win.DISC, r, 0, gh, gw, T)
        ftotal, fcounts = fwd.mask_counts(gh, gw, T, r)
        assert total == ftotal and np.array_equal(counts, fcounts)


def test_square_window_counts_have_a_closed_form():
    """A query at (y, x) sees the clipped box of half side ceil(r) - 1 around it, plus the text tokens."""
    gh, gw, T = 17, 23, 5
    for r in (1.0, 2.5, 3.0, 8.0, 40.0):
        h = math.ceil(r) - 1
        ys, xs = grid_xy(gh, gw)
        want = T + (np.minimum(ys + h, gh - 1) - np.maximum(ys - h, 0) + 1) * (np.minimum(xs + h, gw - 1) - np.maximum(xs - h, 0) + 1)
        _, counts = win.mask_counts(win.SQUARE, r, 0, gh, gw, T)
        assert np.array_equal(counts[T:], want) and (counts[:T] == T + gh * gw).all()


def test_circle_costs_about_pi_over_four_of_the_square():
    """Sec. 3.2: against the corresponding square window the circular one costs about pi / 4.  Interior queries,
    where the windows are whole: (2r - 1)^2 keys in the square."""
    gh = gw = 96
    centre = gh // 2 * gw + gw // 2
    ratios = []
    for r in (8, 16, 32):
        _, disc = win.mask_counts(win.DISC, r, 0, gh, gw, 0)
        _, square = win.mask_counts(win.SQUARE, r, 0, gh, gw, 0)
        assert square[centre] == (2 * r - 1) ** 2
        ratios.append(disc[centre] / square[centre])
    # 193/225, 793/961, 3205/3969: down towards pi / 4 from above
    assert ratios == sorted(ratios, reverse=True) and all(x > math.pi / 4 for x in ratios)
    assert abs(ratios[0] - 193 / 225) < 1e-12 and abs(ratios[-1] - math.pi / 4) < 0.025


def test_flop_figures_the_paper_prints_for_the_windowed_baselines():
    """Tab. 1 (1024px: 64 x 64 grid, 512 text tokens, c = 3072): Swin windows of 16 and the strided mask at ratio 4
    both print 67.7 GFLOPS; 4 * sum(M) * c gives 67.65 for either (a window or a stride class holds 256 keys)."""
    for kind, a, b in ((win.WINDOWS, 16, 0), (win.STRIDED, 4, 0), (win.STRIDED, 4, 7)):
        total, counts = win.mask_counts(kind, a, b, 64, 64, 512)
        assert (counts[512:] == 512 + 256).all()
        assert abs(4 * total * 3072 / 1e9 - 67.7) < 0.1
    shifted, _ = win.mask_counts(win.WINDOWS, 16, 8, 64, 64, 512)      # odd layers: border windows are smaller
    assert shifted < total


@pytest.mark.parametrize("kind,a,b", [(win.SQUARE, 2.5, 0), (win.SQUARE, 4.0, 0), (win.WINDOWS, 4, 2), (win.STRIDED, 2, 1)])
def test_attention_equals_brute_force_with_the_explicit_mask(kind, a, b):
    gh, gw, T, d = 6, 7, 3, 8
    N = T + gh * gw
    rng = np.random.default_rng(kind * 10 + int(a))
    q, k, v = (rng.standard_normal((1, 2, N, d)) for _ in range(3))
    got = win.attn(q, k, v, gh, gw, T, kind, a, b, 0.4)
    M = torch.tensor(explicit_mask(kind, a, b, gh, gw, T))
    s = (0.4 * torch.tensor(q) @ torch.tensor(k).transpose(-1, -2)).masked_fill(~M, float("-inf"))
    want = (torch.softmax(s, dim=-1) @ torch.tensor(v)).numpy()
    np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-13)


def test_disc_attention_is_the_forward_oracles():
    gh, gw, T, d = 7, 9, 4, 8
    rng = np.random.default_rng(3)
    q, k, v = (rng.standard_normal((1, 1, T + gh * gw, d)) for _ in range(3))
    a = win.attn(q, k, v, gh, gw, T, win.DISC, 2.5, 0, 0.3)
    np.testing.assert_allclose(a, fwd.attn(q, k, v, gh, gw, T, 2.5, 0.3), rtol=1e-12, atol=1e-14)
    with pytest.raises(ValueError):
        win.attn(q, k, v, gh, gw, T, 7, 2.5, 0, 0.3)
