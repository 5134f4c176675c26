"""Pins for the fp64 CPU oracle: each test checks it against something other than itself.

- values the paper prints (the FLOP tables, `tests/golden/paper_flops.txt`);
- closed forms (lattice-point counts of the clipped disc, moments of the allowed set);
- special cases that reduce to textbook attention;
- brute force with an explicit N x N mask matrix written independently here.
"""
import math
import os
from decimal import ROUND_HALF_UP, Decimal

import numpy as np
import pytest
import torch

from oracle import clear_oracle as oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_flops.txt")


# ----------------------------------------------------------------------------------------------
# independent helpers (none of these call the oracle)
# ----------------------------------------------------------------------------------------------
def explicit_mask(gh, gw, T, r2_real):
    """N x N 0/1 matrix of Eq. 3 from coordinate arrays, real-valued comparison d^2 < r^2."""
    n = gh * gw
    N = T + n
    ys, xs = np.divmod(np.arange(n), gw)
    d2 = (xs[:, None] - xs[None, :]) ** 2 + (ys[:, None] - ys[None, :]) ** 2
    M = np.ones((N, N), dtype=bool)
    M[T:, T:] = d2.astype(np.float64) < r2_real
    return M


def dense_masked_attention(q, k, v, M, scale):
    """softmax(scale * Q K^T + log M) V with numpy matrices, fp64, all heads."""
    s = np.einsum("bhid,bhjd->bhij", q, k) * scale
    s = np.where(M[None, None], s, -np.inf)
    s = s - s.max(axis=-1, keepdims=True)
    p = np.exp(s)
    p = p / p.sum(axis=-1, keepdims=True)
    return np.einsum("bhij,bhjd->bhid", p, v)


def closed_form_count(y, x, gh, gw, T, thr):
    """Keys an image query at (y, x) may see: T text keys + lattice points of the open disc of
    squared radius thr around it, clipped to the grid (row by row: half-width m(dy) is the
    largest m with m^2 + dy^2 < thr)."""
    c = T
    for yy in range(gh):
        dy2 = (yy - y) ** 2
        if dy2 >= thr:
            continue
        m = math.isqrt(thr - 1 - dy2)
        c += min(x + m, gw - 1) - max(x - m, 0) + 1
    return c


def rand_qkv(B, H, N, d, seed):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((B, H, N, d)), rng.standard_normal((B, H, N, d)),
            rng.standard_normal((B, H, N, d)))


# ----------------------------------------------------------------------------------------------
# the paper's printed numbers
# ----------------------------------------------------------------------------------------------
def _golden_rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            res, setting, val, unit, digits, src = line.split()
            rows.append((int(res), setting, val, unit, int(digits), src))
    return rows


_SUM_CACHE = {}


def _sum_mask(res, setting):
    key = (res, setting)
    if key not in _SUM_CACHE:
        g = res // 16
        if setting == "dense":
            _SUM_CACHE[key] = (512 + g * g) ** 2
        else:
            _SUM_CACHE[key] = oracle.mask_counts(g, g, 512, float(setting), want_counts=False)[0]
    return _SUM_CACHE[key]


@pytest.mark.parametrize("res,setting,val,unit,digits,src", _golden_rows())
def test_mask_total_reproduces_printed_flops(res, setting, val, unit, digits, src):
    """4 * sum(M) * c with c = 3072 must round to every figure the paper prints."""
    flops = 4 * _sum_mask(res, setting) * 3072
    want = Decimal(val)
    q = Decimal(1).scaleb(-digits)
    if unit == "G":
        got = {(Decimal(flops) / Decimal(10 ** 9)).quantize(q, ROUND_HALF_UP)}
    else:
        # TFLOPS cells: rounded directly, or from the one-decimal GFLOPS figure the other tables
        # print (13084.97 G -> 13085.0 G -> 13.09 T is the one cell where the two differ)
        direct = (Decimal(flops) / Decimal(10 ** 12)).quantize(q, ROUND_HALF_UP)
        giga = (Decimal(flops) / Decimal(10 ** 9)).quantize(Decimal("0.1"), ROUND_HALF_UP)
        got = {direct, (giga / 1000).quantize(q, ROUND_HALF_UP)}
    assert want in got, (res, setting, flops, val, src)


def test_headline_saving_is_the_r8_8k_cell():
    """'99.5% fewer attention computations' = 1 - FLOPs(r=8) / FLOPs(dense) at 8192."""
    frac = 1.0 - _sum_mask(8192, "8") / _sum_mask(8192, "dense")
    assert f"{100 * frac:.1f}" == "99.5"


def test_alternative_readings_do_not_reproduce_the_table():
    """'<=' at distance r, or NATTEN-style constant-size border windows, miss the printed 63.5."""
    g, T, r = 64, 512, 8
    M_le = explicit_mask(g, g, T, r * r + 0.5)           # d2 <= r^2 for integer d2
    assert f"{4 * int(M_le.sum()) * 3072 / 1e9:.1f}" != "63.5"
    M_lt = explicit_mask(g, g, T, r * r)
    assert f"{4 * int(M_lt.sum()) * 3072 / 1e9:.1f}" == "63.5"
    interior = 193                                       # every image query sees a full disc
    natten_total = T * (T + g * g) + g * g * (T + interior)
    assert f"{4 * natten_total * 3072 / 1e9:.1f}" != "63.5"


# ----------------------------------------------------------------------------------------------
# mask: brute force, closed form, structure
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("gh,gw,T,r", [(5, 7, 3, 2.0), (6, 4, 0, 2.5), (4, 9, 2, math.sqrt(2.0)),
                                        (7, 7, 5, 1.0), (3, 11, 1, 3.0), (8, 8, 4, 100.0),
                                        (13, 19, 7, 4.0)])
def test_mask_rows_equal_explicit_matrix(gh, gw, T, r):
    M = explicit_mask(gh, gw, T, r * r)
    N = T + gh * gw
    got = np.stack([oracle.mask_row(i, gh, gw, T, r) for i in range(N)]).astype(bool)
    assert np.array_equal(got, M)
    assert np.array_equal(got, got.T)                    # Eq. 3 is symmetric in (i, j)
    total, counts = oracle.mask_counts(gh, gw, T, r)
    assert total == int(M.sum())
    assert np.array_equal(counts, M.sum(axis=1))


@pytest.mark.parametrize("r,interior", [(4, 45), (8, 193), (16, 793), (32, 3205)])
def test_interior_count_is_gauss_circle_minus_axis_points(r, interior):
    """Open disc of integer radius r: lattice points with d2 <= r^2 minus those at exactly r
    (r^2 in {16, 64, 256, 1024} is a sum of two squares only as r^2 + 0)."""
    closed = sum(1 for dy in range(-r, r + 1) for dx in range(-r, r + 1) if dx * dx + dy * dy <= r * r)
    assert closed - 4 == interior
    g = 2 * r + 3
    T = 5
    i = T + (r + 1) * g + (r + 1)
    assert int(oracle.mask_row(i, g, g, T, float(r)).sum()) - T == interior


@pytest.mark.parametrize("gh,gw,T,r", [(16, 16, 16, 4.0), (13, 19, 7, 4.0), (40, 24, 0, 8.0),
                                        (9, 33, 130, 5.5), (64, 64, 512, 8.0)])
def test_per_query_counts_equal_closed_form(gh, gw, T, r):
    thr = math.ceil(r * r)
    total, counts = oracle.mask_counts(gh, gw, T, r)
    N = T + gh * gw
    assert np.all(counts[:T] == N)
    want = np.array([closed_form_count(y, x, gh, gw, T, thr) for y in range(gh) for x in range(gw)])
    assert np.array_equal(counts[T:], want)
    assert total == T * N + int(want.sum())
    # mask_row (used by the attention loop) and mask_counts are two code paths: tie them together
    for i in [0, T, T + gw - 1, T + gw, N - 1, T + (gh // 2) * gw + gw // 2]:
        if i < N:
            assert int(oracle.mask_row(i, gh, gw, T, r).sum()) == counts[i]


def test_circle_to_square_ratio_tends_to_pi_over_4():
    """Sec. 3.2: a circular window costs about pi/4 of the square one."""
    ratios = [n / (2 * r - 1) ** 2 for r, n in [(16, 793), (32, 3205)]]
    assert ratios[0] > ratios[1] > math.pi / 4
    assert abs(ratios[1] - math.pi / 4) < 0.03


# ----------------------------------------------------------------------------------------------
# attention values
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("gh,gw,T,r,d,seed", [(5, 7, 3, 2.0, 8, 1), (6, 4, 0, 2.5, 4, 2),
                                               (4, 9, 2, math.sqrt(2.0), 16, 3), (7, 5, 6, 3.0, 5, 4)])
def test_attention_equals_brute_force_with_explicit_mask(gh, gw, T, r, d, seed):
    N = T + gh * gw
    q, k, v = rand_qkv(2, 3, N, d, seed)
    scale = 0.37
    want = dense_masked_attention(q, k, v, explicit_mask(gh, gw, T, r * r), scale)
    got = oracle.attn(q, k, v, gh, gw, T, r, scale)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


def test_large_radius_is_full_joint_attention():
    """r beyond the grid diagonal: every pair allowed -> torch's softmax attention."""
    gh, gw, T, d = 6, 9, 4, 16
    N = T + gh * gw
    q, k, v = rand_qkv(1, 2, N, d, 7)
    r = math.hypot(gh - 1, gw - 1) + 1e-3
    scale = 1 / math.sqrt(d)
    tq, tk, tv = (torch.from_numpy(a) for a in (q, k, v))
    want = torch.softmax(tq @ tk.transpose(-1, -2) * scale, dim=-1) @ tv
    got = oracle.attn(q, k, v, gh, gw, T, r, scale)
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-12, atol=1e-13)
    # just inside the diagonal the two far corners stop seeing each other
    r_in = math.hypot(gh - 1, gw - 1)
    row = oracle.mask_row(T, gh, gw, T, r_in)
    assert row[-1] == 0 and row.sum() == N - 1


def test_radius_one_without_text_is_identity_on_values():
    gh, gw, d = 5, 6, 8
    q, k, v = rand_qkv(1, 2, gh * gw, d, 11)
    got = oracle.attn(q, k, v, gh, gw, 0, 1.0, 0.5)
    np.testing.assert_allclose(got, v, rtol=0, atol=1e-15)


def test_rows_are_convex_combinations():
    gh, gw, T, d = 9, 7, 5, 6
    N = T + gh * gw
    q, k, v = rand_qkv(1, 2, N, d, 13)
    ones = np.ones_like(v)
    np.testing.assert_allclose(oracle.attn(q, k, ones, gh, gw, T, 3.0, 0.8), ones, rtol=0, atol=1e-14)
    out = oracle.attn(q, k, v, gh, gw, T, 3.0, 0.8)
    assert np.all(out <= v.max(axis=2, keepdims=True) + 1e-12)
    assert np.all(out >= v.min(axis=2, keepdims=True) - 1e-12)


def test_zero_queries_give_moments_of_the_allowed_set():
    """Q = 0 -> uniform weights: out_i = mean of V over A_i.  With V columns
    (1, x, y, x^2, y^2, is_text) the image rows have closed forms from the clipped disc."""
    gh, gw, T, r = 11, 14, 3, 3.5
    thr = math.ceil(r * r)
    n = gh * gw
    N = T + n
    ys, xs = np.divmod(np.arange(n), gw)
    v = np.zeros((1, 1, N, 6))
    v[..., 0] = 1.0
    v[0, 0, T:, 1] = xs
    v[0, 0, T:, 2] = ys
    v[0, 0, T:, 3] = xs ** 2
    v[0, 0, T:, 4] = ys ** 2
    v[0, 0, :T, 5] = 1.0
    q = np.zeros((1, 1, N, 6))
    k = np.random.default_rng(5).standard_normal((1, 1, N, 6))
    out = oracle.attn(q, k, v, gh, gw, T, r, 1.0)[0, 0]
    for y in range(gh):
        for x in range(gw):
            sx = sy = sxx = syy = cnt = 0
            for yy in range(gh):
                dy2 = (yy - y) ** 2
                if dy2 >= thr:
                    continue
                m = math.isqrt(thr - 1 - dy2)
                lo, hi = max(x - m, 0), min(x + m, gw - 1)
                w = hi - lo + 1
                cnt += w
                sx += (lo + hi) * w // 2
                sxx += sum(t * t for t in range(lo, hi + 1))
                sy += yy * w
                syy += yy * yy * w
            tot = cnt + T
            want = np.array([1.0, sx / tot, sy / tot, sxx / tot, syy / tot, T / tot])
            np.testing.assert_allclose(out[T + y * gw + x], want, rtol=1e-13, atol=1e-13)
    # text rows average over everything
    np.testing.assert_allclose(out[0], v[0, 0].mean(axis=0), rtol=1e-13)


def test_planted_key_membership_at_the_threshold_and_across_row_wrap():
    """A one-hot V column reads membership and count: out = 1/|A_i| if the key is allowed else 0."""
    gh, gw, T, r = 9, 9, 2, 3.0          # thr = 9
    N = T + gh * gw
    q = np.zeros((1, 1, N, 2))
    k = np.zeros((1, 1, N, 2))

    def probe(qy, qx, ky, kx):
        v = np.zeros((1, 1, N, 2))
        v[0, 0, T + ky * gw + kx, 0] = 1.0
        return oracle.attn_rows(q, k, v, gh, gw, T, r, 1.0, [[0, 0, T + qy * gw + qx]])[0, 0]

    cnt = closed_form_count(4, 4, gh, gw, T, 9)
    assert probe(4, 4, 4, 6) == pytest.approx(1 / cnt)      # d2 = 4 < 9
    assert probe(4, 4, 6, 6) == pytest.approx(1 / cnt)      # d2 = 8 = thr - 1
    assert probe(4, 4, 4, 7) == 0.0                         # d2 = 9 = thr: excluded (strict <)
    assert probe(4, 4, 7, 4) == 0.0
    # (4, 8) and (5, 0) are neighbours in token order but 8 columns apart on the grid
    assert probe(4, 8, 5, 0) == 0.0
    assert probe(5, 0, 4, 8) == 0.0
    assert probe(4, 8, 5, 8) == pytest.approx(1 / closed_form_count(4, 8, gh, gw, T, 9))


def test_softmax_weights_follow_the_logits():
    """Two allowed keys with logits a and b: weights are the logistic function of (a - b)."""
    gh, gw, T, d = 1, 2, 0, 1
    q = np.array([1.5, 1.5]).reshape(1, 1, 2, 1)
    k = np.array([0.2, -0.7]).reshape(1, 1, 2, 1)
    v = np.array([1.0, 0.0]).reshape(1, 1, 2, 1)
    scale = 2.0
    out = oracle.attn(q, k, v, gh, gw, T, 1.5, scale)
    w0 = 1 / (1 + math.exp(-scale * 1.5 * (0.2 + 0.7)))
    np.testing.assert_allclose(out[0, 0, :, 0], [w0, w0], rtol=1e-14)


def test_transposing_the_grid_permutes_the_outputs():
    gh, gw, T, d, r = 5, 8, 3, 4, 2.5
    n = gh * gw
    q, k, v = rand_qkv(1, 1, T + n, d, 17)
    out = oracle.attn(q, k, v, gh, gw, T, r, 0.6)
    perm = np.arange(n).reshape(gh, gw).T.reshape(-1)        # token order of the transposed grid
    idx = np.concatenate([np.arange(T), T + perm])
    out_t = oracle.attn(q[:, :, idx], k[:, :, idx], v[:, :, idx], gw, gh, T, r, 0.6)
    np.testing.assert_allclose(out_t, out[:, :, idx], rtol=1e-13, atol=1e-14)


def test_text_rows_and_text_keys_ignore_the_radius():
    gh, gw, T, d = 6, 6, 4, 8
    N = T + gh * gw
    q, k, v = rand_qkv(1, 2, N, d, 19)
    a = oracle.attn(q, k, v, gh, gw, T, 1.0, 0.5)
    b = oracle.attn(q, k, v, gh, gw, T, 4.0, 0.5)
    np.testing.assert_allclose(a[:, :, :T], b[:, :, :T], rtol=1e-14)
    assert np.abs(a[:, :, T:] - b[:, :, T:]).max() > 1e-3
    # an image query at r = 1 sees the text keys and itself only
    i = T + 2 * gw + 3
    sel = np.r_[np.arange(T), i]
    s = (q[0, 0, i] @ k[0, 0, sel].T) * 0.5
    p = np.exp(s - s.max())
    p /= p.sum()
    np.testing.assert_allclose(a[0, 0, i], p @ v[0, 0, sel], rtol=1e-13)


def test_input_widths_are_widened_exactly():
    """bf16 bits, fp32 and fp64 carriers of the same values give the same result."""
    gh, gw, T, d = 4, 5, 3, 8
    N = T + gh * gw
    g = torch.Generator().manual_seed(3)
    q, k, v = (torch.randn(1, 2, N, d, generator=g).to(torch.bfloat16) for _ in range(3))
    o16 = oracle.attn(q, k, v, gh, gw, T, 2.0, 0.3)
    o32 = oracle.attn(q.float(), k.float(), v.float(), gh, gw, T, 2.0, 0.3)
    o64 = oracle.attn(q.double().numpy(), k.double().numpy(), v.double().numpy(), gh, gw, T, 2.0, 0.3)
    assert np.array_equal(o16, o32) and np.array_equal(o32, o64)
    rows = [[0, 1, 0], [0, 0, T + 7], [0, 1, N - 1]]
    sub = oracle.attn_rows(q, k, v, gh, gw, T, 2.0, 0.3, rows)
    assert np.array_equal(sub, np.stack([o16[b, h, i] for b, h, i in rows]))


def test_bad_arguments_are_rejected():
    q = np.zeros((1, 1, 4, 2))
    for r in (0.0, -1.0, float("nan"), float("inf")):
        with pytest.raises(ValueError):
            oracle.attn(q, q, q, 2, 2, 0, r, 1.0)
    with pytest.raises(ValueError):
        oracle.attn(q, q, q, 2, 3, 0, 1.0, 1.0)
    with pytest.raises(ValueError):
        oracle.attn_rows(q, q, q, 2, 2, 0, 1.0, 1.0, [[0, 0, 4]])
