"""Pins of the backward oracle (`oracle/clear_oracle_bwd.c`) to things other than itself: automatic
differentiation of a dense masked attention written here, finite differences of the FORWARD oracle,
closed forms and invariants of the softmax.  All CPU."""
import math

import numpy as np
import pytest
import torch

from oracle import clear_oracle as fwd
from oracle import clear_oracle_bwd as bwd


def explicit_mask(gh, gw, T, r):
    """M of Eq. 3 as an N x N boolean matrix by broadcasting, with a real-valued comparison."""
    n = gh * gw
    ys, xs = np.divmod(np.arange(n), gw)
    d2 = (ys[:, None] - ys[None, :]) ** 2 + (xs[:, None] - xs[None, :]) ** 2
    M = np.ones((T + n, T + n), dtype=bool)
    M[T:, T:] = d2.astype(np.float64) < float(r) * float(r)
    return M


def autograd_reference(q, k, v, go, M, scale):
    q, k, v = (torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (q, k, v))
    s = scale * (q @ k.transpose(-1, -2))
    s = s.masked_fill(~torch.tensor(M), float("-inf"))
    out = torch.softmax(s, dim=-1) @ v
    out.backward(torch.tensor(go, dtype=torch.float64))
    return q.grad.numpy(), k.grad.numpy(), v.grad.numpy()


def rand_inputs(B, H, N, d, seed):
    rng = np.random.default_rng(seed)
    return [rng.standard_normal((B, H, N, d)) for _ in range(4)]


@pytest.mark.parametrize("gh,gw,T,r,d", [(5, 7, 3, 2.5, 8), (4, 4, 0, math.sqrt(2.0), 4), (6, 3, 5, 1.0, 16),
                                          (3, 9, 2, 3.0, 8), (1, 11, 1, 2.0, 4)])
def test_gradients_equal_autograd_of_a_dense_masked_attention(gh, gw, T, r, d):
    N = T + gh * gw
    q, k, v, go = rand_inputs(2, 2, N, d, seed=gh * 10 + gw)
    scale = 0.37
    dq, dk, dv = bwd.attn_bwd(q, k, v, go, gh, gw, T, r, scale)
    rq, rk, rv = autograd_reference(q, k, v, go, explicit_mask(gh, gw, T, r), scale)
    for got, want in ((dq, rq), (dk, rk), (dv, rv)):
        np.testing.assert_allclose(got, want, rtol=1e-10, atol=1e-12)


def test_radius_beyond_the_diagonal_is_plain_attention():
    gh, gw, T, d = 4, 5, 2, 8
    N = T + gh * gw
    q, k, v, go = rand_inputs(1, 2, N, d, seed=4)
    dq, dk, dv = bwd.attn_bwd(q, k, v, go, gh, gw, T, 100.0, 0.5)
    tq, tk, tv = (torch.tensor(a, requires_grad=True) for a in (q, k, v))
    out = torch.softmax(0.5 * tq @ tk.transpose(-1, -2), dim=-1) @ tv
    out.backward(torch.tensor(go))
    for got, want in ((dq, tq.grad), (dk, tk.grad), (dv, tv.grad)):
        np.testing.assert_allclose(got, want.numpy(), rtol=1e-10, atol=1e-12)


def test_gradients_equal_central_differences_of_the_forward_oracle():
    gh, gw, T, r, d = 4, 5, 2, 2.5, 4
    N = T + gh * gw
    q, k, v, go = rand_inputs(1, 1, N, d, seed=11)
    scale = 0.8
    dq, dk, dv = bwd.attn_bwd(q, k, v, go, gh, gw, T, r, scale)
    loss = lambda a, b, c: float((fwd.attn(a, b, c, gh, gw, T, r, scale) * go).sum())
    h = 1e-5
    rng = np.random.default_rng(2)
    for which, grad in ((0, dq), (1, dk), (2, dv)):
        for _ in range(6):
            idx = (0, 0, int(rng.integers(0, N)), int(rng.integers(0, d)))
            args = [q.copy(), k.copy(), v.copy()]
            args[which][idx] += h
            up = loss(*args)
            args[which][idx] -= 2 * h
            down = loss(*args)
            assert abs((up - down) / (2 * h) - grad[idx]) <= 1e-6 * max(1.0, abs(grad[idx]))


def test_zero_queries_give_closed_forms():
    """Q = 0: p_ij = 1 / count_i on the allowed keys.  With dO = 1 everywhere dV_j = sum over the queries that
    see key j of 1 / count_i in every channel, dK = 0 (it is a sum of multiples of the q_i), and
    dQ_i = scale * sum_j p_ij (dP_ij - mean_j dP_ij) k_j."""
    gh, gw, T, r, d = 6, 5, 3, 2.0, 4
    N = T + gh * gw
    rng = np.random.default_rng(5)
    k, v = rng.standard_normal((1, 1, N, d)), rng.standard_normal((1, 1, N, d))
    q = np.zeros((1, 1, N, d))
    go = np.ones((1, 1, N, d))
    dq, dk, dv = bwd.attn_bwd(q, k, v, go, gh, gw, T, r, 0.6)
    M = explicit_mask(gh, gw, T, r)
    P = M / M.sum(axis=1, keepdims=True)
    np.testing.assert_allclose(dv[0, 0], np.repeat(P.sum(axis=0)[:, None], d, axis=1), rtol=1e-12)
    assert np.abs(dk).max() == 0.0
    dP = v[0, 0].sum(axis=1)[None, :].repeat(N, axis=0)
    dS = P * (dP - (P * dP).sum(axis=1, keepdims=True))
    np.testing.assert_allclose(dq[0, 0], 0.6 * dS @ k[0, 0], rtol=1e-10, atol=1e-13)


def test_shift_invariance_of_the_softmax_shows_in_the_key_gradient():
    """Adding one vector to every key shifts all logits of a row alike and leaves the output as it is, so
    the key gradients of a (batch, head) slice sum to zero; and identity on V (radius 1, no text) passes the
    upstream gradient through."""
    gh, gw, T, r, d = 5, 6, 4, 3.0, 8
    N = T + gh * gw
    q, k, v, go = rand_inputs(2, 1, N, d, seed=8)
    dq, dk, dv = bwd.attn_bwd(q, k, v, go, gh, gw, T, r, 0.3)
    assert np.abs(dk.sum(axis=2)).max() <= 1e-12
    # every query's weights sum to one: the value gradients sum to the upstream gradients
    np.testing.assert_allclose(dv.sum(axis=2), go.sum(axis=2), rtol=1e-12)
    q, k, v, go = rand_inputs(1, 1, gh * gw, d, seed=9)
    dq, dk, dv = bwd.attn_bwd(q, k, v, go, gh, gw, 0, 1.0, 0.3)
    assert np.abs(dq).max() == 0.0 and np.abs(dk).max() == 0.0
    np.testing.assert_array_equal(dv, go)


def test_bf16_and_fp32_carriers_are_widened_exactly():
    gh, gw, T, r, d = 3, 4, 2, 2.0, 8
    N = T + gh * gw
    g = torch.Generator().manual_seed(1)
    q, k, v = (torch.randn(1, 1, N, d, generator=g).to(torch.bfloat16) for _ in range(3))
    go = torch.randn(1, 1, N, d, generator=g, dtype=torch.float64)
    a = bwd.attn_bwd(q, k, v, go, gh, gw, T, r, 0.5)
    b = bwd.attn_bwd(q.float(), k.float(), v.float(), go, gh, gw, T, r, 0.5)
    c = bwd.attn_bwd(q.double(), k.double(), v.double(), go, gh, gw, T, r, 0.5)
    for x, y, z in zip(a, b, c):
        assert np.array_equal(x, y) and np.array_equal(x, z)
    with pytest.raises(ValueError):
        bwd.attn_bwd(q, k, v, go, gh, gw, T, 0.0, 0.5)
