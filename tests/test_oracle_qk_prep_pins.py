"""Pins of the Q/K preparation oracle (RMS normalisation, rotary embedding on the feature map's two axes with an
NTK factor, log-scale attention factor) against what the mathematics fixes: closed forms, invariants, the
complex-number form of a rotation, and the defining property of a rotary embedding -- a logit depends on the
relative offset of query and key only (Sec. 3.1 speaks of exactly these relative distances on the two axes).
"""
import numpy as np
import pytest

from oracle import clear_oracle_qk_prep as O

AXES = (16, 56, 56)


def test_rms_norm_rows_have_unit_mean_square():
    rng = np.random.default_rng(1)
    x = rng.normal(size=(3, 5, 64)) * 7.0
    y = O.rms_norm(x, None, 0.0)
    np.testing.assert_allclose(np.mean(y * y, axis=-1), 1.0, rtol=1e-13)
    # no dependence on the row's scale, a gain multiplies channel by channel
    np.testing.assert_allclose(O.rms_norm(3.0 * x, None, 0.0), y, rtol=1e-13)
    g = rng.normal(size=64)
    np.testing.assert_allclose(O.rms_norm(x, g, 0.0), y * g, rtol=1e-13)


def test_rms_norm_closed_forms():
    # a constant row c becomes sign(c); one hot of height a over d channels becomes sqrt(d) there
    np.testing.assert_allclose(O.rms_norm(np.full((1, 8), -2.5), None, 0.0), -1.0)
    x = np.zeros((1, 16))
    x[0, 3] = 4.0
    y = O.rms_norm(x, None, 0.0)
    assert y[0, 3] == pytest.approx(4.0) and np.count_nonzero(y) == 1
    # eps enters under the root next to the mean square: x = (1, 1, 1, 1), eps = 3 -> 1 / sqrt(1 + 3)
    np.testing.assert_allclose(O.rms_norm(np.ones((1, 4)), None, 3.0), 0.5)


def test_frequencies_closed_forms_and_the_ntk_property():
    w = O.rope_frequencies(56, 10000.0, 1.0)
    assert w.shape == (28,) and w[0] == 1.0
    assert w[1] == pytest.approx(10000.0 ** (-2.0 / 56.0), rel=1e-14)
    assert w[-1] == pytest.approx(10000.0 ** (-54.0 / 56.0), rel=1e-14)
    assert np.all(np.diff(np.log(w)) < 0) and np.allclose(np.diff(np.log(w)), np.log(w[1]))  # geometric
    # the NTK-aware base leaves the highest frequency alone and divides the lowest by the factor exactly
    for ntk in (2.0, 10.0):
        v = O.rope_frequencies(56, 10000.0, ntk)
        assert v[0] == 1.0
        assert v[-1] == pytest.approx(w[-1] / ntk, rel=1e-13)
        assert np.all(v[1:] < w[1:])
    with pytest.raises(ValueError):
        O.rope_frequencies(7, 10000.0, 1.0)


def test_token_positions():
    pos = O.token_positions(3, 5, 4)
    assert pos.shape == (19, 3)
    assert not pos[:4].any() and not pos[:, 0].any()
    assert tuple(pos[4]) == (0, 0, 0) and tuple(pos[4 + 7]) == (0, 1, 2) and tuple(pos[-1]) == (0, 2, 4)


def test_rope_is_a_rotation_of_every_pair_by_position_times_frequency():
    rng = np.random.default_rng(2)
    gh, gw, T, d = 5, 7, 3, 128
    x = rng.normal(size=(2, gh * gw + T, d))
    pos = O.token_positions(gh, gw, T)
    y = O.rope(x, pos, AXES, 10000.0, 1.0)
    # the same thing with complex numbers: pair (2k, 2k+1) is z = a + ib, turned by exp(i * angle)
    z = x[..., 0::2] + 1j * x[..., 1::2]
    ang = np.concatenate([pos[:, a:a + 1] * O.rope_frequencies(AXES[a], 10000.0, 1.0)[None, :] for a in range(3)], axis=1)
    zr = z * np.exp(1j * ang)
    np.testing.assert_allclose(y[..., 0::2], zr.real, atol=1e-13)
    np.testing.assert_allclose(y[..., 1::2], zr.imag, atol=1e-13)
    # lengths of pairs are kept; text tokens and the first axis group (position 0 everywhere) are untouched
    np.testing.assert_allclose(np.abs(zr), np.abs(z), rtol=1e-13)
    np.testing.assert_array_equal(y[:, :T], x[:, :T])
    np.testing.assert_array_equal(y[..., :AXES[0]], x[..., :AXES[0]])


def test_rope_single_pair_closed_form():
    # one axis group of two channels: frequency 1, so the pair (1, 0) at x = 1 becomes (cos 1, sin 1)
    x = np.zeros((2, 2))
    x[:, 0] = 1.0
    pos = np.array([[0, 0, 0], [0, 0, 1]])
    y = O.rope(x, pos, (0, 0, 2), 10000.0, 1.0)
    np.testing.assert_allclose(y[0], [1.0, 0.0])
    np.testing.assert_allclose(y[1], [np.cos(1.0), np.sin(1.0)], rtol=1e-15)
    # sign convention: a quarter turn takes (1, 0) to (0, 1): frequency 1 at "position" pi / 2
    y = O.rope(x[:1], np.array([[0.0, 0.0, np.pi / 2]]), (0, 0, 2), 10000.0, 1.0)
    np.testing.assert_allclose(y[0], [0.0, 1.0], atol=1e-15)


@pytest.mark.parametrize("ntk", [1.0, 10.0])
def test_logits_depend_on_the_relative_offset_only(ntk):
    rng = np.random.default_rng(3)
    gh, gw, d = 6, 8, 128
    qv, kv = rng.normal(size=d), rng.normal(size=d)
    pos = O.token_positions(gh, gw, 0)
    q = O.rope(np.tile(qv, (gh * gw, 1)), pos, AXES, 10000.0, ntk)
    k = O.rope(np.tile(kv, (gh * gw, 1)), pos, AXES, 10000.0, ntk)
    s = (q @ k.T).reshape(gh, gw, gh, gw)   # [yq, xq, yk, xk]
    ref = {}
    for yq in range(gh):
        for xq in range(gw):
            for yk in range(gh):
                for xk in range(gw):
                    key = (yk - yq, xk - xq)
                    ref.setdefault(key, s[yq, xq, yk, xk])
                    assert s[yq, xq, yk, xk] == pytest.approx(ref[key], abs=1e-10)
    # and it does depend on it: some pair of offsets gives different logits
    assert abs(ref[(0, 0)] - ref[(1, 0)]) > 1e-3 and abs(ref[(0, 1)] - ref[(1, 0)]) > 1e-6


def test_rope_composes_additively():
    rng = np.random.default_rng(4)
    x = rng.normal(size=(4, 128))
    p1 = np.array([[0, 1, 2], [0, 3, 0], [0, 0, 5], [0, 2, 2]])
    p2 = np.array([[0, 4, 1], [0, 0, 0], [0, 7, 7], [0, 1, 3]])
    a = O.rope(O.rope(x, p1, AXES, 10000.0, 1.0), p2, AXES, 10000.0, 1.0)
    b = O.rope(x, p1 + p2, AXES, 10000.0, 1.0)
    np.testing.assert_allclose(a, b, atol=1e-12)


def test_log_scale_factor_closed_forms():
    assert O.log_scale_factor(4096, 4096) == 1.0
    assert O.log_scale_factor(4096 ** 2, 4096) == pytest.approx(np.sqrt(2.0), rel=1e-15)
    # the paper's step from 1024^2 to 2048^2 pixels (4096 + 512 to 16384 + 512 tokens): a few percent
    f = O.log_scale_factor(16896, 4608)
    assert f == pytest.approx(np.sqrt(np.log(16896.0) / np.log(4608.0))) and 1.07 < f < 1.08


def test_qk_prep_is_norm_then_rope_then_factor():
    rng = np.random.default_rng(5)
    gh, gw, T, d = 4, 6, 2, 64
    axes = (8, 28, 28)
    q = rng.normal(size=(1, 2, T + gh * gw, d))
    k = rng.normal(size=(1, 2, T + gh * gw, d))
    gq, gk = rng.normal(size=d), rng.normal(size=d)
    q2, k2 = O.qk_prep(q, k, gq, gk, gh, gw, T, axes, 10000.0, 1.0, 1e-6, 1.25)
    # pair lengths: rotation keeps them, so they are those of the normalised, gained rows (times the factor)
    nq = O.rms_norm(q, gq, 1e-6)
    nk = O.rms_norm(k, gk, 1e-6)
    np.testing.assert_allclose(np.hypot(q2[..., 0::2], q2[..., 1::2]), 1.25 * np.hypot(nq[..., 0::2], nq[..., 1::2]), rtol=1e-12)
    np.testing.assert_allclose(np.hypot(k2[..., 0::2], k2[..., 1::2]), np.hypot(nk[..., 0::2], nk[..., 1::2]), rtol=1e-12)
    # text rows: normalisation and factor only
    np.testing.assert_allclose(q2[:, :, :T], 1.25 * nq[:, :, :T], rtol=1e-13)
    np.testing.assert_allclose(k2[:, :, :T], nk[:, :, :T], rtol=1e-13)
    # the factor on Q is the factor on every logit
    q1, _ = O.qk_prep(q, k, gq, gk, gh, gw, T, axes, 10000.0, 1.0, 1e-6, 1.0)
    np.testing.assert_allclose(q2 @ np.swapaxes(k2, -1, -2), 1.25 * (q1 @ np.swapaxes(k2, -1, -2)), rtol=1e-12, atol=1e-12)


def test_round_to_bf16():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -7, -0.3, 3.14159, 1e-3, 0.0])
    r = O.round_to_bf16(x)
    # ties go to the even neighbour: 1 + 2^-8 -> 1, 1 + 3 * 2^-8 -> 1 + 2^-6
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 + 2.0 ** -6 and r[3] == 1.0 + 2.0 ** -7 and r[7] == 0.0
    import torch
    t = torch.tensor(x, dtype=torch.float64).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(r, t)
    rng = np.random.default_rng(6)
    y = rng.normal(size=10000)
    np.testing.assert_array_equal(O.round_to_bf16(y), torch.tensor(y).to(torch.bfloat16).to(torch.float64).numpy())
