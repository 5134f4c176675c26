"""GPU parity of the Q/K preparation (`clear_qk_norm_rope`, through the C ABI) against its fp64 CPU oracle:
element by element on small shapes, on sampled tokens at the full benchmark sizes, and chained with the
attention call."""
import math

import numpy as np
import pytest
import torch

from oracle import clear_oracle as oracle
from oracle import clear_oracle_qk_prep as oracle_prep
from paper_2412_16112_b200 import binding as clear
from paper_2412_16112_b200 import workloads

pytestmark = pytest.mark.gpu


def _bound(ref: np.ndarray, dtype: str) -> np.ndarray:
    """fp32 arithmetic: a few 1e-7 relative per operation, and an angle is good to about 1.2e-7 of its size (at
    most 6e-5 rad at position 511), which moves an element by that times the length of its rotary pair.  For bf16
    outputs add the rounding of the result: at most half a unit in the last of 8 significant bits."""
    a = np.abs(ref)
    pair = np.repeat(np.hypot(ref[..., 0::2], ref[..., 1::2]), 2, axis=-1)
    compute = 1e-4 * pair + 1e-6
    if dtype == "bf16":
        return 2.0 ** -8 * a + compute
    return compute


def _run(q, k, gh, gw, T, axes, gq, gk, theta, ntk, eps, qf, in_place=False):
    dev = torch.device("cuda:0")
    qd, kd = q.to(dev), k.to(dev)
    if in_place:
        qo, ko = qd, kd
    else:
        qo, ko = torch.full_like(qd, float("nan")), torch.full_like(kd, float("nan"))
    clear.clear_qk_norm_rope(qd, kd, qo, ko, gh, gw, T, axes, None if gq is None else gq.to(dev),
                             None if gk is None else gk.to(dev), theta, ntk, eps, qf)
    torch.cuda.synchronize()
    return qo.cpu().to(torch.float64).numpy(), ko.cpu().to(torch.float64).numpy()


@pytest.mark.parametrize("gh,gw,T,d,axes,dtype,gains,ntk,qf", [
    (16, 16, 16, 64, (8, 28, 28), "f32", True, 1.0, 1.0),      # the tiny fp32 configuration's shape
    (13, 19, 7, 128, (16, 56, 56), "bf16", True, 1.0, 1.0),    # the model's split of 128 channels, ragged grid
    (13, 19, 7, 128, (16, 56, 56), "bf16", False, 10.0, 1.07),  # NTK factor 10 and a factor on Q, unit gains
    (8, 16, 0, 128, (0, 64, 64), "f32", True, 10.0, 0.5),      # no text, no position-free group
    (1, 70, 2, 64, (2, 2, 60), "bf16", True, 1.0, 1.0),        # single-row grid, two-channel groups
    (33, 9, 130, 128, (128, 0, 0), "f32", False, 1.0, 1.0),    # no rotation at all: normalisation only
    (24, 40, 5, 64, (0, 0, 64), "bf16", True, 2.0, 1.0),       # x axis only
])
def test_prep_matches_the_oracle_everywhere(gh, gw, T, d, axes, dtype, gains, ntk, qf):
    B, H = 2, 3
    q, k, _ = workloads.make_custom(B, H, gh, gw, T, d, dtype=dtype, qk_norm=False, seed=gh * 17 + gw)
    q = q * 3.0   # rows far from unit mean square
    gq, gk = workloads.make_gains(d, seed=d) if gains else (None, None)
    want_q, want_k = oracle_prep.qk_prep(q.to(torch.float64).numpy(), k.to(torch.float64).numpy(),
                                         None if gq is None else gq.numpy(), None if gk is None else gk.numpy(),
                                         gh, gw, T, axes, 10000.0, ntk, 1e-6, qf)
    for in_place in (False, True):
        got_q, got_k = _run(q, k, gh, gw, T, axes, gq, gk, 10000.0, ntk, 1e-6, qf, in_place)
        for name, got, ref in (("q", got_q, want_q), ("k", got_k, want_k)):
            assert np.isfinite(got).all(), name
            excess = np.abs(got - ref) - _bound(ref, dtype)
            assert excess.max() <= 0, (name, in_place, float(np.abs(got - ref).max()))


@pytest.mark.parametrize("name", ["c2_2048px_r16", "c4_8k_r16"])
def test_prep_at_full_size_on_sampled_tokens(name):
    """The benchmark shapes (24 heads of 128 channels, 512 text tokens): every (batch, head) row of 600 sampled
    tokens -- first and last text token, the grid's corners and edges, positions up to 511 on both axes."""
    w = workloads.WORKLOADS[name]
    N, d, H = w.n_tokens, w.head_dim, w.H
    axes = (16, 56, 56)
    dev = torch.device("cuda:0")
    gen = torch.Generator(device="cuda:0").manual_seed(2024)
    # raw projections drawn on the device (the oracle reads back exactly these bits); bounded host memory
    q = torch.randn(1, H, N, d, generator=gen, device=dev, dtype=torch.float32).mul_(2.0).to(torch.bfloat16)
    k = torch.randn(1, H, N, d, generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    gq, gk = workloads.make_gains(d, seed=3)
    qo, ko = torch.empty_like(q), torch.empty_like(k)
    ntk, qf = 10.0, clear.clear_log_scale_factor(N, 4608)
    clear.clear_qk_norm_rope(q, k, qo, ko, w.grid_h, w.grid_w, w.n_text, axes, gq.to(dev), gk.to(dev), 10000.0, ntk, 1e-6, qf)
    torch.cuda.synchronize()
    rng = np.random.default_rng(5)
    gh, gw, T = w.grid_h, w.grid_w, w.n_text
    fixed = [0, T - 1, T, T + gw - 1, T + (gh - 1) * gw, N - 1, T + gw, T + 2 * gw - 1]
    idx = np.unique(np.concatenate([np.array(fixed), rng.integers(0, N, size=600 - len(fixed))]))
    pos = oracle_prep.token_positions(gh, gw, T)[idx]
    ti = torch.from_numpy(idx).to(dev)
    for src, dst, gain, factor, label in ((q, qo, gq, qf, "q"), (k, ko, gk, 1.0, "k")):
        x = src[:, :, ti].cpu().to(torch.float64).numpy()
        ref = oracle_prep.rope(oracle_prep.rms_norm(x, gain.numpy(), 1e-6), pos, axes, 10000.0, ntk) * factor
        got = dst[:, :, ti].cpu().to(torch.float64).numpy()
        excess = np.abs(got - ref) - _bound(ref, "bf16")
        assert excess.max() <= 0, (label, float(np.abs(got - ref).max()))
    # nothing outside the tensors' own values: every output element finite, rows of K of the right length
    assert torch.isfinite(qo).all() and torch.isfinite(ko).all()
    row_ms = ko[0, 0].to(torch.float32).pow(2).mean(dim=-1)
    assert 0.7 < float(row_ms.min()) and float(row_ms.max()) < 1.5   # gains near one: mean square near one


def test_log_scale_factor_matches_the_oracle():
    for n, n_train in ((16896, 4608), (66048, 4608), (262656, 4608), (4608, 4608), (4096 ** 2, 4096)):
        assert clear.clear_log_scale_factor(n, n_train) == pytest.approx(oracle_prep.log_scale_factor(n, n_train), rel=1e-6)


def test_prepared_q_and_k_through_the_attention_call():
    """Raw projections -> preparation -> attention, against the same chain of oracles (the oracle rounds the
    prepared Q and K to bf16 as the attention call receives them)."""
    gh, gw, T, d, r = 20, 24, 40, 128, 6.0
    axes = (16, 56, 56)
    q, k, v = workloads.make_custom(1, 2, gh, gw, T, d, dtype="bf16", qk_norm=False, seed=99)
    gq, gk = workloads.make_gains(d, seed=1)
    qf = oracle_prep.log_scale_factor(16896, 4608)
    scale = 1 / math.sqrt(d)
    pq, pk = oracle_prep.qk_prep(q.to(torch.float64).numpy(), k.to(torch.float64).numpy(), gq.numpy(), gk.numpy(),
                                 gh, gw, T, axes, 10000.0, 10.0, 1e-6, qf)
    pq, pk = oracle_prep.round_to_bf16(pq), oracle_prep.round_to_bf16(pk)
    want = oracle.attn(torch.from_numpy(pq), torch.from_numpy(pk), v.to(torch.float64), gh, gw, T, r, scale)
    dev = torch.device("cuda:0")
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    clear.clear_qk_norm_rope(qd, kd, qd, kd, gh, gw, T, axes, gq.to(dev), gk.to(dev), 10000.0, 10.0, 1e-6, qf)
    out = torch.full_like(qd, float("nan"))
    clear.clear_attn_fwd(qd, kd, vd, out, gh, gw, T, r, scale)
    torch.cuda.synchronize()
    err = np.abs(out.cpu().to(torch.float64).numpy() - np.asarray(want))
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (float(err.max()), float(err.mean()))
