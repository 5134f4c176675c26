"""GPU parity of the backward pass (`clear_attn_bwd_f32`, through the C ABI) against its fp64 CPU oracle,
element by element on small shapes."""
import math

import numpy as np
import pytest
import torch

from oracle import clear_oracle_bwd as oracle_bwd
from paper_2412_16112_b200 import binding as clear
from paper_2412_16112_b200 import workloads

pytestmark = pytest.mark.gpu

# fp32 arithmetic with fp32 atomic sums of up to a few hundred terms of order one
BWD_ATOL = 1e-4


@pytest.mark.parametrize("gh,gw,T,r,d", [
    (16, 16, 16, 4.0, 64),      # the tiny fp32 configuration
    (13, 19, 7, 4.0, 128),      # ragged on both axes
    (8, 16, 0, 1.0, 128),       # no text, self only: dv = d_out, dq = dk = 0
    (9, 33, 0, 5.5, 40),        # head size that is no multiple of 32, non-integer radius
    (20, 50, 3, 100.0, 64),     # radius beyond the diagonal: full attention
    (1, 70, 2, 3.0, 96),        # single-row grid
    (24, 40, 130, 8.0, 64),
])
def test_backward_matches_the_oracle_everywhere(gh, gw, T, r, d):
    q, k, v = workloads.make_custom(1, 2, gh, gw, T, d, dtype="f32", qk_norm=False, seed=gh * 31 + gw)
    g = torch.Generator(device="cpu").manual_seed(gh + gw)
    d_out = torch.randn(q.shape, generator=g, dtype=torch.float32)
    scale = 1 / math.sqrt(d)
    want = oracle_bwd.attn_bwd(q, k, v, d_out, gh, gw, T, r, scale)
    dev = torch.device("cuda:0")
    qd, kd, vd, gd = (t.to(dev) for t in (q, k, v, d_out))
    dq, dk, dv = (torch.full_like(qd, float("nan")) for _ in range(3))
    for _ in range(2):      # the second call finds dk, dv dirty and must start them at zero again
        clear.clear_attn_bwd_f32(qd, kd, vd, gd, dq, dk, dv, gh, gw, T, r, scale)
    torch.cuda.synchronize()
    for name, got, ref in (("dq", dq, want[0]), ("dk", dk, want[1]), ("dv", dv, want[2])):
        err = np.abs(got.cpu().double().numpy() - ref)
        assert np.isfinite(err).all(), f"{name}: non-finite"
        assert err.max() <= BWD_ATOL, f"{name}: max {err.max():.3e}"
    clear.clear_cache_clear()


def test_backward_argument_errors():
    dev = torch.device("cuda:0")
    x = torch.zeros(1, 1, 272, 64, device=dev)
    p = x.data_ptr()
    lib = clear.load()
    assert lib.clear_attn_bwd_f32(p, p, p, p, p, p, p, 1, 1, 16, 16, 16, 64, 0.0, 0.125, None) == clear.ERR_INVALID_ARG
    assert lib.clear_attn_bwd_f32(p, p, p, None, p, p, p, 1, 1, 16, 16, 16, 64, 4.0, 0.125, None) == clear.ERR_INVALID_ARG
    assert lib.clear_attn_bwd_f32(p, p, p, p, p, p + 4, p, 1, 1, 16, 16, 16, 64, 4.0, 0.125, None) == clear.ERR_MISALIGNED
    assert lib.clear_attn_bwd_f32(p, p, p, p, p, p, p, 1, 1, 16, 16, 16, 64, 4.0, float("nan"), None) == clear.ERR_INVALID_ARG


def test_backward_repeats_bit_for_bit_and_from_two_streams():
    """One writer per output element and a fixed order of summation: the same bits on every call, also when two
    streams call for the same shape at once (the library orders them: they share the row statistics)."""
    gh, gw, T, r, d = 24, 40, 130, 8.0, 64
    q, k, v = workloads.make_custom(1, 3, gh, gw, T, d, dtype="f32", qk_norm=False, seed=5)
    g = torch.Generator(device="cpu").manual_seed(6)
    d_out = torch.randn(q.shape, generator=g, dtype=torch.float32)
    scale = 1 / math.sqrt(d)
    dev = torch.device("cuda:0")
    qd, kd, vd, gd = (t.to(dev) for t in (q, k, v, d_out))
    first = [torch.full_like(qd, float("nan")) for _ in range(3)]
    clear.clear_attn_bwd_f32(qd, kd, vd, gd, *first, gh, gw, T, r, scale)
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    # the second stream gets other inputs, so a mix-up of the shared statistics would show
    q2 = (qd * 1.5).contiguous()
    outs = [[torch.full_like(qd, float("nan")) for _ in range(3)] for _ in range(2)]
    for rep in range(3):
        for s, (qq, o) in zip(streams, ((qd, outs[0]), (q2, outs[1]))):
            with torch.cuda.stream(s):
                clear.clear_attn_bwd_f32(qq, kd, vd, gd, *o, gh, gw, T, r, scale, stream=s)
    torch.cuda.synchronize()
    for a, b in zip(first, outs[0]):
        assert torch.equal(a, b)
    want = oracle_bwd.attn_bwd(q * 1.5, k, v, d_out, gh, gw, T, r, scale)
    for got, ref in zip(outs[1], want):
        assert np.abs(got.cpu().double().numpy() - ref).max() <= BWD_ATOL
    clear.clear_cache_clear()


@pytest.mark.parametrize("gh,gw,T,r,d", [(16, 24, 20, 4.0, 128), (13, 19, 7, 2.5, 64), (24, 40, 130, 8.0, 128)])
def test_bf16_backward_matches_the_oracle(gh, gw, T, r, d):
    """bf16 tensors in and out, fp32 arithmetic: the error is the rounding of each gradient to bf16 (half a unit
    in the last of 8 significant bits) on top of the fp32 kernel's."""
    q, k, v = workloads.make_custom(1, 2, gh, gw, T, d, dtype="bf16", seed=gh + gw)
    g = torch.Generator(device="cpu").manual_seed(gh * gw)
    d_out = torch.randn(q.shape, generator=g, dtype=torch.float32).to(torch.bfloat16)
    scale = 1 / math.sqrt(d)
    want = oracle_bwd.attn_bwd(q, k, v, d_out, gh, gw, T, r, scale)
    dev = torch.device("cuda:0")
    qd, kd, vd, gd = (t.to(dev) for t in (q, k, v, d_out))
    dq, dk, dv = (torch.full_like(qd, float("nan")) for _ in range(3))
    clear.clear_attn_bwd_bf16(qd, kd, vd, gd, dq, dk, dv, gh, gw, T, r, scale)
    torch.cuda.synchronize()
    for name, got, ref in (("dq", dq, want[0]), ("dk", dk, want[1]), ("dv", dv, want[2])):
        err = np.abs(got.cpu().double().numpy() - ref)
        assert np.isfinite(err).all(), f"{name}: non-finite"
        assert (err <= 2.0 ** -8 * np.abs(ref) + BWD_ATOL).all(), f"{name}: max {err.max():.3e}"
    clear.clear_cache_clear()


# ----------------------------------------------------------------------------------------------
# tensor-core backward (bf16)
# ----------------------------------------------------------------------------------------------
def _tc_bound(ref):
    """P and dS enter the MMAs rounded to bf16 and every gradient is stored as bf16: errors of a few 1e-3 of the
    tensor's largest gradient were observed; the bound is 1e-2 of it."""
    return 1e-2 * np.abs(ref).max()


@pytest.mark.parametrize("gh,gw,T,r,d", [
    (16, 16, 16, 4.0, 64),       # the tiny configuration's shape
    (13, 19, 7, 2.5, 128),       # ragged patches, non-integer radius
    (24, 40, 130, 8.0, 128),     # two text tiles, the second with two rows
    (20, 50, 3, 100.0, 64),      # radius beyond the diagonal: full attention
    (33, 35, 0, 5.5, 128),       # no text
    (8, 16, 300, 3.0, 128),      # more text than image
    (1, 70, 2, 3.0, 64),         # single-row grid
])
def test_tensor_core_backward_matches_the_oracle(gh, gw, T, r, d):
    q, k, v = workloads.make_custom(1, 2, gh, gw, T, d, dtype="bf16", seed=gh + gw)
    g = torch.Generator(device="cpu").manual_seed(gh * gw)
    d_out = torch.randn(q.shape, generator=g, dtype=torch.float32).to(torch.bfloat16)
    scale = 1 / math.sqrt(d)
    want = oracle_bwd.attn_bwd(q, k, v, d_out, gh, gw, T, r, scale)
    dev = torch.device("cuda:0")
    qd, kd, vd, gd = (t.to(dev) for t in (q, k, v, d_out))
    outs = [torch.full_like(qd, float("nan")) for _ in range(3)]
    again = [torch.full_like(qd, float("nan")) for _ in range(3)]
    clear.clear_attn_bwd_bf16_tc(qd, kd, vd, gd, *outs, gh, gw, T, r, scale)
    clear.clear_attn_bwd_bf16_tc(qd, kd, vd, gd, *again, gh, gw, T, r, scale)
    torch.cuda.synchronize()
    clear.clear_cache_check()
    for name, got, rep, ref in zip(("dq", "dk", "dv"), outs, again, want):
        gn = got.cpu().double().numpy()
        assert np.isfinite(gn).all(), f"{name}: non-finite"
        assert np.abs(gn - ref).max() <= _tc_bound(ref), f"{name}: max {np.abs(gn - ref).max():.3e}"
        assert torch.equal(got, rep), f"{name}: not repeatable"
    clear.clear_cache_clear()


@pytest.mark.parametrize("name,heads", [("c1_1024px_r8", 2), ("c2_2048px_r16", 1)])
def test_tensor_core_backward_at_workload_sizes(name, heads):
    """Whole tensors against the oracle at the 1024px and 2048px shapes (fewer heads: the oracle is a CPU loop)."""
    w = workloads.WORKLOADS[name]
    q, k, v = workloads.make_inputs(w, heads=heads)
    g = torch.Generator(device="cpu").manual_seed(3)
    d_out = torch.randn(q.shape, generator=g, dtype=torch.float32).to(torch.bfloat16)
    want = oracle_bwd.attn_bwd(q, k, v, d_out, w.grid_h, w.grid_w, w.n_text, w.radius, w.scale)
    dev = torch.device("cuda:0")
    qd, kd, vd, gd = (t.to(dev) for t in (q, k, v, d_out))
    outs = [torch.full_like(qd, float("nan")) for _ in range(3)]
    clear.clear_attn_bwd_bf16_tc(qd, kd, vd, gd, *outs, w.grid_h, w.grid_w, w.n_text, w.radius, w.scale)
    torch.cuda.synchronize()
    clear.clear_cache_check()
    for nm, got, ref in zip(("dq", "dk", "dv"), outs, want):
        gn = got.cpu().double().numpy()
        assert np.isfinite(gn).all(), f"{nm}: non-finite"
        err = np.abs(gn - ref)
        assert err.max() <= _tc_bound(ref), f"{nm}: max {err.max():.3e} of {np.abs(ref).max():.3e}"
        assert err.mean() <= 1e-3 * np.abs(ref).max(), f"{nm}: mean {err.mean():.3e}"
    clear.clear_cache_clear()


def test_tensor_core_backward_argument_errors():
    dev = torch.device("cuda:0")
    x = torch.zeros(1, 1, 272, 64, device=dev, dtype=torch.bfloat16)
    p = x.data_ptr()
    lib = clear.load()
    assert lib.clear_attn_bwd_bf16_tc(p, p, p, p, p, p, p, 1, 1, 16, 16, 16, 96, 4.0, 0.125, None) == clear.ERR_UNSUPPORTED
    assert lib.clear_attn_bwd_bf16_tc(p, p, p, p, p, p, p, 1, 1, 16, 16, 16, 64, 4.0, 0.0, None) == clear.ERR_UNSUPPORTED
    assert lib.clear_attn_bwd_bf16_tc(p, p, p, p, p, p, p, 1, 1, 16, 16, 16, 64, 4.0, float("nan"), None) == clear.ERR_INVALID_ARG
    assert lib.clear_attn_bwd_bf16_tc(p, p, p, None, p, p, p, 1, 1, 16, 16, 16, 64, 4.0, 0.125, None) == clear.ERR_INVALID_ARG
    assert lib.clear_attn_bwd_bf16_tc(p, p, p, p, p, p + 4, p, 1, 1, 16, 16, 16, 64, 4.0, 0.125, None) == clear.ERR_MISALIGNED
