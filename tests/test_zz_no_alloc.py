"""The no-allocation entry point, `clear_attn_fwd_static`, against the planned entry points and the oracle.

Some callers cannot allocate device memory where attention runs: a host that works inside a fixed,
pre-partitioned memory budget, a plug-in whose embedding framework owns every device byte, a process whose
caching allocator has already taken all free memory (a cudaMalloc there fails or stalls other streams).
For them the library keeps its schedule tables and split-KV scratch in one fixed-size array inside the
library image.  This file is collected last so that a run stopping at the first failure has already run
every other test; it must also pass alone in a fresh process.
"""
import math

import numpy as np
import pytest
import torch

from oracle import clear_oracle as oracle
from paper_2412_16112_b200 import binding as clear
from paper_2412_16112_b200 import workloads

pytestmark = pytest.mark.gpu

BF16_MAX, BF16_MEAN = 2e-2, 2e-3     # the tolerance of the parity tests


def _close(a, b):
    err = (a.float() - b.float()).abs()
    return bool(torch.isfinite(err).all()) and float(err.max()) <= BF16_MAX and float(err.mean()) <= BF16_MEAN


def test_static_entry_point_matches_the_planned_one_twice_in_a_row():
    assert torch.cuda.is_available()
    dev = torch.device("cuda:0")
    # text-query rows are split over key ranges here, so the scratch in the static array is in use
    gh, gw, T, r, d = 96, 96, 200, 6.0, 128
    assert clear.Plan(1, 2, gh, gw, T, d, r, host_only=True).info().n_text_splits > 1
    q, k, v = workloads.make_custom(1, 2, gh, gw, T, d, seed=123)
    scale = 1 / math.sqrt(d)
    qd, kd, vd = (t.to(dev) for t in (q, k, v))
    want = torch.full_like(qd, float("nan"))
    clear.clear_attn_fwd(qd, kd, vd, want, gh, gw, T, r, scale)
    # the same kernel through a plan of its own (cudaMalloc'ed tables and scratch): equal bit for bit
    same = torch.full_like(qd, float("nan"))
    plan = clear.Plan(1, 2, gh, gw, T, d, r, kernel=clear.KERNEL_TCGEN05)
    plan.forward(qd, kd, vd, same, scale)
    plan.check()
    torch.cuda.synchronize()

    got = torch.full_like(qd, float("nan"))
    clear.clear_attn_fwd_static(qd, kd, vd, got, gh, gw, T, r, scale)   # first call: set-up + table upload
    torch.cuda.synchronize()
    assert _close(got, want) and torch.equal(got, same)
    # the second call reuses tables and dirty scratch, and the device's free memory does not move across it
    got.fill_(float("nan"))
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    clear.clear_attn_fwd_static(qd, kd, vd, got, gh, gw, T, r, scale)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "the no-allocation entry point changed the free device memory"
    assert _close(got, want) and torch.equal(got, same)
    # and against the CPU oracle on sampled rows
    rows = np.array([(0, h, i) for h in (0, 1) for i in (0, T - 1, T, T + 97, T + gh * gw // 2, T + gh * gw - 1)], dtype=np.int64)
    ref = oracle.attn_rows(q, k, v, gh, gw, T, r, scale, rows)
    err = np.abs(got.cpu()[rows[:, 0], rows[:, 1], rows[:, 2]].double().numpy() - ref)
    assert err.max() <= BF16_MAX and err.mean() <= BF16_MEAN

    # another shape in between forces a table re-upload into the same array, then back again
    gh2, gw2, T2, r2 = 24, 40, 130, 8.0
    q2, k2, v2 = (t.to(dev) for t in workloads.make_custom(1, 2, gh2, gw2, T2, d, seed=124))
    want2 = torch.full_like(q2, float("nan"))
    got2 = torch.full_like(q2, float("nan"))
    clear.clear_attn_fwd(q2, k2, v2, want2, gh2, gw2, T2, r2, scale)
    clear.clear_attn_fwd_static(q2, k2, v2, got2, gh2, gw2, T2, r2, scale)
    got = torch.full_like(qd, float("nan"))
    clear.clear_attn_fwd_static(qd, kd, vd, got, gh, gw, T, r, scale)
    torch.cuda.synchronize()
    assert _close(got2, want2)
    assert _close(got, want) and torch.equal(got, same)
    plan.destroy()
    clear.clear_cache_clear()


def test_static_entry_point_rejects_shapes_beyond_its_capacity():
    dev = torch.device("cuda:0")
    x = torch.zeros(4096, dtype=torch.bfloat16, device=dev)
    p = x.data_ptr()
    lib = clear.load()
    # 4096px FLUX shape: 57.5 MB of split-KV partial results > 32 MiB; rejected before any launch
    assert lib.clear_attn_fwd_static(p, p, p, p, 1, 24, 256, 256, 512, 128, 16.0, 0.0884, None) == clear.ERR_TOO_LARGE
    assert lib.clear_attn_fwd_static(p, p, p, p, 1, 24, 256, 256, 512, 96, 16.0, 0.0884, None) == clear.ERR_UNSUPPORTED
    assert lib.clear_attn_fwd_static(p, p, p, p, 1, 24, 16, 16, 16, 128, 4.0, -1.0, None) == clear.ERR_UNSUPPORTED
    assert lib.clear_attn_fwd_static(None, p, p, p, 1, 1, 16, 16, 16, 128, 4.0, 1.0, None) == clear.ERR_INVALID_ARG
    assert "capacity" in clear.status_string(clear.ERR_TOO_LARGE)
