"""The exchange step of the row-band form (Sec. 3.4) with gloo ranks on the CPU: after the halo exchange every
rank's local K and V are exactly the slice of the whole tensors that its layout names, and the gathered records
arrive in rank order.  No arithmetic of the method runs here (that is the GPU tests' part)."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _whole(B, H, gh, gw, T, d, seed):
    g = torch.Generator().manual_seed(seed)
    N = T + gh * gw
    return torch.randn(B, H, N, d, generator=g), torch.randn(B, H, N, d, generator=g)


def _rank_main(rank, world, port, case, results):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    sys.path.insert(0, ROOT)
    from paper_2412_16112_b200 import band_parallel as bp
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        B, H, gh, gw, T, d, r = case
        k_all, v_all = _whole(B, H, gh, gw, T, d, 11)
        lays = bp.all_layouts(gh, gw, T, r, world)
        me = lays[rank]
        want_k, want_v = bp.slice_local(k_all, me), bp.slice_local(v_all, me)
        # a rank starts with the text tokens and its own band; the halo rows hold garbage
        k, v = torch.full_like(want_k, float("nan")), torch.full_like(want_v, float("nan"))
        own = me.token_range(me.q_row_begin, me.q_row_end)
        for dst, src in ((k, want_k), (v, want_v)):
            dst[:, :, :T] = src[:, :, :T]
            dst[:, :, own] = src[:, :, own]
        bp.exchange_halos(k, v, lays, rank)
        ok = bool(torch.equal(k, want_k) and torch.equal(v, want_v))
        rec = torch.full((B * H, max(T, 1), d + 2), float(rank))
        gathered = bp.gather_records(rec, world)
        ok_gather = all(bool((gathered[p] == float(p)).all()) for p in range(world))
        results[rank] = (ok, ok_gather, me.local_rows, me.halo_lo, me.halo_hi)
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,case", [
    (2, (1, 2, 24, 10, 5, 8, 3.0)),
    (2, (2, 1, 64, 16, 130, 4, 16.0)),    # halo of 15 rows, rounded up to 16 above the second band
    (3, (1, 1, 30, 7, 0, 4, 4.5)),        # middle rank has two neighbours; no text
    (2, (1, 1, 9, 5, 3, 4, 1.0)),         # the window sees its own row only: nothing travels
])
def test_halo_exchange_reproduces_the_slices_of_the_whole_tensors(world, case):
    port = 29500 + ((os.getpid() * 7 + world * 13 + int(case[6] * 10)) % 2000)
    with mp.Manager() as mgr:
        results = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, case, results), nprocs=world, join=True)
        got = dict(results)
    assert set(got) == set(range(world))
    for rank in range(world):
        ok, ok_gather, *_ = got[rank]
        assert ok, f"rank {rank}: local K/V differ from the slice of the whole tensors"
        assert ok_gather


def test_layouts():
    sys.path.insert(0, ROOT)
    from paper_2412_16112_b200 import band_parallel as bp
    lays = bp.all_layouts(512, 512, 512, 16.0, 8)
    assert [(l.y0, l.y1) for l in lays] == [(64 * p, 64 * p + 64) for p in range(8)]
    assert lays[0].halo_lo == 0 and lays[0].halo_hi == 15 and lays[7].halo_hi == 0
    assert all(l.halo_lo == 16 for l in lays[1:])          # 15 rows of reach, rounded up to whole patches
    assert all(l.q_row_begin % 8 == 0 for l in lays)
    assert lays[3].local_rows == 16 + 64 + 15 and lays[3].n_local_tokens == 512 + 95 * 512
    # bands thinner than the reach of the window are refused
    with pytest.raises(ValueError):
        bp.all_layouts(64, 16, 0, 16.0, 8)
    # one rank: the whole grid, no halo
    one = bp.all_layouts(40, 16, 3, 8.0, 1)[0]
    assert (one.y0, one.y1, one.halo_lo, one.halo_hi) == (0, 40, 0, 0)
