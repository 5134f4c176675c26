"""Host-side checks of the CUDA library that need no GPU: exported symbols, status codes and the
tile schedule (built with clear_plan_create_host) against the oracle's mask."""
import ctypes
import math
import os
import re

import numpy as np
import pytest

from oracle import clear_oracle as oracle
from paper_2412_16112_b200 import binding as clear

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(inc, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(clear_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol():
    lib = clear.load()
    names = declared_functions()
    assert len(names) >= 13
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"
    assert set(clear.EXPORTS) <= set(names)


def test_status_strings():
    assert clear.status_string(0) == "ok"
    seen = {clear.status_string(s) for s in range(-7, 1)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert clear.status_string(-99) == "unknown status"


@pytest.mark.parametrize("kwargs,status", [
    (dict(B=0), clear.ERR_INVALID_ARG), (dict(H=-1), clear.ERR_INVALID_ARG),
    (dict(grid_h=0), clear.ERR_INVALID_ARG), (dict(n_text=-1), clear.ERR_INVALID_ARG),
    (dict(radius=0.0), clear.ERR_INVALID_ARG), (dict(radius=float("nan")), clear.ERR_INVALID_ARG),
    (dict(radius=float("inf")), clear.ERR_INVALID_ARG), (dict(dtype=5), clear.ERR_INVALID_ARG),
    (dict(head_dim=512), clear.ERR_UNSUPPORTED), (dict(head_dim=20), clear.ERR_UNSUPPORTED),
    (dict(head_dim=96, kernel=clear.KERNEL_TCGEN05), clear.ERR_UNSUPPORTED),
    (dict(dtype=clear.F32, kernel=clear.KERNEL_TCGEN05), clear.ERR_UNSUPPORTED),
])
def test_plan_rejects_bad_shapes(kwargs, status):
    base = dict(B=1, H=2, grid_h=16, grid_w=16, n_text=16, head_dim=64, radius=4.0, dtype=clear.BF16,
                kernel=clear.KERNEL_AUTO)
    base.update(kwargs)
    with pytest.raises(clear.ClearError) as e:
        clear.Plan(host_only=True, **base)
    assert e.value.status == status


def test_host_plan_cannot_run_and_null_arguments_are_rejected():
    lib = clear.load()
    p = clear.Plan(1, 1, 8, 16, 0, 64, 2.0, host_only=True)
    buf = (ctypes.c_char * 64)()
    addr = (ctypes.addressof(buf) + 15) & ~15
    assert lib.clear_attn_fwd_planned(p.handle, addr, addr, addr, addr, 1.0, None) == clear.ERR_PLAN_MISMATCH
    assert lib.clear_attn_fwd_planned(p.handle, None, addr, addr, addr, 1.0, None) == clear.ERR_INVALID_ARG
    assert lib.clear_attn_fwd_planned(p.handle, addr + 4, addr, addr, addr, 1.0, None) == clear.ERR_MISALIGNED
    assert lib.clear_attn_fwd_planned(p.handle, addr, addr, addr, addr, float("nan"), None) == clear.ERR_INVALID_ARG
    assert lib.clear_plan_info(None, None) == clear.ERR_INVALID_ARG
    assert lib.clear_plan_destroy(None) == clear.OK
    assert lib.clear_attn_fwd(None, None, None, None, 1, 1, 4, 4, 0, 64, 1.0, 1.0, None) == clear.ERR_INVALID_ARG
    assert lib.clear_attn_fwd(addr, addr, addr, addr, 1, 1, 4, 4, 0, 64, -1.0, 1.0, None) == clear.ERR_INVALID_ARG


def test_kernel_selection():
    assert clear.Plan(1, 1, 16, 16, 16, 128, 4.0, host_only=True).info().kernel == clear.KERNEL_TCGEN05
    assert clear.Plan(1, 1, 16, 16, 16, 64, 4.0, host_only=True).info().kernel == clear.KERNEL_TCGEN05
    assert clear.Plan(1, 1, 16, 16, 16, 96, 4.0, host_only=True).info().kernel == clear.KERNEL_SIMT
    assert clear.Plan(1, 1, 16, 16, 16, 64, 4.0, dtype=clear.F32, host_only=True).info().kernel == clear.KERNEL_SIMT


SHAPES = [(16, 16, 16, 4.0), (13, 19, 7, 4.0), (24, 40, 130, 8.0), (9, 33, 0, 5.5), (40, 24, 256, 16.0),
          (8, 16, 5, 1.0), (20, 50, 3, 100.0), (1, 70, 2, 3.0), (33, 1, 0, 2.5)]


@pytest.mark.parametrize("gh,gw,T,r", SHAPES)
def test_geometry_matches_the_oracle_mask(gh, gw, T, r):
    total, counts = oracle.mask_counts(gh, gw, T, r)
    for kernel in (clear.KERNEL_SIMT, clear.KERNEL_TCGEN05):
        p = clear.Plan(2, 3, gh, gw, T, 64, r, kernel=kernel, host_only=True)
        info = p.info()
        assert info.sum_mask == total
        assert info.flops == 4.0 * total * 64 * 3 * 2
        _, _, hw = p.tables()
        thr = info.radius_sq_ceil
        assert thr == min(math.ceil(r * r), (gh - 1) ** 2 + (gw - 1) ** 2 + 1)
        # half_width[dy] read off the oracle's mask row of a query in the grid's first column
        for dy, m in enumerate(hw):
            row = oracle.mask_row(T, gh, gw, T, r)[T:].reshape(gh, gw)
            assert int(row[dy].sum()) - 1 == m
        if len(hw) < gh:
            assert oracle.mask_row(T, gh, gw, T, r)[T:].reshape(gh, gw)[len(hw)].sum() == 0


@pytest.mark.parametrize("gh,gw,T,r", SHAPES)
def test_tile_schedule_covers_each_allowed_pair_exactly_once(gh, gw, T, r):
    p = clear.Plan(1, 1, gh, gw, T, 128, r, kernel=clear.KERNEL_TCGEN05, host_only=True)
    info = p.info()
    items, tiles, _ = p.tables()
    N = T + gh * gw
    assert info.tile_h * info.tile_w == 128
    th, tw = info.tile_h, info.tile_w
    assert [it.tile_count for it in items] == sorted((it.tile_count for it in items), reverse=True)
    assert info.executed_pairs == sum(it.tile_count for it in items) * 128 * 128
    assert info.max_item_tiles == max(it.tile_count for it in items)

    seen_queries = np.zeros(N, dtype=np.int64)
    text_cover = {}
    slots = set()
    for it in items:
        assert it.tile_count >= 1
        its = tiles[it.tile_begin: it.tile_begin + it.tile_count]
        if it.kind == 1:
            # text-query tile: linear key tiles only, together a contiguous token range
            assert it.qx % 128 == 0 and it.n_rows == min(128, T - it.qx)
            toks = []
            for t in its:
                assert t.flags & clear.TILE_LINEAR
                assert t.n_valid == min(128, N - t.x) and bool(t.flags & clear.TILE_MASKED) == (t.n_valid < 128)
                toks += list(range(t.x, t.x + t.n_valid))
            assert toks == list(range(toks[0], toks[-1] + 1))
            text_cover.setdefault(it.qx, []).extend(toks)
            if info.n_text_splits > 1:
                assert it.partial_slot >= 0 and it.partial_slot not in slots
                assert it.partial_slot // info.n_text_splits == it.qx // 128
                slots.add(it.partial_slot)
            else:
                assert it.partial_slot == -1
            continue
        # image-query patch
        assert it.partial_slot == -1 and it.qx % tw == 0 and it.qy % th == 0
        qs = [(y, x) for y in range(it.qy, min(it.qy + th, gh)) for x in range(it.qx, min(it.qx + tw, gw))]
        assert it.n_rows == len(qs)
        cover = np.zeros(N, dtype=np.int64)
        unmasked = np.zeros(N, dtype=bool)
        for t in its:
            if t.flags & clear.TILE_LINEAR:
                assert t.x + t.n_valid <= T          # image queries reach text keys only through these
                idx = np.arange(t.x, t.x + t.n_valid)
                assert bool(t.flags & clear.TILE_MASKED) == (t.n_valid < 128)
            else:
                ys, xs = np.meshgrid(np.arange(t.y, t.y + th), np.arange(t.x, t.x + tw), indexing="ij")
                ok = (ys >= 0) & (ys < gh) & (xs >= 0) & (xs < gw)
                idx = (T + ys * gw + xs)[ok]
                if not (t.flags & clear.TILE_MASKED):
                    assert ok.all()
                    unmasked[idx] = True
            cover[idx] += 1
        assert cover.max() <= 1
        for (y, x) in qs:
            i = T + y * gw + x
            seen_queries[i] += 1
            row = oracle.mask_row(i, gh, gw, T, r).astype(bool)
            assert not (row & (cover == 0)).any(), "an allowed key is in no tile of the item"
            assert row[unmasked].all(), "a tile flagged mask-free holds a disallowed pair"
        # no useless tile: every image tile holds at least one allowed pair
        for t in its:
            if not (t.flags & clear.TILE_LINEAR):
                hit = False
                for (y, x) in qs:
                    row = oracle.mask_row(T + y * gw + x, gh, gw, T, r)[T:].reshape(gh, gw)
                    sub = row[max(t.y, 0): t.y + th, max(t.x, 0): t.x + tw]
                    hit = hit or bool(sub.any())
                assert hit
    assert np.all(seen_queries[T:] == 1)
    for q0 in range(0, T, 128):
        assert sorted(text_cover[q0]) == list(range(N))
    if info.n_text_splits > 1:
        assert len(slots) == math.ceil(T / 128) * info.n_text_splits
        assert info.workspace_bytes == len(slots) * 128 * (128 + 2) * 4


def test_text_rows_are_split_for_long_sequences():
    p = clear.Plan(1, 24, 512, 512, 512, 128, 16.0, host_only=True)
    info = p.info()
    assert info.kernel == clear.KERNEL_TCGEN05
    assert info.sum_mask == 471125568                   # matches the 5.79 TFLOPS cell of the paper
    assert info.n_text_splits > 1
    items, tiles, _ = p.tables()
    longest = max(it.tile_count for it in items)
    assert longest <= 64
    interior = [it for it in items if it.kind == 0 and it.tile_count == 19]
    assert len(interior) > 1500                          # 15 key patches + 4 text tiles away from borders
    g = info.sum_mask / info.executed_pairs
    assert 0.55 < g < 0.70
