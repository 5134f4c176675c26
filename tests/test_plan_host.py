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
    (dict(head_dim=96, kernel=clear.KERNEL_TCGEN05_WS), clear.ERR_UNSUPPORTED),
    (dict(dtype=clear.F32, kernel=clear.KERNEL_TCGEN05_WS), clear.ERR_UNSUPPORTED),
    (dict(kernel=4), clear.ERR_INVALID_ARG),
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
    assert clear.Plan(1, 1, 16, 16, 16, 128, 4.0, host_only=True).info().kernel == clear.KERNEL_TCGEN05_WS
    assert clear.Plan(1, 1, 16, 16, 16, 64, 4.0, host_only=True).info().kernel == clear.KERNEL_TCGEN05_WS
    assert clear.Plan(1, 1, 16, 16, 16, 64, 4.0, kernel=clear.KERNEL_TCGEN05,
                      host_only=True).info().kernel == clear.KERNEL_TCGEN05
    assert clear.Plan(1, 1, 16, 16, 16, 96, 4.0, host_only=True).info().kernel == clear.KERNEL_SIMT
    assert clear.Plan(1, 1, 16, 16, 16, 64, 4.0, dtype=clear.F32, host_only=True).info().kernel == clear.KERNEL_SIMT


SHAPES = [(16, 16, 16, 4.0), (13, 19, 7, 4.0), (24, 40, 130, 8.0), (9, 33, 0, 5.5), (40, 24, 256, 16.0),
          (8, 16, 5, 1.0), (20, 50, 3, 100.0), (1, 70, 2, 3.0), (33, 1, 0, 2.5)]


@pytest.mark.parametrize("gh,gw,T,r", SHAPES)
def test_geometry_matches_the_oracle_mask(gh, gw, T, r):
    total, counts = oracle.mask_counts(gh, gw, T, r)
    for kernel in (clear.KERNEL_SIMT, clear.KERNEL_TCGEN05, clear.KERNEL_TCGEN05_WS):
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


def key_tokens(x, y, linear, n_valid, gh, gw, T, th, tw):
    """Token indices a key tile holds (existing keys only), and whether all 128 exist."""
    if linear:
        return np.arange(x, x + n_valid), n_valid == 128
    ys, xs = np.meshgrid(np.arange(y, y + th), np.arange(x, x + tw), indexing="ij")
    ok = (ys >= 0) & (ys < gh) & (xs >= 0) & (xs < gw)
    return (T + ys * gw + xs)[ok], bool(ok.all())


def check_mask_table(p, items, steps, gh, gw, T, r, th, tw):
    """Every masked 2-D tile's table entry, restricted to the keys on the grid, is the oracle's mask;
    the clip flag is set exactly when part of the key patch is off the grid."""
    table = p.mask_table()
    for it in items:
        if it.kind != 0:
            continue
        for st in steps[it.step_begin: it.step_begin + it.step_count]:
            if st.flags & clear.STEP_LINEAR:
                continue
            for side in range(it.n_sides):
                if not st.flags & (clear.STEP_USE1 if side else clear.STEP_USE0):
                    continue
                x, y, e = (st.x1, st.y1, st.n_valid1) if side else (st.x0, st.y0, st.n_valid0)
                qy = it.qy1 if side else it.qy0
                ys, xs = np.meshgrid(np.arange(y, y + th), np.arange(x, x + tw), indexing="ij")
                on_grid = ((ys >= 0) & (ys < gh) & (xs >= 0) & (xs < gw)).reshape(-1)
                clip = bool(st.flags & (clear.STEP_CLIP1 if side else clear.STEP_CLIP0))
                assert clip == (not on_grid.all())
                if not st.flags & (clear.STEP_MASKED1 if side else clear.STEP_MASKED0):
                    continue
                assert 0 <= e < len(table), "masked 2-D tile without a mask-table entry"
                bits = ((table[e][:, :, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(128, 128).astype(bool)
                toks = (T + ys * gw + xs).reshape(-1)
                for rr in range(128):
                    q_y, q_x = qy + rr // tw, it.qx + rr % tw
                    if q_y >= gh or q_x >= gw:
                        continue
                    row = oracle.mask_row(T + q_y * gw + q_x, gh, gw, T, r).astype(bool)
                    assert np.array_equal(bits[rr][on_grid], row[toks[on_grid]])


@pytest.mark.parametrize("gh,gw,T,r", SHAPES + [(40, 40, 300, 9.0), (17, 16, 129, 4.0)])
def test_pair_schedule_covers_each_allowed_pair_exactly_once(gh, gw, T, r):
    p = clear.Plan(1, 1, gh, gw, T, 128, r, kernel=clear.KERNEL_TCGEN05_WS, host_only=True)
    info = p.info()
    items, steps = p.pair_tables()
    N = T + gh * gw
    th, tw = info.tile_h, info.tile_w
    assert th * tw == 128 and info.n_work_items == len(items)
    n_text_items = sum(1 for it in items if it.kind == 1)
    assert all(it.kind == 1 for it in items[:n_text_items]) and all(it.kind == 0 for it in items[n_text_items:])
    img_counts = [it.step_count for it in items[n_text_items:]]
    assert img_counts == sorted(img_counts, reverse=True)
    assert info.max_item_tiles == max(it.step_count for it in items)

    executed = 0
    seen_queries = np.zeros(N, dtype=np.int64)
    text_cover = {}
    slots = set()
    for it in items:
        assert it.step_count >= 1 and it.n_sides in (1, 2)
        sts = steps[it.step_begin: it.step_begin + it.step_count]
        # ring bookkeeping: K and V of each distinct key tile of a step take one stage each, in the order
        # K(s), V(s) for every step s
        def tiles_of(st):
            return int(bool(st.flags & clear.STEP_USE0)) + int(bool(st.flags & clear.STEP_USE1) and
                                                               not st.flags & clear.STEP_SHARED)
        order = []
        for i in range(len(sts)):
            order.append(("K", i))
            order.append(("V", i))
        pos, where = 0, {}
        for kind, i in order:
            where[(kind, i)] = pos
            pos += tiles_of(sts[i])
        loads = 0
        for i, st in enumerate(sts):
            assert st.load_base & 0xffff == where[("K", i)] and st.load_base >> 16 == where[("V", i)]
            use0, use1 = bool(st.flags & clear.STEP_USE0), bool(st.flags & clear.STEP_USE1)
            shared = bool(st.flags & clear.STEP_SHARED)
            assert use0 or use1
            if shared:
                assert use0 and use1 and (st.x0, st.y0) == (st.x1, st.y1)
            if it.n_sides == 1:
                assert not use1
            if use0 and use1 and not shared and not (st.flags & clear.STEP_LINEAR):
                assert (st.x0, st.y0) != (st.x1, st.y1)
            loads += 2 * (int(use0) + int(use1 and not shared))
            executed += (int(use0) + int(use1)) * 128 * 128
        assert it.n_loads == loads
        for side in range(it.n_sides):
            use_bit = clear.STEP_USE1 if side else clear.STEP_USE0
            mask_bit = clear.STEP_MASKED1 if side else clear.STEP_MASKED0
            mine = [st for st in sts if st.flags & use_bit]
            assert mine, "a query tile with no key tile"
            tiles = [((st.x1, st.y1, st.n_valid1) if side else (st.x0, st.y0, st.n_valid0)) +
                     (bool(st.flags & clear.STEP_LINEAR), bool(st.flags & mask_bit)) for st in mine]
            slot = it.partial_slot1 if side else it.partial_slot0
            n_rows = it.n_rows1 if side else it.n_rows0
            if it.kind == 1:
                q0 = it.qx + 128 * side
                assert q0 % 128 == 0 and n_rows == min(128, T - q0) and n_rows > 0
                toks = []
                for (x, y, nv, linear, masked) in tiles:
                    assert linear and nv == min(128, N - x) and masked == (nv < 128)
                    toks += list(range(x, x + nv))
                assert toks == list(range(toks[0], toks[-1] + 1))
                text_cover.setdefault(q0, []).extend(toks)
                if info.n_text_splits > 1:
                    assert slot >= 0 and slot not in slots and slot // info.n_text_splits == q0 // 128
                    slots.add(slot)
                else:
                    assert slot == -1
                continue
            qy = it.qy1 if side else it.qy0
            assert slot == -1 and it.qx % tw == 0 and qy % th == 0
            if side:
                assert it.qy1 == it.qy0 + th
            qs = [(y, x) for y in range(qy, min(qy + th, gh)) for x in range(it.qx, min(it.qx + tw, gw))]
            assert n_rows == len(qs) and n_rows > 0
            cover = np.zeros(N, dtype=np.int64)
            unmasked = np.zeros(N, dtype=bool)
            rows = {q: oracle.mask_row(T + q[0] * gw + q[1], gh, gw, T, r).astype(bool) for q in qs}
            for (x, y, nv, linear, masked) in tiles:
                idx, whole = key_tokens(x, y, linear, nv, gh, gw, T, th, tw)
                if linear:
                    assert x + nv <= T and masked == (nv < 128)
                else:
                    # no useless tile: it holds at least one allowed pair
                    assert any(rows[q][idx].any() for q in qs)
                    if not masked:
                        assert whole
                        unmasked[idx] = True
                cover[idx] += 1
            assert cover.max() <= 1
            for q in qs:
                seen_queries[T + q[0] * gw + q[1]] += 1
                assert not (rows[q] & (cover == 0)).any(), "an allowed key is in no tile of the query tile"
                assert rows[q][unmasked].all(), "a tile flagged mask-free holds a disallowed pair"
    assert info.executed_pairs == executed
    assert np.all(seen_queries[T:] == 1)
    check_mask_table(p, items, steps, gh, gw, T, r, th, tw)
    for q0 in range(0, T, 128):
        assert sorted(text_cover[q0]) == list(range(N))
    if info.n_text_splits > 1:
        assert len(slots) == math.ceil(T / 128) * info.n_text_splits
        assert info.workspace_bytes == len(slots) * 128 * (128 + 2) * 4


def test_mask_table_cap_sends_patches_to_the_table_free_path(monkeypatch):
    monkeypatch.setenv("CLEAR_MAX_MASK_ENTRIES", "3")
    p = clear.Plan(1, 1, 40, 40, 0, 128, 9.0, kernel=clear.KERNEL_TCGEN05_WS, host_only=True)
    items, steps = p.pair_tables()
    assert len(p.mask_table()) == 3
    ids = set()
    for it in items:
        for st in steps[it.step_begin: it.step_begin + it.step_count]:
            if st.flags & clear.STEP_LINEAR:
                continue
            if st.flags & clear.STEP_USE0 and st.flags & clear.STEP_MASKED0:
                ids.add(st.n_valid0)
            if st.flags & clear.STEP_USE1 and st.flags & clear.STEP_MASKED1:
                ids.add(st.n_valid1)
    assert ids == {-1, 0, 1, 2}


def test_pair_schedule_at_the_8k_workload():
    p = clear.Plan(1, 24, 512, 512, 512, 128, 16.0, host_only=True)
    info = p.info()
    assert info.kernel == clear.KERNEL_TCGEN05_WS
    assert info.sum_mask == 471125568
    items, steps = p.pair_tables()
    interior = [it for it in items if it.kind == 0 and it.step_count == 19]
    assert len(interior) > 800                           # 4 text + 3 one-sided pairs + 12 shared key patches
    it = interior[0]
    sts = steps[it.step_begin: it.step_begin + it.step_count]
    assert sum(1 for st in sts if st.flags & clear.STEP_SHARED) == 16 and it.n_loads == 2 * 22
    # every query tile still executes 19 key tiles: the same geometric efficiency as one tile per block
    one = clear.Plan(1, 24, 512, 512, 512, 128, 16.0, kernel=clear.KERNEL_TCGEN05, host_only=True).info()
    assert info.executed_pairs == one.executed_pairs
    assert max(it.step_count for it in items) <= 64


def test_text_rows_are_split_for_long_sequences():
    p = clear.Plan(1, 24, 512, 512, 512, 128, 16.0, kernel=clear.KERNEL_TCGEN05, host_only=True)
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


def test_key_lists_beyond_the_step_records_positions_fall_back():
    """A pair item that stages more than 65535 key / value tiles cannot be named by the 16-bit ring positions of
    the step records: the warp-specialised kernel refuses the shape, and a plan that leaves the choice to the
    library runs it on the CUDA-core kernel."""
    gh = gw = 2048          # 32768 key patches, every one within reach of every query patch at this radius
    with pytest.raises(clear.ClearError) as e:
        clear.Plan(1, 1, gh, gw, 0, 128, 4096.0, kernel=clear.KERNEL_TCGEN05_WS, host_only=True)
    assert e.value.status == clear.ERR_UNSUPPORTED
    p = clear.Plan(1, 1, gh, gw, 0, 128, 4096.0, host_only=True)
    assert p.info().kernel == clear.KERNEL_SIMT
    n = gh * gw
    assert p.info().sum_mask == n * n


@pytest.mark.parametrize("gh,gw,T,r", [(16, 16, 16, 4.0), (13, 19, 7, 2.5), (40, 24, 256, 16.0), (4, 100, 3, 30.0)])
def test_square_window_geometry_and_schedules(gh, gw, T, r):
    """The square window of Neighborhood Attention through the same plan interface: half widths, sum(M) and the
    mask table against the window oracle; every allowed pair lies in exactly one listed key tile."""
    from oracle import clear_oracle_windows as win
    total, _ = win.mask_counts(win.SQUARE, r, 0, gh, gw, T)
    h = math.ceil(r) - 1
    for kernel in (clear.KERNEL_SIMT, clear.KERNEL_TCGEN05, clear.KERNEL_TCGEN05_WS):
        p = clear.Plan(1, 1, gh, gw, T, 128, r, kernel=kernel, host_only=True, mask_kind=clear.MASK_SQUARE)
        assert p.info().sum_mask == total
        _, _, hw = p.tables()
        assert hw == [min(h, gw - 1)] * (min(h, gh - 1) + 1)
    # tile kernel: the listed key tiles of every query patch hold every allowed key of its queries
    p = clear.Plan(1, 1, gh, gw, T, 128, r, kernel=clear.KERNEL_TCGEN05, host_only=True, mask_kind=clear.MASK_SQUARE)
    items, tiles, _ = p.tables()
    N = T + gh * gw
    for it in items:
        if it.kind != 0:
            continue
        covered = np.zeros(N, dtype=bool)
        for kt in tiles[it.tile_begin: it.tile_begin + it.tile_count]:
            if kt.flags & clear.TILE_LINEAR:
                covered[kt.x: kt.x + kt.n_valid] = True
            else:
                for yy in range(kt.y, min(kt.y + 8, gh)):
                    covered[T + yy * gw + kt.x: T + yy * gw + min(kt.x + 16, gw)] = True
        for qy in range(it.qy, min(it.qy + 8, gh)):
            for qx in range(it.qx, min(it.qx + 16, gw)):
                row = win.mask_row(win.SQUARE, r, 0, T + qy * gw + qx, gh, gw, T).astype(bool)
                assert not (row & ~covered).any()
    with pytest.raises(clear.ClearError):
        clear.Plan(1, 1, gh, gw, T, 128, r, host_only=True, mask_kind=5)


@pytest.mark.parametrize("kind,a,b,gh,gw,T", [
    ("windows", 16, 0, 64, 64, 512), ("windows", 16, 8, 64, 64, 512), ("windows", 5, 2, 13, 19, 7),
    ("windows", 100, 3, 9, 11, 0), ("strided", 4, 0, 64, 64, 512), ("strided", 4, 5, 20, 13, 3),
    ("strided", 7, 30, 9, 40, 0), ("strided", 1, 0, 6, 5, 2),
])
def test_window_grid_and_strided_plans_count_the_oracles_pairs(kind, a, b, gh, gw, T):
    from oracle import clear_oracle_windows as win
    okind = win.WINDOWS if kind == "windows" else win.STRIDED
    ckind = clear.MASK_WINDOWS if kind == "windows" else clear.MASK_STRIDED
    p = clear.Plan(1, 24, gh, gw, T, 128, a, host_only=True, mask_kind=ckind, mask_param=b)
    info = p.info()
    assert info.kernel == clear.KERNEL_SIMT          # no window around the query: the CUDA-core kernel
    assert info.sum_mask == win.mask_counts(okind, a, b, gh, gw, T)[0]
    assert info.flops == 4.0 * info.sum_mask * 128 * 24


def test_comparison_masks_reproduce_the_papers_flop_figure():
    # Tab. 1 prints 67.7 GFLOPS for both the Swin-window and the strided baseline at 1024 x 1024 (64 x 64 tokens
    # + 512 text tokens, c = 3072): 4 * sum(M) * c through the plan
    for kind, a in ((clear.MASK_WINDOWS, 16), (clear.MASK_STRIDED, 4)):
        info = clear.Plan(1, 24, 64, 64, 512, 128, a, host_only=True, mask_kind=kind).info()
        assert round(info.flops / 1e9, 1) in (67.6, 67.7)


def test_comparison_mask_plans_reject_bad_arguments():
    import ctypes

    def rc(kind, size, param, dtype=clear.BF16, d=128):
        h = ctypes.c_void_p()
        out = clear.load().clear_plan_create_mask(ctypes.byref(h), 1, 1, 8, 8, 2, d, dtype, kind, size, param, 1)
        if out == 0:
            clear.load().clear_plan_destroy(h)
        return out
    assert rc(clear.MASK_WINDOWS, 4.0, 1) == 0 and rc(clear.MASK_STRIDED, 3.0, 7, clear.F32, 40) == 0
    assert rc(clear.MASK_DISC, 4.0, 0) == 0
    assert rc(clear.MASK_WINDOWS, 4.5, 0) == clear.ERR_INVALID_ARG     # a window is a whole number of cells
    assert rc(clear.MASK_STRIDED, 0.5, 0) == clear.ERR_INVALID_ARG
    assert rc(clear.MASK_WINDOWS, 4.0, -1) == clear.ERR_INVALID_ARG
    assert rc(clear.MASK_DISC, 4.0, 3) == clear.ERR_INVALID_ARG        # the disc takes no second parameter
    assert rc(7, 4.0, 0) == clear.ERR_INVALID_ARG
    # the tensor-core kernels' tables do not carry these masks
    with pytest.raises(clear.ClearError):
        clear.Plan(1, 1, 8, 8, 2, 128, 4, kernel=clear.KERNEL_TCGEN05_WS, host_only=True, mask_kind=clear.MASK_WINDOWS)
