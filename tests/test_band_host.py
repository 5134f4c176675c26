"""Host logic of the row-band form (Sec. 3.4), no GPU: band geometry against the band oracle, the claim that a band
plus its halo rows holds every key its image queries can see (from the attention oracle's mask rows), and the
schedules of the two band parts against the oracle's mask on the local grid."""
import numpy as np
import pytest

from oracle import clear_oracle as oracle
from oracle import clear_oracle_bands as bands
from paper_2412_16112_b200 import binding as clear

from test_plan_host import check_mask_table, key_tokens

CASES = [(24, 20, 5, 3.0, 3), (40, 16, 130, 4.5, 4), (33, 35, 0, 8.0, 2), (16, 16, 16, 4.0, 1), (64, 16, 3, 16.0, 3)]


@pytest.mark.parametrize("gh,r,G", [(512, 16.0, 8), (128, 16.0, 8), (13, 2.5, 4), (7, 1.0, 7), (100, 32.0, 3), (10, 100.0, 2)])
def test_band_geometry_matches_the_oracle(gh, r, G):
    R = bands.reach(r)
    for p in range(G):
        y0, y1, lo, hi = clear.band_geometry(gh, r, G, p)
        assert (y0, y1) == bands.band_rows(gh, G, p)
        assert lo == min(R, y0) and hi == min(R, gh - y1)
    # the square window reaches ceil(r) - 1 rows
    assert clear.band_geometry(100, 4.5, 2, 1, mask_kind=clear.MASK_SQUARE)[2] == 4


def test_band_geometry_rejects_bad_arguments():
    lib = clear.load()
    for args in ((0, 4.0, 0, 1, 0), (8, 4.0, 0, 9, 0), (8, 4.0, 0, 2, 2), (8, 0.0, 0, 2, 0), (8, 4.0, 5, 2, 0), (8, 4.0, 0, 0, 0)):
        assert lib.clear_band_geometry(*args, None, None, None, None) == clear.ERR_INVALID_ARG


@pytest.mark.parametrize("gh,gw,T,r,G", CASES)
def test_a_band_and_its_halo_hold_every_key_of_its_image_queries(gh, gw, T, r, G):
    """Mask rows of the whole grid, for every query of the band: no key outside the band's local rows, and inside
    them the same pattern as the mask rows of the local grid (the local border is the true border or out of reach)."""
    for p in range(G):
        y0, y1, lo, hi = clear.band_geometry(gh, r, G, p)
        a, b = y0 - lo, y1 + hi
        for y in range(y0, y1):
            for x in (0, gw // 2, gw - 1):
                row = oracle.mask_row(T + y * gw + x, gh, gw, T, r).astype(bool)
                img = row[T:].reshape(gh, gw)
                assert not img[:a].any() and not img[b:].any()
                local = oracle.mask_row(T + (y - a) * gw + x, b - a, gw, T, r).astype(bool)
                assert np.array_equal(local[:T], row[:T]) and np.array_equal(local[T:].reshape(b - a, gw), img[a:b])


@pytest.mark.parametrize("gh,gw,T,r,G", CASES)
def test_band_image_schedule_covers_the_bands_queries(gh, gw, T, r, G):
    for p in range(G):
        y0, y1, lo, hi = clear.band_geometry(gh, r, G, p)
        rows, qb, qe = lo + (y1 - y0) + hi, lo, lo + (y1 - y0)
        plan = clear.BandPlan(1, 1, rows, gw, T, 128, r, clear.PART_BAND_IMAGE, qb, qe, host_only=True)
        info = plan.info()
        items, steps = plan.pair_tables()
        th, tw = info.tile_h, info.tile_w
        N = T + rows * gw
        assert all(it.kind == 0 for it in items) and info.n_text_splits == 0 and info.workspace_bytes == 0
        seen = np.zeros((rows, gw), dtype=np.int64)
        pairs = 0
        for it in items:
            sts = steps[it.step_begin: it.step_begin + it.step_count]
            for side in range(it.n_sides):
                use_bit = clear.STEP_USE1 if side else clear.STEP_USE0
                mask_bit = clear.STEP_MASKED1 if side else clear.STEP_MASKED0
                qy = it.qy1 if side else it.qy0
                # only patches that hold rows of the band
                assert qy < qe and qy + th > qb
                cover = np.zeros(N, dtype=np.int64)
                for st in sts:
                    if not st.flags & use_bit:
                        continue
                    x, y, nv = (st.x1, st.y1, st.n_valid1) if side else (st.x0, st.y0, st.n_valid0)
                    linear = bool(st.flags & clear.STEP_LINEAR)
                    idx, _ = key_tokens(x, y, linear, nv, rows, gw, T, th, tw)
                    if linear:
                        assert x + nv <= T
                    cover[idx] += 1
                assert cover.max() <= 1
                for yy in range(qy, min(qy + th, rows)):
                    for xx in range(it.qx, min(it.qx + tw, gw)):
                        seen[yy, xx] += 1
                        row = oracle.mask_row(T + yy * gw + xx, rows, gw, T, r).astype(bool)
                        assert not (row & (cover == 0)).any()
                        if qb <= yy < qe:
                            pairs += int(row.sum())
        assert np.all(seen[qb:qe] == 1) and seen.max() <= 1
        assert info.sum_mask == pairs
        check_mask_table(plan, items, steps, rows, gw, T, r, th, tw)


@pytest.mark.parametrize("gh,gw,T,r,G", [c for c in CASES if c[2] > 0] + [(300, 64, 200, 8.0, 2)])
@pytest.mark.parametrize("text_keys", [True, False])
def test_band_text_schedule_covers_the_bands_keys(gh, gw, T, r, G, text_keys):
    for p in range(G):
        y0, y1, lo, hi = clear.band_geometry(gh, r, G, p)
        rows, qb, qe = lo + (y1 - y0) + hi, lo, lo + (y1 - y0)
        plan = clear.BandPlan(1, 1, rows, gw, T, 128, r, clear.PART_BAND_TEXT, qb, qe, text_keys=text_keys, host_only=True)
        info = plan.info()
        items, steps = plan.pair_tables()
        want = (list(range(T)) if text_keys else []) + list(range(T + qb * gw, T + qe * gw))
        assert info.sum_mask == T * len(want) and info.n_text_splits >= 1
        assert all(it.kind == 1 for it in items)
        cover, slots = {}, set()
        for it in items:
            sts = steps[it.step_begin: it.step_begin + it.step_count]
            for side in range(it.n_sides):
                q0 = it.qx + 128 * side
                slot = it.partial_slot1 if side else it.partial_slot0
                # always partial results, one slot per (text tile, key split)
                assert slot >= 0 and slot not in slots and slot // info.n_text_splits == q0 // 128
                slots.add(slot)
                for st in sts:
                    assert st.flags & clear.STEP_LINEAR and st.flags & (clear.STEP_USE1 if side else clear.STEP_USE0)
                    nv = st.n_valid1 if side else st.n_valid0
                    assert bool(st.flags & (clear.STEP_MASKED1 if side else clear.STEP_MASKED0)) == (nv < 128)
                    cover.setdefault(q0, []).extend(range(st.x0, st.x0 + nv))
        for q0 in range(0, T, 128):
            assert sorted(cover[q0]) == want
        assert len(slots) == -(-T // 128) * info.n_text_splits
        assert info.workspace_bytes == len(slots) * 128 * (128 + 2) * 4


def test_band_plans_reject_bad_arguments():
    def rc(**kw):
        a = dict(B=1, H=1, rows=20, gw=16, T=4, d=128, r=4.0, kind=0, part=clear.PART_BAND_IMAGE, qb=3, qe=11, tk=1)
        a.update(kw)
        import ctypes
        h = ctypes.c_void_p()
        out = clear.load().clear_plan_create_band(ctypes.byref(h), a["B"], a["H"], a["rows"], a["gw"], a["T"], a["d"], a["r"],
                                                  a["kind"], a["part"], a["qb"], a["qe"], a["tk"], 1)
        if out == 0:
            clear.load().clear_plan_destroy(h)
        return out
    assert rc() == 0
    assert rc(part=0) == clear.ERR_INVALID_ARG and rc(part=3) == clear.ERR_INVALID_ARG
    assert rc(qb=11, qe=11) == clear.ERR_INVALID_ARG and rc(qe=21) == clear.ERR_INVALID_ARG and rc(qb=-1) == clear.ERR_INVALID_ARG
    assert rc(part=clear.PART_BAND_TEXT, T=0) == clear.ERR_INVALID_ARG
    assert rc(d=96) == clear.ERR_UNSUPPORTED
    # a band-text plan is not run by the ordinary planned call, nor an ordinary plan by the partial call
    p = clear.BandPlan(1, 1, 20, 16, 4, 128, 4.0, clear.PART_BAND_TEXT, 3, 11, host_only=True)
    assert clear.load().clear_attn_fwd_planned(p.handle, 0x1000, 0x1000, 0x1000, 0x2000, 1.0, None) == clear.ERR_PLAN_MISMATCH
    q = clear.Plan(1, 1, 20, 16, 4, 128, 4.0, host_only=True)
    assert clear.load().clear_attn_text_partial(q.handle, 0x1000, 0x1000, 0x1000, 0x2000, 1.0, None) == clear.ERR_PLAN_MISMATCH
    lib = clear.load()
    assert lib.clear_text_merge(None, 2, 1, 1, 4, 128, 0, 0x1000, 20, None) == clear.ERR_INVALID_ARG
    assert lib.clear_text_merge(0x1000, 2, 1, 1, 4, 128, 2, 0x1000, 20, None) == clear.ERR_INVALID_ARG
    assert lib.clear_text_merge(0x1000, 2, 1, 1, 4, 96, 0, 0x1000, 20, None) == clear.ERR_UNSUPPORTED
    assert lib.clear_text_merge(0x1000, 2, 1, 1, 4, 128, 0, 0x1008, 20, None) == clear.ERR_MISALIGNED
