"""GPU parity of the row-band form (Sec. 3.4).  One GPU plays the ranks one after the other (no kernel waits for
another): each band gets the local tensors its layout names, its two plans run, and the merged result must be the
single-GPU operator's -- against the attention oracle for the exact merge, against the patch-average oracle for
Eq. 7 -- on small shapes everywhere and at the 8K shape's band sizes on sampled rows."""
import math

import numpy as np
import pytest
import torch

from oracle import clear_oracle as oracle
from oracle import clear_oracle_bands as oracle_bands
from paper_2412_16112_b200 import band_parallel as bp
from paper_2412_16112_b200 import binding as clear
from paper_2412_16112_b200 import workloads

pytestmark = pytest.mark.gpu

BF16_MAX, BF16_MEAN = 2e-2, 2e-3


def run_bands(q, k, v, gh, gw, T, r, scale, world, text_mode, dev):
    """All ranks in turn on one device.  Returns the assembled [B, H, N, d] output (CPU, fp64)."""
    B, H, N, d = q.shape
    lays = bp.all_layouts(gh, gw, T, r, world)
    out = torch.full((B, H, N, d), float("nan"), dtype=torch.float64)
    records, keep = [], []
    for p, lay in enumerate(lays):
        ql, kl, vl = (bp.slice_local(t, lay).to(dev) for t in (q, k, v))
        # halo rows of Q are never read: poison them
        ql[:, :, lay.token_range(0, lay.q_row_begin)] = float("nan")
        ql[:, :, lay.token_range(lay.q_row_end, lay.local_rows)] = float("nan")
        ol = torch.full_like(ql, float("nan"))
        img = clear.BandPlan(B, H, lay.local_rows, gw, T, d, r, clear.PART_BAND_IMAGE, lay.q_row_begin, lay.q_row_end)
        img.forward(ql, kl, vl, ol, scale)
        img.check()
        band = lay.token_range(lay.q_row_begin, lay.q_row_end)
        out[:, :, T + lay.y0 * gw: T + lay.y1 * gw] = ol[:, :, band].cpu().to(torch.float64)
        # text rows are not this plan's to write
        assert torch.isnan(ol[:, :, :T].float()).all()
        if T > 0:
            txt = clear.BandPlan(B, H, lay.local_rows, gw, T, d, r, clear.PART_BAND_TEXT, lay.q_row_begin, lay.q_row_end,
                                 text_keys=(p == 0 or text_mode == "average"))
            rec = torch.full((B * H, T, d + 2), float("nan"), dtype=torch.float32, device=dev)
            txt.text_partial(ql, kl, vl, rec, scale)
            txt.check()
            records.append(rec)
            keep.append(txt)
    if T > 0:
        gathered = torch.stack(records).contiguous()
        assert torch.isfinite(gathered).all()
        merged = torch.full((B, H, T + 8, d), float("nan"), dtype=torch.bfloat16, device=dev)
        clear.clear_text_merge(gathered, merged, T, clear.TEXT_MERGE_EXACT if text_mode == "exact" else clear.TEXT_MERGE_AVERAGE)
        torch.cuda.synchronize()
        assert torch.isnan(merged[:, :, T:].float()).all()       # rows past the text rows are left alone
        out[:, :, :T] = merged[:, :, :T].cpu().to(torch.float64)
    return out.numpy()


@pytest.mark.parametrize("gh,gw,T,r,d,world", [
    (24, 20, 5, 3.0, 128, 3),      # ragged patches, three bands
    (40, 16, 130, 4.5, 64, 4),     # two text tiles, head size 64
    (33, 35, 0, 8.0, 128, 2),      # no text
    (64, 16, 3, 16.0, 128, 3),     # reach 15: halos of 15 and 16 rows
    (16, 48, 200, 4.0, 128, 1),    # one band: the whole operator through the band plans
    (30, 7, 9, 1.0, 64, 5),        # windows that see their own row only: no halo
])
def test_exact_band_form_matches_the_oracle_everywhere(gh, gw, T, r, d, world):
    q, k, v = workloads.make_custom(1, 2, gh, gw, T, d, dtype="bf16", seed=gh + 3 * world)
    scale = 1 / math.sqrt(d)
    want = oracle.attn(q, k, v, gh, gw, T, r, scale)
    got = run_bands(q, k, v, gh, gw, T, r, scale, world, "exact", torch.device("cuda:0"))
    assert np.isfinite(got).all()
    err = np.abs(got - want)
    assert err.max() <= BF16_MAX and err.mean() <= BF16_MEAN, (float(err.max()), float(err.mean()))


@pytest.mark.parametrize("gh,gw,T,r,d,world", [(24, 20, 5, 3.0, 128, 3), (40, 16, 130, 4.5, 64, 4), (64, 32, 256, 8.0, 128, 2)])
def test_patch_average_of_the_text_rows_matches_its_oracle(gh, gw, T, r, d, world):
    q, k, v = workloads.make_custom(1, 2, gh, gw, T, d, dtype="bf16", seed=gh + 5 * world)
    scale = 1 / math.sqrt(d)
    want_text = oracle_bands.text_rows_patch_average(q.to(torch.float64).numpy(), k.to(torch.float64).numpy(),
                                                     v.to(torch.float64).numpy(), gh, gw, T, scale, world)
    want_img = oracle.attn(q, k, v, gh, gw, T, r, scale)[:, :, T:]
    got = run_bands(q, k, v, gh, gw, T, r, scale, world, "average", torch.device("cuda:0"))
    err_t, err_i = np.abs(got[:, :, :T] - want_text), np.abs(got[:, :, T:] - want_img)
    assert err_t.max() <= BF16_MAX and err_t.mean() <= BF16_MEAN, (float(err_t.max()), float(err_t.mean()))
    assert err_i.max() <= BF16_MAX and err_i.mean() <= BF16_MEAN


def test_band_of_the_8k_shape_on_sampled_rows():
    """Band 3 of 8 of the 512 x 512 grid (24 heads, 512 text tokens, r = 16) at full size: sampled image rows of
    the band against the oracle on the whole grid, and the text records of this band against fp64 sums over its
    keys (2^(s - m) weights as the header defines them)."""
    w = workloads.WORKLOADS["c4_8k_r16"]
    gh, gw, T, d, H, r = w.grid_h, w.grid_w, w.n_text, w.head_dim, 3, w.radius
    dev = torch.device("cuda:0")
    q, k, v = workloads.make_inputs(w, heads=H)
    lays = bp.all_layouts(gh, gw, T, r, 8)
    lay = lays[3]
    assert (lay.y0, lay.y1, lay.halo_lo, lay.halo_hi) == (192, 256, 16, 15)
    ql, kl, vl = (bp.slice_local(t, lay).to(dev) for t in (q, k, v))
    ol = torch.full_like(ql, float("nan"))
    img = clear.BandPlan(1, H, lay.local_rows, gw, T, d, r, clear.PART_BAND_IMAGE, lay.q_row_begin, lay.q_row_end)
    img.forward(ql, kl, vl, ol, w.scale)
    txt = clear.BandPlan(1, H, lay.local_rows, gw, T, d, r, clear.PART_BAND_TEXT, lay.q_row_begin, lay.q_row_end, text_keys=False)
    rec = torch.empty(H, T, d + 2, dtype=torch.float32, device=dev)
    txt.text_partial(ql, kl, vl, rec, w.scale)
    torch.cuda.synchronize()
    img.check(); txt.check()
    band = ol[:, :, lay.token_range(lay.q_row_begin, lay.q_row_end)]
    assert torch.isfinite(band.float()).all()
    rng = np.random.default_rng(8)
    ys = np.concatenate([[192, 192, 255, 255, 200], rng.integers(192, 256, size=60)])
    xs = np.concatenate([[0, 511, 0, 511, 17], rng.integers(0, gw, size=60)])
    rows = (T + ys * gw + xs).astype(np.int64)
    for h in range(H):
        triples = np.stack([np.zeros_like(rows), np.full_like(rows, h), rows], axis=1)
        want = oracle.attn_rows(q, k, v, gh, gw, T, r, w.scale, triples)
        local = torch.from_numpy(T + (ys - lay.y0 + lay.halo_lo) * gw + xs).to(dev)
        got = ol[0, h, local].cpu().to(torch.float64).numpy()
        err = np.abs(got - want)
        assert err.max() <= BF16_MAX and err.mean() <= BF16_MEAN, (h, float(err.max()))
    # text records of this band: keys are its 64 * 512 image tokens only
    qt = q[0, :, :T].to(torch.float64)
    kb = k[0, :, T + lay.y0 * gw: T + lay.y1 * gw].to(torch.float64)
    vb = v[0, :, T + lay.y0 * gw: T + lay.y1 * gw].to(torch.float64)
    s = torch.einsum("hid,hjd->hij", qt[:, :64], kb) * (w.scale * math.log2(math.e))
    rec_c = rec.cpu().to(torch.float64)
    m, l, o = rec_c[:, :64, d], rec_c[:, :64, d + 1], rec_c[:, :64, :d]
    wgt = torch.exp2(s - m[..., None])
    assert torch.allclose(wgt.sum(-1), l, rtol=5e-3)
    ref_o = torch.einsum("hij,hjd->hid", wgt, vb)
    assert (o - ref_o).abs().max() <= 5e-3 * ref_o.abs().max()
    # normalised, they are this band's own softmax: weights at most 2^8 by the kernel's rescale rule
    assert float(wgt.max()) <= 2.0 ** 8 * 1.01


def test_band_attention_object_on_one_rank():
    """The orchestration class with a world of one (no process group needed): whole operator through it."""
    gh, gw, T, d, r = 32, 32, 64, 128, 6.0
    q, k, v = workloads.make_custom(1, 2, gh, gw, T, d, dtype="bf16", seed=77)
    scale = 1 / math.sqrt(d)
    dev = torch.device("cuda:0")
    att = bp.BandAttention(1, 2, gh, gw, T, d, r, rank=0, world=1)
    qd, kd, vd = (t.to(dev) for t in (q, k, v))
    out = torch.full_like(qd, float("nan"))
    att.forward(qd, kd, vd, out, scale)
    torch.cuda.synchronize()
    att.check()
    want = oracle.attn(q, k, v, gh, gw, T, r, scale)
    err = np.abs(out.cpu().to(torch.float64).numpy() - want)
    assert err.max() <= BF16_MAX and err.mean() <= BF16_MEAN
