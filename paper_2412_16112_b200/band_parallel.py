"""Row-band parallel CLEAR attention over several GPUs (Sec. 3.4), one process per GPU.

Every rank owns a band of image rows and holds the text tokens.  Its LOCAL tensors are
``[B, H, n_text + local_rows * grid_w, d]``: the text tokens, then the rows ``y0 - halo_lo .. y1 + halo_hi - 1`` of the
grid.  One call does, on the rank's own stream:

  1. halo exchange: the first / last rows of the band's K and V go to the previous / next rank (point-to-point
     send / recv through ``torch.distributed`` into contiguous local buffers, then into the halo rows of the local
     tensors): the only image-token traffic, O(r * W) per neighbour;
  2. the band's image queries (``PART_BAND_IMAGE`` plan) over band + halo keys and the text keys;
  3. the text queries over the rank's own keys (``PART_BAND_TEXT`` plan) as one record of d + 2 floats per row;
  4. all-gather of the records and their merge: exact, or the patch-wise average of Eq. 7.

All arithmetic is in the CUDA library; this module moves bytes and calls entry points.  The exchange functions work
on CPU tensors with the gloo backend as well, which is how their index arithmetic is tested without GPUs.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch
import torch.distributed as dist

from . import binding as clear

PATCH_ROWS = 8  # query patches are 8 grid rows tall: halos rounded up to it keep the band's patches aligned


@dataclass(frozen=True)
class BandLayout:
    y0: int            # first grid row of the band
    y1: int            # one past its last row
    halo_lo: int       # rows held above the band
    halo_hi: int       # rows held below it
    grid_w: int
    n_text: int

    @property
    def band_rows(self) -> int:
        return self.y1 - self.y0

    @property
    def local_rows(self) -> int:
        return self.halo_lo + self.band_rows + self.halo_hi

    @property
    def q_row_begin(self) -> int:
        return self.halo_lo

    @property
    def q_row_end(self) -> int:
        return self.halo_lo + self.band_rows

    @property
    def n_local_tokens(self) -> int:
        return self.n_text + self.local_rows * self.grid_w

    def token_range(self, row_begin: int, row_end: int) -> slice:
        """Tokens of local rows [row_begin, row_end)."""
        return slice(self.n_text + row_begin * self.grid_w, self.n_text + row_end * self.grid_w)


def band_layout(grid_h: int, grid_w: int, n_text: int, radius: float, world: int, rank: int,
                mask_kind: int = clear.MASK_DISC) -> BandLayout:
    """Layout of one rank.  The halo above the band is rounded up to whole query patches where the grid has the
    rows (more keys than the window reaches change nothing), so that the band's patches start on a patch row."""
    y0, y1, lo, hi = clear.band_geometry(grid_h, radius, world, rank, mask_kind)
    if lo > 0:
        lo = min(y0, -(-lo // PATCH_ROWS) * PATCH_ROWS)
    return BandLayout(y0, y1, lo, hi, grid_w, n_text)


def all_layouts(grid_h, grid_w, n_text, radius, world, mask_kind=clear.MASK_DISC):
    lays = [band_layout(grid_h, grid_w, n_text, radius, world, p, mask_kind) for p in range(world)]
    for p, lay in enumerate(lays):
        if p > 0 and lay.halo_lo > lays[p - 1].band_rows or p + 1 < world and lay.halo_hi > lays[p + 1].band_rows:
            raise ValueError("a band is thinner than its neighbour's halo: use fewer ranks for this radius")
    return lays


def slice_local(x: torch.Tensor, lay: BandLayout) -> torch.Tensor:
    """Local tensor of a rank cut out of the whole [B, H, N, d] tensor (what a rank holds after the exchange)."""
    a, b = lay.y0 - lay.halo_lo, lay.y1 + lay.halo_hi
    T, W = lay.n_text, lay.grid_w
    return torch.cat([x[:, :, :T], x[:, :, T + a * W: T + b * W]], dim=2).contiguous()


def exchange_halos(k: torch.Tensor, v: torch.Tensor, lays, rank: int, group=None) -> None:
    """Fill the halo rows of this rank's local K and V from the neighbours' bands (in place)."""
    world = len(lays)
    me = lays[rank]
    ops, recvs = [], []

    def pack(row_begin, row_end):
        sl = me.token_range(row_begin, row_end)
        return torch.stack([k[:, :, sl], v[:, :, sl]]).contiguous()

    def buffer(rows):
        B, H, _, d = k.shape
        return torch.empty(2, B, H, rows * me.grid_w, d, dtype=k.dtype, device=k.device)

    keep = []
    if rank > 0:
        up = lays[rank - 1]
        if up.halo_hi > 0:   # my first rows are the previous rank's lower halo
            keep.append(pack(me.q_row_begin, me.q_row_begin + up.halo_hi))
            ops.append(dist.P2POp(dist.isend, keep[-1], rank - 1, group))
        if me.halo_lo > 0:
            buf = buffer(me.halo_lo)
            recvs.append((buf, 0, me.halo_lo))
            ops.append(dist.P2POp(dist.irecv, buf, rank - 1, group))
    if rank + 1 < world:
        down = lays[rank + 1]
        if down.halo_lo > 0:  # my last rows are the next rank's upper halo
            keep.append(pack(me.q_row_end - down.halo_lo, me.q_row_end))
            ops.append(dist.P2POp(dist.isend, keep[-1], rank + 1, group))
        if me.halo_hi > 0:
            buf = buffer(me.halo_hi)
            recvs.append((buf, me.q_row_end, me.q_row_end + me.halo_hi))
            ops.append(dist.P2POp(dist.irecv, buf, rank + 1, group))
    if ops:
        for work in dist.batch_isend_irecv(ops):
            work.wait()
    for buf, row_begin, row_end in recvs:
        sl = me.token_range(row_begin, row_end)
        k[:, :, sl] = buf[0]
        v[:, :, sl] = buf[1]


def gather_records(records: torch.Tensor, world: int, group=None) -> torch.Tensor:
    """[B * H, n_text, d + 2] of every rank -> [world, B * H, n_text, d + 2] on every rank."""
    out = torch.empty((world,) + tuple(records.shape), dtype=records.dtype, device=records.device)
    if world == 1:
        out[0] = records
    else:
        # concatenation along the first axis: rank p's records land in out[p]
        dist.all_gather_into_tensor(out.view((world * records.shape[0],) + tuple(records.shape[1:])), records.contiguous(),
                                    group=group)
    return out


class BandAttention:
    """The operator on one rank of a row-band parallel run."""

    def __init__(self, B, H, grid_h, grid_w, n_text, head_dim, radius, rank, world, group=None, text_mode="exact",
                 mask_kind=clear.MASK_DISC):
        if text_mode not in ("exact", "average"):
            raise ValueError("text_mode is 'exact' or 'average' (Eq. 7)")
        self.rank, self.world, self.group = rank, world, group
        self.lays = all_layouts(grid_h, grid_w, n_text, radius, world, mask_kind)
        self.lay = lay = self.lays[rank]
        self.n_text, self.B, self.H, self.d = n_text, B, H, head_dim
        self.mode = clear.TEXT_MERGE_EXACT if text_mode == "exact" else clear.TEXT_MERGE_AVERAGE
        self.image_plan = clear.BandPlan(B, H, lay.local_rows, grid_w, n_text, head_dim, radius, clear.PART_BAND_IMAGE,
                                         lay.q_row_begin, lay.q_row_end, mask_kind=mask_kind)
        self.text_plan = None
        if n_text > 0:
            # the text keys count once in the exact merge (on rank 0), on every rank in Eq. 7's average
            text_keys = rank == 0 or text_mode == "average"
            self.text_plan = clear.BandPlan(B, H, lay.local_rows, grid_w, n_text, head_dim, radius, clear.PART_BAND_TEXT,
                                            lay.q_row_begin, lay.q_row_end, text_keys=text_keys, mask_kind=mask_kind)
        self._records = None

    def forward(self, q, k, v, out, scale, exchange=True):
        """q, k, v, out: this rank's local bf16 tensors.  K and V need only hold the text and band rows on entry
        (``exchange=True`` fills the halo rows); ``out`` gets the band's image rows and every text row."""
        if exchange and self.world > 1:
            exchange_halos(k, v, self.lays, self.rank, self.group)
        self.image_plan.forward(q, k, v, out, scale)
        if self.text_plan is not None:
            if self._records is None:
                self._records = torch.empty(self.B * self.H, self.n_text, self.d + 2, dtype=torch.float32, device=q.device)
            self.text_plan.text_partial(q, k, v, self._records, scale)
            gathered = gather_records(self._records, self.world, self.group)
            clear.clear_text_merge(gathered, out, self.n_text, self.mode)
        return out

    def check(self):
        self.image_plan.check()
        if self.text_plan is not None:
            self.text_plan.check()
