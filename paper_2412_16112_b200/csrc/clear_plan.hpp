// Host-side schedule of the CLEAR attention kernels (no CUDA in this header).
#pragma once

#include <cstdint>
#include <vector>

#include "clear_attn.h"

namespace clear {

constexpr int kTileH = 8;      // query / key patch: 8 grid rows ...
constexpr int kTileW = 16;     // ... by 16 grid columns = 128 tokens
constexpr int kTileTokens = 128;
constexpr int kSplitTargetTiles = 64;  // key tiles per split of a text-query tile
constexpr int kMaxMaskEntries = 512;   // relative patch offsets with a precomputed mask (2 KB each)

struct Shape {
    int B = 0, H = 0, grid_h = 0, grid_w = 0, n_text = 0, head_dim = 0;
    float radius = 0.f;
    int dtype = 0;
    int kernel = 0;
    int mask_kind = 0;  // CLEAR_MASK_*: `radius` is r of the disc / square, the window size, or the stride
    int mask_param = 0; // CLEAR_MASK_WINDOWS: shift of the window grid; CLEAR_MASK_STRIDED: layer index
    // Row-band parallel form (Sec. 3.4): the grid of this shape is a band of image rows with the halo rows around
    // it; `part` selects what the plan computes of it (CLEAR_PART_*).
    int part = 0;
    int q_row_begin = 0, q_row_end = 0;  // rows of the band inside the grid (band parts only)
    int text_keys = 1;                   // CLEAR_PART_BAND_TEXT: are the text tokens among the keys
    int no_text_split = 0;               // tile schedule: one item per text tile over all its keys (backward pass)
    bool operator==(const Shape &o) const
    {
        return B == o.B && H == o.H && grid_h == o.grid_h && grid_w == o.grid_w && n_text == o.n_text &&
               head_dim == o.head_dim && radius == o.radius && dtype == o.dtype && kernel == o.kernel &&
               mask_kind == o.mask_kind && mask_param == o.mask_param && part == o.part && q_row_begin == o.q_row_begin &&
               q_row_end == o.q_row_end && text_keys == o.text_keys && no_text_split == o.no_text_split;
    }
};

struct Schedule {
    int64_t thr = 0;                     // ceil(radius^2): the disc allows dx^2 + dy^2 < thr (Eq. 3)
    std::vector<int32_t> half_width;     // half_width[dy] = max |dx| allowed at row offset dy (the window, whatever its kind)
    std::vector<clear_work_item_t> items;
    std::vector<clear_kv_tile_t> tiles;
    std::vector<clear_pair_item_t> pair_items;   // TCGEN05_WS: text items first, then image items
    std::vector<clear_pair_step_t> pair_steps;
    int n_text_pair_items = 0;
    bool pair_overflow = false;                  // an item stages more tiles than its 16-bit positions can name
    std::vector<uint32_t> mask_table;            // TCGEN05_WS: [entry][128 query rows][4 words]
    int n_text_tiles = 0;                // text-query tiles of 128 rows
    int n_text_splits = 0;               // splits per text-query tile (1 = no partial results)
    int n_partial_slots = 0;
    int max_item_tiles = 0;
    int64_t sum_mask = 0;
    int64_t executed_pairs = 0;
};

// Largest row offset |dy| at which the window lets an image query see a key on an unbounded grid (capped at 2^20).
int64_t window_reach(float radius, int mask_kind);

// Validate the arguments every entry point shares.  Returns a clear_status.
int validate_shape(const Shape &s);

// Integer geometry common to both kernels: thr, half_width[], sum_mask.
void build_geometry(const Shape &s, Schedule &sch);

// Work items and key-tile lists of the tensor-core kernel (calls build_geometry first).
void build_tile_schedule(const Shape &s, Schedule &sch);

// Pair items and step lists of the warp-specialised tensor-core kernel (calls build_geometry first).
void build_pair_schedule(const Shape &s, Schedule &sch);

}  // namespace clear
