// Host-side schedule of the CLEAR attention kernels: Eq. 3 turned into integer geometry,
// the 2-D tile-pair lists, the split of the text-query rows and the work order.
#include "clear_plan.hpp"

#include <algorithm>
#include <cmath>
#include <climits>
#include <cstdlib>
#include <map>
#include <utility>

namespace clear {

static int64_t isqrt64(int64_t v)
{
    if (v <= 0) return 0;
    int64_t r = (int64_t)std::sqrt((double)v);
    while (r * r > v) --r;
    while ((r + 1) * (r + 1) <= v) ++r;
    return r;
}

int64_t window_reach(float radius, int mask_kind)
{
    const double r = (double)radius;
    if (!(r < 1048576.0)) return 1048576;
    if (mask_kind == CLEAR_MASK_SQUARE) return (int64_t)std::ceil(r) - 1;
    return isqrt64((int64_t)std::ceil(r * r) - 1);
}

int validate_shape(const Shape &s)
{
    if (s.B <= 0 || s.H <= 0 || s.grid_h <= 0 || s.grid_w <= 0 || s.n_text < 0 || s.head_dim <= 0)
        return CLEAR_ERR_INVALID_ARG;
    if (!(s.radius > 0.f) || !std::isfinite(s.radius)) return CLEAR_ERR_INVALID_ARG;
    if (s.dtype != CLEAR_BF16 && s.dtype != CLEAR_F32) return CLEAR_ERR_INVALID_ARG;
    if (s.kernel < CLEAR_KERNEL_AUTO || s.kernel > CLEAR_KERNEL_TCGEN05_WS) return CLEAR_ERR_INVALID_ARG;
    if (s.mask_kind < CLEAR_MASK_DISC || s.mask_kind > CLEAR_MASK_STRIDED) return CLEAR_ERR_INVALID_ARG;
    if (s.mask_kind == CLEAR_MASK_WINDOWS || s.mask_kind == CLEAR_MASK_STRIDED) {
        // window size / stride: a whole number of grid cells; shift / layer index: not negative
        if (s.radius < 1.f || s.radius != std::floor(s.radius) || s.radius > 1048576.f || s.mask_param < 0)
            return CLEAR_ERR_INVALID_ARG;
        // masks that are no window around the query run on the CUDA-core kernel only, and not as band parts
        if (s.kernel != CLEAR_KERNEL_AUTO && s.kernel != CLEAR_KERNEL_SIMT) return CLEAR_ERR_UNSUPPORTED;
        if (s.part != CLEAR_PART_ALL) return CLEAR_ERR_UNSUPPORTED;
    } else if (s.mask_param != 0) {
        return CLEAR_ERR_INVALID_ARG;
    }
    if (s.part != CLEAR_PART_ALL) {
        if (s.part != CLEAR_PART_BAND_IMAGE && s.part != CLEAR_PART_BAND_TEXT) return CLEAR_ERR_INVALID_ARG;
        if (s.q_row_begin < 0 || s.q_row_end <= s.q_row_begin || s.q_row_end > s.grid_h) return CLEAR_ERR_INVALID_ARG;
        if (s.part == CLEAR_PART_BAND_TEXT && s.n_text <= 0) return CLEAR_ERR_INVALID_ARG;
        // band parts exist for the warp-specialised tensor-core kernel only
        if (s.kernel != CLEAR_KERNEL_AUTO && s.kernel != CLEAR_KERNEL_TCGEN05_WS) return CLEAR_ERR_UNSUPPORTED;
        if (s.dtype != CLEAR_BF16 || (s.head_dim != 64 && s.head_dim != 128)) return CLEAR_ERR_UNSUPPORTED;
    }
    const int64_t n = (int64_t)s.grid_h * s.grid_w;
    const int64_t N = n + s.n_text;
    if (N > (int64_t)1 << 30) return CLEAR_ERR_UNSUPPORTED;  // token indices stay in int32
    if ((int64_t)s.B * s.H > 65535) return CLEAR_ERR_UNSUPPORTED;  // (batch, head) is a grid's y axis
    if (s.head_dim > 256) return CLEAR_ERR_UNSUPPORTED;
    // 16-byte rows keep every per-token vector access and TMA stride aligned
    const int esz = s.dtype == CLEAR_BF16 ? 2 : 4;
    if ((s.head_dim * esz) % 16 != 0) return CLEAR_ERR_UNSUPPORTED;
    if (s.kernel == CLEAR_KERNEL_TCGEN05 || s.kernel == CLEAR_KERNEL_TCGEN05_WS) {
        if (s.dtype != CLEAR_BF16) return CLEAR_ERR_UNSUPPORTED;
        if (s.head_dim != 64 && s.head_dim != 128) return CLEAR_ERR_UNSUPPORTED;
    }
    return CLEAR_OK;
}

// Allowed (query, key) pairs along one axis of `len` cells for the two masks that factor over the axes.
static int64_t axis_pairs(const Shape &s, int64_t len, bool y_axis)
{
    const int64_t a = (int64_t)s.radius;
    int64_t pairs = 0;
    if (s.mask_kind == CLEAR_MASK_WINDOWS) {
        // cells c with the same floor((c + shift) / w) share a window: segments of the axis, squared
        const int64_t shift = s.mask_param;
        int64_t c = 0;
        while (c < len) {
            const int64_t end = std::min(len, ((c + shift) / a + 1) * a - shift);
            pairs += (end - c) * (end - c);
            c = end;
        }
    } else {
        // strided: key = query + offset (mod stride), offset = layer % stride (x) or (layer / stride) % stride (y)
        const int64_t off = y_axis ? (s.mask_param / a) % a : s.mask_param % a;
        for (int64_t c = 0; c < len; ++c) {
            const int64_t first = (c + off) % a;  // smallest cell congruent to c + off
            if (first < len) pairs += (len - 1 - first) / a + 1;
        }
    }
    return pairs;
}

void build_geometry(const Shape &s, Schedule &sch)
{
    const int64_t gh = s.grid_h, gw = s.grid_w, T = s.n_text;
    const int64_t n = gh * gw, N = n + T;
    if (s.mask_kind == CLEAR_MASK_WINDOWS || s.mask_kind == CLEAR_MASK_STRIDED) {
        // no window around the query: no half widths; the mask factors into a row rule and a column rule
        sch.thr = 0;
        sch.half_width.clear();
        sch.sum_mask = T * N + n * T + axis_pairs(s, gh, true) * axis_pairs(s, gw, false);
        return;
    }
    // Eq. 3 with integer squared distances: d2 < r^2  <=>  d2 < ceil(r^2).  No pair on the grid
    // is farther apart than its diagonal, so the threshold is capped just above it.
    const double r = (double)s.radius;
    const double r2 = std::ceil(r * r);
    const int64_t diag2 = (gh - 1) * (gh - 1) + (gw - 1) * (gw - 1);
    sch.thr = (r2 > (double)(diag2 + 1)) ? diag2 + 1 : (int64_t)r2;

    // The window as half widths per row offset: the open disc of Eq. 3, or the square window of Neighborhood
    // Attention (Sec. 3.2 sets the disc against it), max(|dx|, |dy|) < r, i.e. |dx|, |dy| <= ceil(r) - 1.
    const int64_t reach = s.mask_kind == CLEAR_MASK_SQUARE ? (int64_t)std::ceil(r) - 1 : isqrt64(sch.thr - 1);
    const int64_t R = std::min<int64_t>(reach, gh - 1);  // largest |dy| that still has keys
    sch.half_width.assign((size_t)R + 1, 0);
    int64_t img_img = 0;
    for (int64_t dy = 0; dy <= R; ++dy) {
        const int64_t m = std::min<int64_t>(s.mask_kind == CLEAR_MASK_SQUARE ? reach : isqrt64(sch.thr - 1 - dy * dy), gw - 1);
        sch.half_width[(size_t)dy] = (int32_t)m;
        // keys in row y+dy seen by the gw queries of row y: sum_x (min(x+m, gw-1) - max(x-m, 0) + 1)
        const int64_t row_pairs = gw * (2 * m + 1) - m * (m + 1);
        const int64_t rows = gh - dy;  // query rows y for which y + dy is on the grid
        img_img += (dy == 0 ? 1 : 2) * rows * row_pairs;
    }
    sch.sum_mask = T * N + n * T + img_img;
}

// The window of the schedule as a predicate on offsets: (dy, dx) is allowed iff |dx| <= half_width[|dy|].  The half
// widths do not grow with |dy| (disc and square alike), so of two axis-aligned boxes of offsets SOME pair is allowed
// iff the nearest one is, and EVERY pair iff the farthest one is.
static bool window_allows(const Schedule &sch, int64_t dy, int64_t dx)
{
    dy = dy < 0 ? -dy : dy;
    dx = dx < 0 ? -dx : dx;
    return dy < (int64_t)sch.half_width.size() && dx <= sch.half_width[(size_t)dy];
}

void build_tile_schedule(const Shape &s, Schedule &sch)
{
    build_geometry(s, sch);
    const int gh = s.grid_h, gw = s.grid_w, T = s.n_text;
    const int64_t N = (int64_t)gh * gw + T;
    const int R = (int)sch.half_width.size() - 1;  // rows a window reaches up and down

    sch.items.clear();
    sch.tiles.clear();

    // ---- text-query tiles: dense over all N keys, split over key ranges ------------------------
    const int n_lin = (int)((N + kTileTokens - 1) / kTileTokens);
    sch.n_text_tiles = (T + kTileTokens - 1) / kTileTokens;
    int chunk = n_lin, n_splits = 1;
    if (sch.n_text_tiles > 0 && !s.no_text_split) {
        n_splits = (n_lin + kSplitTargetTiles - 1) / kSplitTargetTiles;
        chunk = (n_lin + n_splits - 1) / n_splits;
        n_splits = (n_lin + chunk - 1) / chunk;
    }
    sch.n_text_splits = sch.n_text_tiles > 0 ? n_splits : 0;
    sch.n_partial_slots = (sch.n_text_tiles > 0 && n_splits > 1) ? sch.n_text_tiles * n_splits : 0;
    for (int tq = 0; tq < sch.n_text_tiles; ++tq) {
        for (int sp = 0; sp < n_splits; ++sp) {
            clear_work_item_t it{};
            it.kind = 1;
            it.qx = tq * kTileTokens;
            it.qy = 0;
            it.n_rows = std::min(kTileTokens, T - it.qx);
            it.tile_begin = (int32_t)sch.tiles.size();
            const int t0 = sp * chunk, t1 = std::min(n_lin, t0 + chunk);
            for (int t = t0; t < t1; ++t) {
                clear_kv_tile_t kt{};
                kt.x = t * kTileTokens;
                kt.y = 0;
                kt.n_valid = (int32_t)std::min<int64_t>(kTileTokens, N - (int64_t)kt.x);
                kt.flags = CLEAR_TILE_LINEAR | (kt.n_valid < kTileTokens ? CLEAR_TILE_MASKED : 0);
                sch.tiles.push_back(kt);
            }
            it.tile_count = t1 - t0;
            it.partial_slot = n_splits > 1 ? tq * n_splits + sp : -1;
            sch.items.push_back(it);
        }
    }

    // ---- image-query patches: text tiles, then the key patches that meet the dilated patch -----
    const int ntx = (gw + kTileW - 1) / kTileW, nty = (gh + kTileH - 1) / kTileH;
    const int reach_x = sch.half_width[0] / kTileW + 1, reach_y = R / kTileH + 1;
    for (int ty = 0; ty < nty; ++ty) {
        for (int tx = 0; tx < ntx; ++tx) {
            clear_work_item_t it{};
            it.kind = 0;
            it.qx = tx * kTileW;
            it.qy = ty * kTileH;
            const int qx1 = std::min(it.qx + kTileW - 1, gw - 1), qy1 = std::min(it.qy + kTileH - 1, gh - 1);
            it.n_rows = (qx1 - it.qx + 1) * (qy1 - it.qy + 1);
            it.tile_begin = (int32_t)sch.tiles.size();
            for (int t0 = 0; t0 < T; t0 += kTileTokens) {
                clear_kv_tile_t kt{};
                kt.x = t0;
                kt.y = 0;
                kt.n_valid = std::min(kTileTokens, T - t0);  // tokens past n_text are image keys: not allowed here
                kt.flags = CLEAR_TILE_LINEAR | (kt.n_valid < kTileTokens ? CLEAR_TILE_MASKED : 0);
                sch.tiles.push_back(kt);
            }
            for (int j = std::max(0, ty - reach_y); j <= std::min(nty - 1, ty + reach_y); ++j) {
                for (int i = std::max(0, tx - reach_x); i <= std::min(ntx - 1, tx + reach_x); ++i) {
                    const int bx = i * kTileW, by = j * kTileH;
                    const int kx1 = std::min(bx + kTileW - 1, gw - 1), ky1 = std::min(by + kTileH - 1, gh - 1);
                    // smallest and largest coordinate differences between the two (clipped) patches
                    const int64_t gx = std::max({0, bx - qx1, it.qx - kx1});
                    const int64_t gy = std::max({0, by - qy1, it.qy - ky1});
                    if (!window_allows(sch, gy, gx)) continue;
                    const int64_t fx = std::max(kx1 - it.qx, qx1 - bx);
                    const int64_t fy = std::max(ky1 - it.qy, qy1 - by);
                    const bool whole = (bx + kTileW <= gw) && (by + kTileH <= gh);
                    clear_kv_tile_t kt{};
                    kt.x = bx;
                    kt.y = by;
                    kt.n_valid = kTileTokens;
                    kt.flags = (whole && window_allows(sch, fy, fx)) ? 0 : CLEAR_TILE_MASKED;
                    sch.tiles.push_back(kt);
                }
            }
            it.tile_count = (int32_t)sch.tiles.size() - it.tile_begin;
            it.partial_slot = -1;
            sch.items.push_back(it);
        }
    }

    // ---- work order: longest lists first (the block scheduler hands items out in this order, so
    // the short border patches fill the tail); stable, so equal items keep their raster order
    std::stable_sort(sch.items.begin(), sch.items.end(),
                     [](const clear_work_item_t &a, const clear_work_item_t &b) { return a.tile_count > b.tile_count; });

    sch.max_item_tiles = 0;
    sch.executed_pairs = 0;
    for (const auto &it : sch.items) {
        sch.max_item_tiles = std::max(sch.max_item_tiles, it.tile_count);
        sch.executed_pairs += (int64_t)it.tile_count * kTileTokens * kTileTokens;
    }
}

// ---- pair schedule of the warp-specialised kernel ------------------------------------------------
namespace {

struct PatchTile {
    int x, y;
    bool masked;
    bool clipped;  // part of the patch lies outside the grid
};

// Key patches (on the 8 x 16 lattice) that hold at least one key allowed to some query of the patch
// at (qx, qy), each with the flag "some pair of the tile is not allowed".
std::vector<PatchTile> patches_of(const Shape &s, const Schedule &sch, int R, int qx, int qy)
{
    const int gh = s.grid_h, gw = s.grid_w;
    const int ntx = (gw + kTileW - 1) / kTileW, nty = (gh + kTileH - 1) / kTileH;
    const int tx = qx / kTileW, ty = qy / kTileH;
    const int reach_x = sch.half_width[0] / kTileW + 1, reach_y = R / kTileH + 1;
    const int qx1 = std::min(qx + kTileW - 1, gw - 1), qy1 = std::min(qy + kTileH - 1, gh - 1);
    std::vector<PatchTile> out;
    for (int j = std::max(0, ty - reach_y); j <= std::min(nty - 1, ty + reach_y); ++j) {
        for (int i = std::max(0, tx - reach_x); i <= std::min(ntx - 1, tx + reach_x); ++i) {
            const int bx = i * kTileW, by = j * kTileH;
            const int kx1 = std::min(bx + kTileW - 1, gw - 1), ky1 = std::min(by + kTileH - 1, gh - 1);
            const int64_t gx = std::max({0, bx - qx1, qx - kx1});
            const int64_t gy = std::max({0, by - qy1, qy - ky1});
            if (!window_allows(sch, gy, gx)) continue;
            const int64_t fx = std::max(kx1 - qx, qx1 - bx);
            const int64_t fy = std::max(ky1 - qy, qy1 - by);
            const bool whole = (bx + kTileW <= gw) && (by + kTileH <= gh);
            out.push_back(PatchTile{bx, by, !(whole && window_allows(sch, fy, fx)), !whole});
        }
    }
    return out;
}

}  // namespace

void build_pair_schedule(const Shape &s, Schedule &sch)
{
    build_geometry(s, sch);
    const int gh = s.grid_h, gw = s.grid_w, T = s.n_text;
    const int64_t N = (int64_t)gh * gw + T;
    const int R = (int)sch.half_width.size() - 1;  // rows a window reaches up and down
    if (s.part == CLEAR_PART_BAND_IMAGE) {
        // allowed pairs of the band's image queries: the text keys, and per row offset the closed form
        // sum_x (min(x+m, gw-1) - max(x-m, 0) + 1) for the rows that are on this grid
        int64_t pairs = 0;
        for (int64_t y = s.q_row_begin; y < s.q_row_end; ++y) {
            pairs += (int64_t)gw * T;
            for (int64_t dy = -R; dy <= R; ++dy) {
                if (y + dy < 0 || y + dy >= gh) continue;
                const int64_t m = sch.half_width[(size_t)(dy < 0 ? -dy : dy)];
                pairs += (int64_t)gw * (2 * m + 1) - m * (m + 1);
            }
        }
        sch.sum_mask = pairs;
    } else if (s.part == CLEAR_PART_BAND_TEXT) {
        sch.sum_mask = (int64_t)T * ((s.text_keys ? T : 0) + (int64_t)(s.q_row_end - s.q_row_begin) * gw);
    }

    sch.pair_items.clear();
    sch.pair_steps.clear();
    sch.mask_table.clear();
    sch.pair_overflow = false;

    // Eq. 3 for a key patch at offset (dy, dx) from a query patch, once per distinct offset
    // (CLEAR_MAX_MASK_ENTRIES lowers the cap of the table; with 0 every masked patch takes the kernel's
    // table-free path, which is otherwise reached only by very large radii)
    int max_entries = kMaxMaskEntries;
    if (const char *e = std::getenv("CLEAR_MAX_MASK_ENTRIES")) max_entries = std::max(0, std::min(kMaxMaskEntries, std::atoi(e)));
    std::map<std::pair<int, int>, int> mask_ids;
    auto mask_entry = [&](int dy, int dx) -> int {
        auto it = mask_ids.find({dy, dx});
        if (it != mask_ids.end()) return it->second;
        if ((int)mask_ids.size() >= max_entries) return -1;
        const int id = (int)mask_ids.size();
        mask_ids[{dy, dx}] = id;
        sch.mask_table.resize((size_t)(id + 1) * kTileTokens * 4, 0u);
        uint32_t *e = sch.mask_table.data() + (size_t)id * kTileTokens * 4;
        for (int r = 0; r < kTileTokens; ++r) {
            const int qy = r / kTileW, qx = r % kTileW;
            for (int j = 0; j < kTileTokens; ++j) {
                const int64_t ddy = dy + j / kTileW - qy, ddx = dx + j % kTileW - qx;
                if (window_allows(sch, ddy, ddx)) e[r * 4 + (j >> 5)] |= 1u << (j & 31);
            }
        }
        return id;
    };

    auto finish_item = [&](clear_pair_item_t &it) {
        // staging order: for every step its K tiles, then its V tiles (the order the MMAs read them in)
        auto n_tiles = [&](int32_t i) {
            const clear_pair_step_t &st = sch.pair_steps[(size_t)i];
            const int a = (st.flags & CLEAR_STEP_USE0) ? 1 : 0;
            const int b = ((st.flags & CLEAR_STEP_USE1) && !(st.flags & CLEAR_STEP_SHARED)) ? 1 : 0;
            return a + b;
        };
        const int32_t first = it.step_begin, end = (int32_t)sch.pair_steps.size();
        int64_t pos = 0;
        for (int32_t i = first; i < end; ++i) {
            const int64_t k_pos = pos, v_pos = pos + n_tiles(i);
            pos = v_pos + n_tiles(i);
            // positions travel in 16 bits each
            if (pos > 0xffff) sch.pair_overflow = true;
            sch.pair_steps[(size_t)i].load_base = (int32_t)((k_pos & 0xffff) | ((v_pos & 0xffff) << 16));
        }
        it.step_count = end - first;
        it.n_loads = (int32_t)std::min<int64_t>(pos, INT_MAX);
        sch.pair_items.push_back(it);
    };
    auto linear_step = [&](int x, int n_valid, int n_sides) {
        clear_pair_step_t st{};
        st.x0 = st.x1 = x;
        st.n_valid0 = st.n_valid1 = n_valid;
        st.flags = CLEAR_STEP_LINEAR | CLEAR_STEP_USE0;
        if (n_valid < kTileTokens) st.flags |= CLEAR_STEP_MASKED0;
        if (n_sides == 2) {
            st.flags |= CLEAR_STEP_USE1 | CLEAR_STEP_SHARED;
            if (n_valid < kTileTokens) st.flags |= CLEAR_STEP_MASKED1;
        }
        sch.pair_steps.push_back(st);
    };

    // ---- text-query tiles, two per item, dense over their keys, split over key ranges ----------
    // The keys of a text query as runs of tokens: all N of them; for the text part of a band, the text tokens
    // (if this band counts them) and the image tokens of the band's own rows.
    std::vector<std::pair<int64_t, int64_t>> key_runs;
    if (s.part == CLEAR_PART_ALL) {
        key_runs.push_back({0, N});
    } else if (s.part == CLEAR_PART_BAND_TEXT) {
        if (s.text_keys) key_runs.push_back({0, T});
        key_runs.push_back({T + (int64_t)s.q_row_begin * gw, T + (int64_t)s.q_row_end * gw});
    }
    std::vector<std::pair<int, int>> lin_tiles;  // first token, tokens that count
    for (const auto &run : key_runs)
        for (int64_t t0 = run.first; t0 < run.second; t0 += kTileTokens)
            lin_tiles.push_back({(int)t0, (int)std::min<int64_t>(kTileTokens, run.second - t0)});
    const int n_lin = (int)lin_tiles.size();
    sch.n_text_tiles = n_lin > 0 ? (T + kTileTokens - 1) / kTileTokens : 0;
    int chunk = n_lin, n_splits = 1;
    if (sch.n_text_tiles > 0) {
        n_splits = (n_lin + kSplitTargetTiles - 1) / kSplitTargetTiles;
        chunk = (n_lin + n_splits - 1) / n_splits;
        n_splits = (n_lin + chunk - 1) / chunk;
    }
    // the text part of a band always leaves partial results (they are merged with the other bands')
    const bool partials = n_splits > 1 || s.part == CLEAR_PART_BAND_TEXT;
    sch.n_text_splits = sch.n_text_tiles > 0 ? n_splits : 0;
    sch.n_partial_slots = (sch.n_text_tiles > 0 && partials) ? sch.n_text_tiles * n_splits : 0;
    // key range outermost: the items that stream one key range sit next to each other in the queue
    for (int sp = 0; sp < n_splits && sch.n_text_tiles > 0; ++sp) {
        for (int tq = 0; tq < sch.n_text_tiles; tq += 2) {
            clear_pair_item_t it{};
            it.kind = 1;
            it.n_sides = (tq + 1 < sch.n_text_tiles) ? 2 : 1;
            it.qx = tq * kTileTokens;
            it.n_rows0 = std::min(kTileTokens, T - it.qx);
            it.n_rows1 = it.n_sides == 2 ? std::min(kTileTokens, T - it.qx - kTileTokens) : 0;
            it.step_begin = (int32_t)sch.pair_steps.size();
            const int t0 = sp * chunk, t1 = std::min(n_lin, t0 + chunk);
            for (int t = t0; t < t1; ++t) linear_step(lin_tiles[(size_t)t].first, lin_tiles[(size_t)t].second, it.n_sides);
            it.partial_slot0 = partials ? tq * n_splits + sp : -1;
            it.partial_slot1 = (partials && it.n_sides == 2) ? (tq + 1) * n_splits + sp : -1;
            finish_item(it);
        }
    }
    sch.n_text_pair_items = (int)sch.pair_items.size();

    // ---- image-query patches, two vertically adjacent ones per item ----------------------------
    // (of a band: the patches that hold rows of the band; rows of those patches outside the band are computed
    // and written too, which the caller of a band part is told)
    const int ntx = (gw + kTileW - 1) / kTileW;
    int ty_begin = 0, nty = (gh + kTileH - 1) / kTileH;
    if (s.part == CLEAR_PART_BAND_IMAGE) {
        ty_begin = s.q_row_begin / kTileH;
        nty = (s.q_row_end + kTileH - 1) / kTileH;
    } else if (s.part == CLEAR_PART_BAND_TEXT) {
        nty = 0;
    }
    for (int ty = ty_begin; ty < nty; ty += 2) {
        for (int tx = 0; tx < ntx; ++tx) {
            clear_pair_item_t it{};
            it.kind = 0;
            it.n_sides = (ty + 1 < nty) ? 2 : 1;
            it.qx = tx * kTileW;
            it.qy0 = ty * kTileH;
            it.qy1 = it.qy0 + kTileH;
            const int w = std::min(kTileW, gw - it.qx);
            it.n_rows0 = w * std::min(kTileH, gh - it.qy0);
            it.n_rows1 = it.n_sides == 2 ? w * std::min(kTileH, gh - it.qy1) : 0;
            it.partial_slot0 = it.partial_slot1 = -1;
            it.step_begin = (int32_t)sch.pair_steps.size();
            // text keys: tokens past n_text in the last tile are image keys, not allowed through it
            for (int t0 = 0; t0 < T; t0 += kTileTokens) linear_step(t0, std::min(kTileTokens, T - t0), it.n_sides);

            std::vector<PatchTile> a = patches_of(s, sch, R, it.qx, it.qy0), b;
            if (it.n_sides == 2) b = patches_of(s, sch, R, it.qx, it.qy1);
            auto find = [](const std::vector<PatchTile> &v, const PatchTile &t) -> const PatchTile * {
                for (const PatchTile &u : v)
                    if (u.x == t.x && u.y == t.y) return &u;
                return nullptr;
            };
            std::vector<PatchTile> only_a, only_b;
            std::vector<std::pair<PatchTile, PatchTile>> both;
            for (const PatchTile &t : a) {
                const PatchTile *u = find(b, t);
                if (u)
                    both.push_back({t, *u});
                else
                    only_a.push_back(t);
            }
            for (const PatchTile &t : b)
                if (!find(a, t)) only_b.push_back(t);
            // key patches only one tile needs are taken two at a time, one per tile, so that both
            // tiles stay busy; what is left over runs one-sided
            for (size_t i = 0; i < std::max(only_a.size(), only_b.size()); ++i) {
                clear_pair_step_t st{};
                st.n_valid0 = st.n_valid1 = kTileTokens;
                if (i < only_a.size()) {
                    st.x0 = only_a[i].x;
                    st.y0 = only_a[i].y;
                    st.flags |= CLEAR_STEP_USE0 | (only_a[i].masked ? CLEAR_STEP_MASKED0 : 0) |
                                (only_a[i].clipped ? CLEAR_STEP_CLIP0 : 0);
                    st.n_valid0 = only_a[i].masked ? mask_entry(st.y0 - it.qy0, st.x0 - it.qx) : -1;
                }
                if (i < only_b.size()) {
                    st.x1 = only_b[i].x;
                    st.y1 = only_b[i].y;
                    st.flags |= CLEAR_STEP_USE1 | (only_b[i].masked ? CLEAR_STEP_MASKED1 : 0) |
                                (only_b[i].clipped ? CLEAR_STEP_CLIP1 : 0);
                    st.n_valid1 = only_b[i].masked ? mask_entry(st.y1 - it.qy1, st.x1 - it.qx) : -1;
                }
                sch.pair_steps.push_back(st);
            }
            for (const auto &ab : both) {
                clear_pair_step_t st{};
                st.n_valid0 = st.n_valid1 = kTileTokens;
                st.x0 = st.x1 = ab.first.x;
                st.y0 = st.y1 = ab.first.y;
                st.flags = CLEAR_STEP_USE0 | CLEAR_STEP_USE1 | CLEAR_STEP_SHARED |
                           (ab.first.masked ? CLEAR_STEP_MASKED0 : 0) | (ab.second.masked ? CLEAR_STEP_MASKED1 : 0) |
                           (ab.first.clipped ? (CLEAR_STEP_CLIP0 | CLEAR_STEP_CLIP1) : 0);
                st.n_valid0 = ab.first.masked ? mask_entry(st.y0 - it.qy0, st.x0 - it.qx) : -1;
                st.n_valid1 = ab.second.masked ? mask_entry(st.y1 - it.qy1, st.x1 - it.qx) : -1;
                sch.pair_steps.push_back(st);
            }
            finish_item(it);
            // a list too long for the step records' 16-bit ring positions: this kernel cannot run the
            // shape, and the remaining lists (gigabytes at such radii) are not worth building
            if (sch.pair_overflow) return;
        }
    }

    // ---- work order: text items (the longest lists) first, then image items, longest first; the
    // blocks take items from the queue in this order, so the short border items fill the tail
    std::stable_sort(sch.pair_items.begin() + sch.n_text_pair_items, sch.pair_items.end(),
                     [](const clear_pair_item_t &x, const clear_pair_item_t &y) { return x.step_count > y.step_count; });

    sch.max_item_tiles = 0;
    sch.executed_pairs = 0;
    for (const auto &it : sch.pair_items) {
        sch.max_item_tiles = std::max(sch.max_item_tiles, it.step_count);
        for (int32_t i = 0; i < it.step_count; ++i) {
            const int f = sch.pair_steps[(size_t)(it.step_begin + i)].flags;
            const int uses = ((f & CLEAR_STEP_USE0) ? 1 : 0) + ((f & CLEAR_STEP_USE1) ? 1 : 0);
            sch.executed_pairs += (int64_t)uses * kTileTokens * kTileTokens;
        }
    }
}

}  // namespace clear
