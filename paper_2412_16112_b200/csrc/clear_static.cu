// clear_attn_fwd_static: the tensor-core forward pass for callers that must not allocate device memory.
//
// Everything the planned path keeps in cudaMalloc'ed buffers -- the schedule tables, the status word and
// the split-KV partial results of the text-query rows -- lives here in ONE file-scope device array of fixed
// size.  The array is part of the library image: every GPU that loads the library holds it until exit.
#include <cmath>
#include <cstring>
#include <mutex>

#include "clear_internal.hpp"

namespace clear {
namespace {

// layout of the array: [status | half_width | items | tiles | partial (m, l) | partial O]
constexpr size_t kOffStatus = 0;
constexpr size_t kOffHalfWidth = 256;
constexpr size_t kOffItems = kOffHalfWidth + (size_t)CLEAR_STATIC_MAX_HALF_WIDTH * sizeof(int32_t);
constexpr size_t kOffTiles = kOffItems + (size_t)CLEAR_STATIC_MAX_ITEMS * sizeof(clear_work_item_t);
constexpr size_t kOffPartial = kOffTiles + (size_t)CLEAR_STATIC_MAX_TILES * sizeof(clear_kv_tile_t);
constexpr size_t kStaticBytes = kOffPartial + (size_t)CLEAR_STATIC_SCRATCH_BYTES;
static_assert(kOffItems % 256 == 0 && kOffTiles % 256 == 0 && kOffPartial % 256 == 0, "sections stay 256-byte aligned");

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
struct StaticState {
    std::mutex mutex;
    unsigned char *base = nullptr;  // device address of g_static_scratch on this device
    bool have_tables = false;       // the tables in the array belong to plan.shape
    clear_plan plan;                // host-side schedule + tensor-map cache; its d_* point into the array
};
StaticState g_state[kMaxDevices];

}  // namespace
}  // namespace clear

using namespace clear;

extern "C" int clear_attn_fwd_static(const void *q, const void *k, const void *v, void *out, int B, int H, int grid_h,
                                     int grid_w, int n_text, int head_dim, float radius, float scale, void *stream)
{
    Shape s{B, H, grid_h, grid_w, n_text, head_dim, radius, CLEAR_BF16, CLEAR_KERNEL_TCGEN05};
    int rc = validate_shape(s);
    if (rc != CLEAR_OK) return rc;
    if (!std::isfinite(scale)) return CLEAR_ERR_INVALID_ARG;
    if (!(scale > 0.f)) return CLEAR_ERR_UNSUPPORTED;
    if (!q || !k || !v || !out) return CLEAR_ERR_INVALID_ARG;
    if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15u) return CLEAR_ERR_MISALIGNED;
    int dev = -1;
    CLEAR_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CLEAR_ERR_UNSUPPORTED;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);

    StaticState &st = g_state[dev];
    std::lock_guard<std::mutex> lock(st.mutex);
    if (!st.base) {
        // Set-up, once per device, with that device current.  In host code the array's name is only a
        // stand-in for the symbol; the address a kernel can use comes from the runtime.
        unsigned char *ptr = nullptr;
        CLEAR_CUDA_TRY(cudaGetSymbolAddress((void **)&ptr, g_static_scratch));
        if (!ptr) return CLEAR_ERR_CUDA;
        st.base = ptr;
    }
    clear_plan &p = st.plan;
    if (!(st.have_tables && p.shape == s)) {
        // new shape: rebuild the schedule on the host and check it against the fixed capacities
        st.have_tables = false;
        p.tm_valid = false;
        try {
            build_tile_schedule(s, p.sch);
        } catch (const std::bad_alloc &) {
            return CLEAR_ERR_NO_MEMORY;
        }
        const int64_t rows = (int64_t)s.B * s.H * p.sch.n_partial_slots * kTileTokens;
        const int64_t partial_bytes = rows * (s.head_dim + 2) * (int64_t)sizeof(float);
        if ((int64_t)p.sch.items.size() > CLEAR_STATIC_MAX_ITEMS || (int64_t)p.sch.tiles.size() > CLEAR_STATIC_MAX_TILES ||
            (int64_t)p.sch.half_width.size() > CLEAR_STATIC_MAX_HALF_WIDTH || partial_bytes > (int64_t)CLEAR_STATIC_SCRATCH_BYTES)
            return CLEAR_ERR_TOO_LARGE;
        p.shape = s;
        p.kernel = CLEAR_KERNEL_TCGEN05;
        p.host_only = false;
        p.device = dev;
        p.workspace_bytes = partial_bytes;
        p.d_status = reinterpret_cast<int *>(st.base + kOffStatus);
        p.d_half_width = reinterpret_cast<int32_t *>(st.base + kOffHalfWidth);
        p.d_items = reinterpret_cast<clear_work_item_t *>(st.base + kOffItems);
        p.d_tiles = reinterpret_cast<clear_kv_tile_t *>(st.base + kOffTiles);
        p.d_partial_ml = reinterpret_cast<float *>(st.base + kOffPartial);
        p.d_partial_o = reinterpret_cast<float *>(st.base + kOffPartial + (size_t)rows * 2 * sizeof(float));
        // stream-ordered upload of the tables (pageable source: staged before the call returns)
        CLEAR_CUDA_TRY(cudaMemcpyAsync(p.d_half_width, p.sch.half_width.data(), p.sch.half_width.size() * sizeof(int32_t),
                                       cudaMemcpyHostToDevice, cs));
        CLEAR_CUDA_TRY(cudaMemcpyAsync(p.d_items, p.sch.items.data(), p.sch.items.size() * sizeof(clear_work_item_t),
                                       cudaMemcpyHostToDevice, cs));
        CLEAR_CUDA_TRY(cudaMemcpyAsync(p.d_tiles, p.sch.tiles.data(), p.sch.tiles.size() * sizeof(clear_kv_tile_t),
                                       cudaMemcpyHostToDevice, cs));
        st.have_tables = true;
    }
    // The array keeps the previous call's contents.  Only the status word has to start at zero (a non-zero
    // word makes every CTA leave at once); each partial row that is read is written first by this call.
    CLEAR_CUDA_TRY(cudaMemsetAsync(p.d_status, 0, sizeof(int), cs));
    return launch_tc(p, q, k, v, out, scale, cs);
}
