// C ABI of the CLEAR attention library: argument checks, plans, plan cache, launches.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <list>
#include <memory>
#include <new>

#include "clear_internal.hpp"

namespace clear {

static thread_local int g_last_cuda_error = 0;
static thread_local int g_last_device_status = 0;
void note_cuda_error(int err) { g_last_cuda_error = err; }

namespace {

int select_kernel(const Shape &s)
{
    if (s.kernel != CLEAR_KERNEL_AUTO) return s.kernel;
    if (s.mask_kind == CLEAR_MASK_WINDOWS || s.mask_kind == CLEAR_MASK_STRIDED) return CLEAR_KERNEL_SIMT;
    if (s.dtype == CLEAR_BF16 && (s.head_dim == 64 || s.head_dim == 128)) return CLEAR_KERNEL_TCGEN05_WS;
    return CLEAR_KERNEL_SIMT;
}

template <typename T>
int upload(T **dst, const std::vector<T> &src)
{
    *dst = nullptr;
    if (src.empty()) return CLEAR_OK;
    CLEAR_CUDA_TRY(cudaMalloc((void **)dst, src.size() * sizeof(T)));
    CLEAR_CUDA_TRY(cudaMemcpy(*dst, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice));
    return CLEAR_OK;
}

int free_device_parts(clear_plan *p)
{
    int rc = CLEAR_OK;
    auto rel = [&](void *ptr) {
        if (ptr && cudaFree(ptr) != cudaSuccess) {
            (void)cudaGetLastError();
            rc = CLEAR_ERR_CUDA;
        }
    };
    rel(p->d_half_width);
    rel(p->d_items);
    rel(p->d_tiles);
    rel(p->d_pair_items);
    rel(p->d_pair_steps);
    rel(p->d_mask_table);
    rel(p->d_status);
    rel(p->d_partial_o);
    rel(p->d_partial_ml);
    rel(p->d_bwd_stats);
    if (p->ev_last) {
        (void)cudaEventDestroy(p->ev_last);
        p->ev_last = nullptr;
    }
    for (void *&s : p->d_stage) {
        rel(s);
        s = nullptr;
    }
    p->d_half_width = nullptr;
    p->d_items = nullptr;
    p->d_tiles = nullptr;
    p->d_pair_items = nullptr;
    p->d_pair_steps = nullptr;
    p->d_mask_table = nullptr;
    p->d_status = nullptr;
    p->d_partial_o = nullptr;
    p->d_partial_ml = nullptr;
    p->d_bwd_stats = nullptr;
    return rc;
}

int create_plan(clear_plan_t **out, const Shape &shape_in, bool host_only)
{
    if (!out) return CLEAR_ERR_INVALID_ARG;
    Shape s = shape_in;
    int rc = validate_shape(s);
    if (rc != CLEAR_OK) return rc;
    int kernel = select_kernel(s);
    {
        Shape chk = s;
        chk.kernel = kernel;
        rc = validate_shape(chk);
        if (rc != CLEAR_OK) return rc;
    }
    std::unique_ptr<clear_plan> p(new (std::nothrow) clear_plan());
    if (!p) return CLEAR_ERR_NO_MEMORY;
    p->shape = s;
    p->host_only = host_only;
    try {
        if (kernel == CLEAR_KERNEL_TCGEN05_WS) {
            build_pair_schedule(s, p->sch);
            // An item whose key-tile list outgrows the 16-bit ring positions of the step records (radii of
            // about a thousand tokens on grids of millions) cannot run on this kernel, and tile lists of
            // that length would take gigabytes: the CUDA-core kernel, which walks Eq. 3 without any list,
            // takes over when the choice was left to the library.
            if (p->sch.pair_overflow) {
                if (s.kernel != CLEAR_KERNEL_AUTO) return CLEAR_ERR_UNSUPPORTED;
                kernel = CLEAR_KERNEL_SIMT;
                p->sch = Schedule();
            }
        }
        if (kernel == CLEAR_KERNEL_TCGEN05)
            build_tile_schedule(s, p->sch);
        else if (kernel == CLEAR_KERNEL_SIMT)
            build_geometry(s, p->sch);
    } catch (const std::bad_alloc &) {
        return CLEAR_ERR_NO_MEMORY;
    }
    p->kernel = kernel;
    if (kernel != CLEAR_KERNEL_SIMT && p->sch.n_partial_slots > 0) {
        const int64_t rows = (int64_t)s.B * s.H * p->sch.n_partial_slots * kTileTokens;
        p->workspace_bytes = rows * (s.head_dim + 2) * (int64_t)sizeof(float);
    }
    if (!host_only) {
        CLEAR_CUDA_TRY(cudaGetDevice(&p->device));
        rc = upload(&p->d_half_width, p->sch.half_width);
        if (rc == CLEAR_OK) rc = upload(&p->d_items, p->sch.items);
        if (rc == CLEAR_OK) rc = upload(&p->d_tiles, p->sch.tiles);
        if (rc == CLEAR_OK) rc = upload(&p->d_pair_items, p->sch.pair_items);
        if (rc == CLEAR_OK) rc = upload(&p->d_pair_steps, p->sch.pair_steps);
        if (rc == CLEAR_OK) rc = upload(&p->d_mask_table, p->sch.mask_table);
        if (rc == CLEAR_OK) {
            cudaError_t e = cudaMalloc((void **)&p->d_status, kStatusWords * sizeof(int));
            if (e == cudaSuccess) e = cudaMemset(p->d_status, 0, kStatusWords * sizeof(int));
            // For tests of the error path: the status word starts as if a bounded wait of an earlier block
            // had expired, so the plan's first launch takes the early-leave path (no wait is made to expire).
            if (e == cudaSuccess)
                if (const char *preset = std::getenv("CLEAR_TEST_PRESET_STATUS")) {
                    const int code = std::atoi(preset);
                    if (code != 0) e = cudaMemcpy(p->d_status, &code, sizeof(int), cudaMemcpyHostToDevice);
                }
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->ev_last, cudaEventDisableTiming);
            if (e != cudaSuccess) {
                note_cuda_error((int)e);
                (void)cudaGetLastError();
                rc = CLEAR_ERR_CUDA;
            }
        }
        if (rc == CLEAR_OK && p->workspace_bytes > 0) {
            const int64_t rows = (int64_t)s.B * s.H * p->sch.n_partial_slots * kTileTokens;
            cudaError_t e = cudaMalloc((void **)&p->d_partial_o, (size_t)rows * s.head_dim * sizeof(float));
            if (e == cudaSuccess) e = cudaMalloc((void **)&p->d_partial_ml, (size_t)rows * 2 * sizeof(float));
            if (e != cudaSuccess) {
                note_cuda_error((int)e);
                (void)cudaGetLastError();
                rc = e == cudaErrorMemoryAllocation ? CLEAR_ERR_NO_MEMORY : CLEAR_ERR_CUDA;
            }
        }
        if (rc != CLEAR_OK) {
            free_device_parts(p.get());
            return rc;
        }
    }
    *out = p.release();
    return CLEAR_OK;
}

// Chunks of the host-tensor entry point hold at least this many bytes per tensor (CLEAR_HOST_CHUNK_BYTES
// overrides it): large enough that a chunk's kernels fill the device, small enough that the first
// copy in and the last copy out, which nothing overlaps, stay short.
constexpr size_t kHostChunkBytes = (size_t)96 << 20;

void destroy_host_pipe(clear_plan *p)
{
    HostPipe *h = p->pipe;
    if (!h) return;
    for (clear_plan *&sub : h->sub) {
        (void)clear_plan_destroy(sub);
        sub = nullptr;
    }
    if (h->s_in) (void)cudaStreamDestroy(h->s_in);
    if (h->s_out) (void)cudaStreamDestroy(h->s_out);
    if (h->ev_start) (void)cudaEventDestroy(h->ev_start);
    if (h->ev_out) (void)cudaEventDestroy(h->ev_out);
    for (cudaEvent_t ev : h->ev_in)
        if (ev) (void)cudaEventDestroy(ev);
    for (cudaEvent_t ev : h->ev_done)
        if (ev) (void)cudaEventDestroy(ev);
    (void)cudaGetLastError();
    delete h;
    p->pipe = nullptr;
}

// Builds the copy/compute pipeline of the host-tensor entry point on first use; leaves `plan->pipe`
// null when the problem is too small to be worth cutting.  `slice` = bytes of one (b, h) slice.
int ensure_host_pipe(clear_plan *plan, size_t slice)
{
    if (plan->pipe || plan->pipe_decided) return CLEAR_OK;
    plan->pipe_decided = true;
    const Shape &s = plan->shape;
    const int n_bh = s.B * s.H;
    size_t min_bytes = kHostChunkBytes;
    if (const char *e = std::getenv("CLEAR_HOST_CHUNK_BYTES")) min_bytes = (size_t)std::max(1ll, std::atoll(e));
    int chunk = (int)std::min<size_t>((size_t)n_bh, (min_bytes + slice - 1) / slice);
    chunk = std::max(chunk, (n_bh + kMaxHostChunks - 1) / kMaxHostChunks);
    if (chunk >= n_bh) return CLEAR_OK;
    std::unique_ptr<HostPipe> hp(new (std::nothrow) HostPipe());
    if (!hp) return CLEAR_ERR_NO_MEMORY;
    hp->chunk_heads = chunk;
    hp->n_chunks = (n_bh + chunk - 1) / chunk;
    plan->pipe = hp.release();
    HostPipe &h = *plan->pipe;
    auto fail = [&](int rc) {
        destroy_host_pipe(plan);
        plan->pipe_decided = false;
        return rc;
    };
    Shape sub = s;
    sub.kernel = plan->kernel;
    sub.B = 1;
    sub.H = chunk;
    int rc = create_plan(&h.sub[0], sub, false);
    if (rc != CLEAR_OK) return fail(rc);
    if (n_bh % chunk) {
        sub.H = n_bh % chunk;
        rc = create_plan(&h.sub[1], sub, false);
        if (rc != CLEAR_OK) return fail(rc);
    }
    cudaError_t e = cudaStreamCreateWithFlags(&h.s_in, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h.s_out, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h.ev_start, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h.ev_out, cudaEventDisableTiming);
    for (int c = 0; c < h.n_chunks && e == cudaSuccess; ++c) {
        e = cudaEventCreateWithFlags(&h.ev_in[c], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h.ev_done[c], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) {
        note_cuda_error((int)e);
        (void)cudaGetLastError();
        return fail(CLEAR_ERR_CUDA);
    }
    return CLEAR_OK;
}

int check_tensors(const void *q, const void *k, const void *v, const void *out)
{
    if (!q || !k || !v || !out) return CLEAR_ERR_INVALID_ARG;
    const uintptr_t bits = (uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out;
    if (bits & 15u) return CLEAR_ERR_MISALIGNED;
    return CLEAR_OK;
}

int forward(const clear_plan *p, const void *q, const void *k, const void *v, void *out, float scale, void *stream)
{
    if (!p) return CLEAR_ERR_INVALID_ARG;
    if (!std::isfinite(scale)) return CLEAR_ERR_INVALID_ARG;
    int rc = check_tensors(q, k, v, out);
    if (rc != CLEAR_OK) return rc;
    if (p->host_only) return CLEAR_ERR_PLAN_MISMATCH;
    int dev = -1;
    CLEAR_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != p->device) return CLEAR_ERR_PLAN_MISMATCH;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // launches of one plan run one after the other on the device, whatever streams they are made on
    std::lock_guard<std::mutex> lock(p->launch_mutex);
    if (p->has_last && p->last_stream != st) CLEAR_CUDA_TRY(cudaStreamWaitEvent(st, p->ev_last, 0));
    if (p->kernel == CLEAR_KERNEL_TCGEN05)
        rc = launch_tc(*p, q, k, v, out, scale, st);
    else if (p->kernel == CLEAR_KERNEL_TCGEN05_WS)
        rc = launch_ws(*p, q, k, v, out, scale, st);
    else
        rc = launch_simt(*p, q, k, v, out, scale, st);
    if (rc != CLEAR_OK) return rc;
    CLEAR_CUDA_TRY(cudaEventRecord(p->ev_last, st));
    p->last_stream = st;
    p->has_last = true;
    return CLEAR_OK;
}

// ---- plan cache of the unplanned entry points ----------------------------------------------------
struct CacheEntry {
    Shape shape;
    int device;
    clear_plan_t *plan;
};
std::mutex g_cache_mutex;
std::list<CacheEntry> g_cache;  // most recently used first
// The cache keeps at most this many plans (CLEAR_CACHE_MAX_PLANS overrides it): a plan of the 8K workload owns
// 211 MB of split-KV workspace.  The least recently used plan goes when a new shape arrives.
constexpr int kMaxCachedPlans = 16;

// Finds (or makes) the cached plan of a shape on the current device and calls `launch(plan)` with the cache
// locked: no other thread can evict or clear the plan while it is being launched (launches take microseconds).
template <typename Launch>
int with_cached_plan(const Shape &s, Launch &&launch)
{
    int dev = -1;
    CLEAR_CUDA_TRY(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    clear_plan_t *plan = nullptr;
    for (auto it = g_cache.begin(); it != g_cache.end(); ++it)
        if (it->device == dev && it->shape == s) {
            plan = it->plan;
            g_cache.splice(g_cache.begin(), g_cache, it);
            break;
        }
    if (!plan) {
        int cap = kMaxCachedPlans;
        if (const char *e = std::getenv("CLEAR_CACHE_MAX_PLANS")) cap = std::max(1, std::atoi(e));
        while ((int)g_cache.size() >= cap) {
            // work of the evicted plan may still be in flight
            if (cudaDeviceSynchronize() != cudaSuccess) (void)cudaGetLastError();
            (void)clear_plan_destroy(g_cache.back().plan);
            g_cache.pop_back();
        }
        const int rc = create_plan(&plan, s, false);
        if (rc != CLEAR_OK) return rc;
        g_cache.push_front(CacheEntry{s, dev, plan});
    }
    return launch(plan);
}

int cached_forward(const void *q, const void *k, const void *v, void *out, const Shape &shape, float scale, void *stream)
{
    int rc = validate_shape(shape);
    if (rc != CLEAR_OK) return rc;
    if (!std::isfinite(scale)) return CLEAR_ERR_INVALID_ARG;
    rc = check_tensors(q, k, v, out);
    if (rc != CLEAR_OK) return rc;
    Shape s = shape;
    // the tensor-core kernel needs a positive scale; anything else goes to the CUDA-core kernel
    if (s.kernel == CLEAR_KERNEL_AUTO && !(scale > 0.f)) s.kernel = CLEAR_KERNEL_SIMT;
    return with_cached_plan(s, [&](clear_plan_t *plan) { return forward(plan, q, k, v, out, scale, stream); });
}

}  // namespace
}  // namespace clear

using namespace clear;

extern "C" {

int clear_attn_fwd(const void *q, const void *k, const void *v, void *out, int B, int H, int grid_h, int grid_w,
                   int n_text, int head_dim, float radius, float scale, void *stream)
{
    Shape s{B, H, grid_h, grid_w, n_text, head_dim, radius, CLEAR_BF16, CLEAR_KERNEL_AUTO};
    return cached_forward(q, k, v, out, s, scale, stream);
}

int clear_attn_fwd_f32(const void *q, const void *k, const void *v, void *out, int B, int H, int grid_h, int grid_w,
                       int n_text, int head_dim, float radius, float scale, void *stream)
{
    Shape s{B, H, grid_h, grid_w, n_text, head_dim, radius, CLEAR_F32, CLEAR_KERNEL_SIMT};
    return cached_forward(q, k, v, out, s, scale, stream);
}

static int backward(const void *q, const void *k, const void *v, const void *d_out, void *dq, void *dk, void *dv, int B,
                    int H, int grid_h, int grid_w, int n_text, int head_dim, float radius, float scale, int dtype,
                    void *stream, bool tensor_cores = false)
{
    Shape s{B, H, grid_h, grid_w, n_text, head_dim, radius, dtype, tensor_cores ? CLEAR_KERNEL_TCGEN05 : CLEAR_KERNEL_SIMT};
    s.no_text_split = tensor_cores ? 1 : 0;
    int rc = validate_shape(s);
    if (rc != CLEAR_OK) return rc;
    if (!std::isfinite(scale)) return CLEAR_ERR_INVALID_ARG;
    rc = check_tensors(q, k, v, d_out);
    if (rc == CLEAR_OK) rc = check_tensors(dq, dk, dv, dq);
    if (rc != CLEAR_OK) return rc;
    return with_cached_plan(s, [&](clear_plan_t *plan) -> int {
        // calls of one plan share its row-statistics buffer: ordered on the device like the forward launches
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        std::lock_guard<std::mutex> lock(plan->launch_mutex);
        if (plan->has_last && plan->last_stream != st) CLEAR_CUDA_TRY(cudaStreamWaitEvent(st, plan->ev_last, 0));
        const int rc2 = tensor_cores ? launch_bwd_tc(*plan, q, k, v, d_out, dq, dk, dv, scale, st)
                                     : launch_bwd(*plan, q, k, v, d_out, dq, dk, dv, scale, st);
        if (rc2 != CLEAR_OK) return rc2;
        CLEAR_CUDA_TRY(cudaEventRecord(plan->ev_last, st));
        plan->last_stream = st;
        plan->has_last = true;
        return CLEAR_OK;
    });
}

int clear_attn_bwd_f32(const void *q, const void *k, const void *v, const void *d_out, void *dq, void *dk, void *dv,
                       int B, int H, int grid_h, int grid_w, int n_text, int head_dim, float radius, float scale,
                       void *stream)
{
    return backward(q, k, v, d_out, dq, dk, dv, B, H, grid_h, grid_w, n_text, head_dim, radius, scale, CLEAR_F32, stream);
}

int clear_attn_bwd_bf16(const void *q, const void *k, const void *v, const void *d_out, void *dq, void *dk, void *dv,
                        int B, int H, int grid_h, int grid_w, int n_text, int head_dim, float radius, float scale,
                        void *stream)
{
    return backward(q, k, v, d_out, dq, dk, dv, B, H, grid_h, grid_w, n_text, head_dim, radius, scale, CLEAR_BF16, stream);
}

int clear_attn_bwd_bf16_tc(const void *q, const void *k, const void *v, const void *d_out, void *dq, void *dk, void *dv,
                           int B, int H, int grid_h, int grid_w, int n_text, int head_dim, float radius, float scale,
                           void *stream)
{
    if (head_dim != 64 && head_dim != 128) return CLEAR_ERR_UNSUPPORTED;
    if (!(scale > 0.f)) return std::isfinite(scale) ? CLEAR_ERR_UNSUPPORTED : CLEAR_ERR_INVALID_ARG;
    return backward(q, k, v, d_out, dq, dk, dv, B, H, grid_h, grid_w, n_text, head_dim, radius, scale, CLEAR_BF16, stream,
                    true);
}

int clear_qk_norm_rope(const void *q_in, const void *k_in, void *q_out, void *k_out, const float *gain_q,
                       const float *gain_k, int B, int H, int grid_h, int grid_w, int n_text, int head_dim, int dtype,
                       int axis0_dim, int axis1_dim, int axis2_dim, float theta, float ntk_factor, float eps,
                       float q_factor, void *stream)
{
    if (B <= 0 || H <= 0 || grid_h <= 0 || grid_w <= 0 || n_text < 0) return CLEAR_ERR_INVALID_ARG;
    if (dtype != CLEAR_BF16 && dtype != CLEAR_F32) return CLEAR_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return CLEAR_ERR_UNSUPPORTED;
    const int axes[3] = {axis0_dim, axis1_dim, axis2_dim};
    for (int a = 0; a < 3; ++a)
        if (axes[a] < 0 || (axes[a] & 1)) return CLEAR_ERR_INVALID_ARG;
    if (axis0_dim + axis1_dim + axis2_dim != head_dim) return CLEAR_ERR_INVALID_ARG;
    if (!(theta > 0.f) || !std::isfinite(theta) || !(ntk_factor > 0.f) || !std::isfinite(ntk_factor))
        return CLEAR_ERR_INVALID_ARG;
    if (!(eps >= 0.f) || !std::isfinite(eps) || !std::isfinite(q_factor)) return CLEAR_ERR_INVALID_ARG;
    const int rc = check_tensors(q_in, k_in, q_out, k_out);
    if (rc != CLEAR_OK) return rc;
    if ((((uintptr_t)gain_q) | ((uintptr_t)gain_k)) & 3u) return CLEAR_ERR_MISALIGNED;
    return launch_qk_prep(q_in, k_in, q_out, k_out, gain_q, gain_k, B * H, grid_h, grid_w, n_text, head_dim, dtype, axes,
                          (double)theta, (double)ntk_factor, eps, q_factor, static_cast<cudaStream_t>(stream));
}

float clear_log_scale_factor(long long n_tokens, long long n_train_tokens)
{
    if (n_tokens < 2 || n_train_tokens < 2) return 1.f;
    return (float)std::sqrt(std::log((double)n_tokens) / std::log((double)n_train_tokens));
}

int clear_plan_create(clear_plan_t **plan, int B, int H, int grid_h, int grid_w, int n_text, int head_dim,
                      float radius, int dtype, int kernel)
{
    Shape s{B, H, grid_h, grid_w, n_text, head_dim, radius, dtype, kernel};
    return create_plan(plan, s, false);
}

int clear_plan_create_ex(clear_plan_t **plan, int B, int H, int grid_h, int grid_w, int n_text, int head_dim,
                         float radius, int dtype, int kernel, int mask_kind, int host_only)
{
    Shape s{B, H, grid_h, grid_w, n_text, head_dim, radius, dtype, kernel};
    s.mask_kind = mask_kind;
    return create_plan(plan, s, host_only != 0);
}

int clear_plan_create_mask(clear_plan_t **plan, int B, int H, int grid_h, int grid_w, int n_text, int head_dim, int dtype,
                           int mask_kind, float mask_size, int mask_param, int host_only)
{
    Shape s{B, H, grid_h, grid_w, n_text, head_dim, mask_size, dtype, CLEAR_KERNEL_AUTO};
    s.mask_kind = mask_kind;
    s.mask_param = mask_param;
    return create_plan(plan, s, host_only != 0);
}

int clear_plan_create_host(clear_plan_t **plan, int B, int H, int grid_h, int grid_w, int n_text, int head_dim,
                           float radius, int dtype, int kernel)
{
    Shape s{B, H, grid_h, grid_w, n_text, head_dim, radius, dtype, kernel};
    return create_plan(plan, s, true);
}

int clear_plan_tables(const clear_plan_t *plan, const clear_work_item_t **items, int32_t *n_items,
                      const clear_kv_tile_t **tiles, int32_t *n_tiles, const int32_t **half_width,
                      int32_t *n_half_width)
{
    if (!plan) return CLEAR_ERR_INVALID_ARG;
    if (items) *items = plan->sch.items.data();
    if (n_items) *n_items = (int32_t)plan->sch.items.size();
    if (tiles) *tiles = plan->sch.tiles.data();
    if (n_tiles) *n_tiles = (int32_t)plan->sch.tiles.size();
    if (half_width) *half_width = plan->sch.half_width.data();
    if (n_half_width) *n_half_width = (int32_t)plan->sch.half_width.size();
    return CLEAR_OK;
}

int clear_plan_pair_tables(const clear_plan_t *plan, const clear_pair_item_t **items, int32_t *n_items,
                           const clear_pair_step_t **steps, int32_t *n_steps)
{
    if (!plan) return CLEAR_ERR_INVALID_ARG;
    if (items) *items = plan->sch.pair_items.data();
    if (n_items) *n_items = (int32_t)plan->sch.pair_items.size();
    if (steps) *steps = plan->sch.pair_steps.data();
    if (n_steps) *n_steps = (int32_t)plan->sch.pair_steps.size();
    return CLEAR_OK;
}

int clear_plan_mask_table(const clear_plan_t *plan, const uint32_t **words, int32_t *n_entries)
{
    if (!plan) return CLEAR_ERR_INVALID_ARG;
    if (words) *words = plan->sch.mask_table.data();
    if (n_entries) *n_entries = (int32_t)(plan->sch.mask_table.size() / ((size_t)kTileTokens * 4));
    return CLEAR_OK;
}

int clear_attn_fwd_planned(const clear_plan_t *plan, const void *q, const void *k, const void *v, void *out,
                           float scale, void *stream)
{
    if (plan && plan->shape.part == CLEAR_PART_BAND_TEXT) return CLEAR_ERR_PLAN_MISMATCH;  // clear_attn_text_partial
    return forward(plan, q, k, v, out, scale, stream);
}

int clear_band_geometry(int grid_h, float radius, int mask_kind, int n_bands, int band, int32_t *y0, int32_t *y1,
                        int32_t *halo_lo, int32_t *halo_hi)
{
    if (grid_h <= 0 || n_bands <= 0 || n_bands > grid_h || band < 0 || band >= n_bands) return CLEAR_ERR_INVALID_ARG;
    if (!(radius > 0.f) || !std::isfinite(radius)) return CLEAR_ERR_INVALID_ARG;
    if (mask_kind != CLEAR_MASK_DISC && mask_kind != CLEAR_MASK_SQUARE) return CLEAR_ERR_INVALID_ARG;
    const int base = grid_h / n_bands, extra = grid_h % n_bands;
    const int a = band * base + std::min(band, extra), b = a + base + (band < extra ? 1 : 0);
    const int64_t reach = window_reach(radius, mask_kind);
    if (y0) *y0 = a;
    if (y1) *y1 = b;
    if (halo_lo) *halo_lo = (int32_t)std::min<int64_t>(reach, a);
    if (halo_hi) *halo_hi = (int32_t)std::min<int64_t>(reach, grid_h - b);
    return CLEAR_OK;
}

int clear_plan_create_band(clear_plan_t **plan, int B, int H, int local_rows, int grid_w, int n_text, int head_dim,
                           float radius, int mask_kind, int part, int q_row_begin, int q_row_end, int text_keys,
                           int host_only)
{
    if (part != CLEAR_PART_BAND_IMAGE && part != CLEAR_PART_BAND_TEXT) return CLEAR_ERR_INVALID_ARG;
    Shape s{B, H, local_rows, grid_w, n_text, head_dim, radius, CLEAR_BF16, CLEAR_KERNEL_TCGEN05_WS};
    s.mask_kind = mask_kind;
    s.part = part;
    s.q_row_begin = q_row_begin;
    s.q_row_end = q_row_end;
    s.text_keys = text_keys != 0;
    return create_plan(plan, s, host_only != 0);
}

int clear_attn_text_partial(const clear_plan_t *plan, const void *q, const void *k, const void *v, float *records,
                            float scale, void *stream)
{
    if (!plan) return CLEAR_ERR_INVALID_ARG;
    if (plan->shape.part != CLEAR_PART_BAND_TEXT) return CLEAR_ERR_PLAN_MISMATCH;
    return forward(plan, q, k, v, records, scale, stream);
}

int clear_text_merge(const float *records, int n_parts, int B, int H, int n_text, int head_dim, int mode, void *out,
                     long long out_tokens, void *stream)
{
    if (!records || !out || n_parts <= 0 || B <= 0 || H <= 0 || n_text <= 0 || out_tokens < n_text)
        return CLEAR_ERR_INVALID_ARG;
    if (mode != CLEAR_TEXT_MERGE_EXACT && mode != CLEAR_TEXT_MERGE_AVERAGE) return CLEAR_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return CLEAR_ERR_UNSUPPORTED;
    if ((int64_t)B * H > 65535) return CLEAR_ERR_UNSUPPORTED;
    if ((((uintptr_t)records) & 3u) || (((uintptr_t)out) & 15u)) return CLEAR_ERR_MISALIGNED;
    return launch_text_merge(records, n_parts, B * H, n_text, head_dim, mode, out, out_tokens,
                             static_cast<cudaStream_t>(stream));
}

int clear_attn_fwd_host(clear_plan_t *plan, const void *q_host, const void *k_host, const void *v_host,
                        void *out_host, float scale, void *stream)
{
    if (!plan || !q_host || !k_host || !v_host || !out_host) return CLEAR_ERR_INVALID_ARG;
    if (!std::isfinite(scale)) return CLEAR_ERR_INVALID_ARG;
    if (plan->host_only || plan->shape.part != CLEAR_PART_ALL) return CLEAR_ERR_PLAN_MISMATCH;
    int dev = -1;
    CLEAR_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != plan->device) return CLEAR_ERR_PLAN_MISMATCH;
    const Shape &s = plan->shape;
    const size_t esz = s.dtype == CLEAR_BF16 ? 2 : 4;
    const size_t slice = ((size_t)s.n_text + (size_t)s.grid_h * s.grid_w) * s.head_dim * esz;
    const size_t bytes = (size_t)s.B * s.H * slice;
    for (void *&st : plan->d_stage) {
        if (!st) {
            cudaError_t e = cudaMalloc(&st, bytes);
            if (e != cudaSuccess) {
                st = nullptr;
                note_cuda_error((int)e);
                (void)cudaGetLastError();
                return e == cudaErrorMemoryAllocation ? CLEAR_ERR_NO_MEMORY : CLEAR_ERR_CUDA;
            }
        }
    }
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    int rc = ensure_host_pipe(plan, slice);
    if (rc != CLEAR_OK) return rc;
    if (!plan->pipe) {
        CLEAR_CUDA_TRY(cudaMemcpyAsync(plan->d_stage[0], q_host, bytes, cudaMemcpyHostToDevice, cs));
        CLEAR_CUDA_TRY(cudaMemcpyAsync(plan->d_stage[1], k_host, bytes, cudaMemcpyHostToDevice, cs));
        CLEAR_CUDA_TRY(cudaMemcpyAsync(plan->d_stage[2], v_host, bytes, cudaMemcpyHostToDevice, cs));
        rc = forward(plan, plan->d_stage[0], plan->d_stage[1], plan->d_stage[2], plan->d_stage[3], scale, stream);
        if (rc != CLEAR_OK) return rc;
        CLEAR_CUDA_TRY(cudaMemcpyAsync(out_host, plan->d_stage[3], bytes, cudaMemcpyDeviceToHost, cs));
        return clear_plan_check(plan, stream);
    }

    // Three stages over chunks of the (batch, head) axis: copies in on one stream, kernels on the
    // caller's stream, copies out on a third; events hand each chunk from stage to stage.
    HostPipe &hp = *plan->pipe;
    const int n_bh = s.B * s.H;
    const void *host_in[3] = {q_host, k_host, v_host};
    CLEAR_CUDA_TRY(cudaEventRecord(hp.ev_start, cs));
    CLEAR_CUDA_TRY(cudaStreamWaitEvent(hp.s_in, hp.ev_start, 0));
    CLEAR_CUDA_TRY(cudaStreamWaitEvent(hp.s_out, hp.ev_start, 0));
    rc = CLEAR_OK;
    for (int c = 0; c < hp.n_chunks && rc == CLEAR_OK; ++c) {
        const int first = c * hp.chunk_heads;
        const int heads = std::min(hp.chunk_heads, n_bh - first);
        const size_t off = (size_t)first * slice, len = (size_t)heads * slice;
        for (int t = 0; t < 3; ++t)
            CLEAR_CUDA_TRY(cudaMemcpyAsync((char *)plan->d_stage[t] + off, (const char *)host_in[t] + off, len,
                                           cudaMemcpyHostToDevice, hp.s_in));
        CLEAR_CUDA_TRY(cudaEventRecord(hp.ev_in[c], hp.s_in));
        CLEAR_CUDA_TRY(cudaStreamWaitEvent(cs, hp.ev_in[c], 0));
        const clear_plan *sub = heads == hp.chunk_heads ? hp.sub[0] : hp.sub[1];
        rc = forward(sub, (char *)plan->d_stage[0] + off, (char *)plan->d_stage[1] + off,
                     (char *)plan->d_stage[2] + off, (char *)plan->d_stage[3] + off, scale, stream);
        if (rc != CLEAR_OK) break;
        CLEAR_CUDA_TRY(cudaEventRecord(hp.ev_done[c], cs));
        CLEAR_CUDA_TRY(cudaStreamWaitEvent(hp.s_out, hp.ev_done[c], 0));
        CLEAR_CUDA_TRY(cudaMemcpyAsync((char *)out_host + off, (char *)plan->d_stage[3] + off, len,
                                       cudaMemcpyDeviceToHost, hp.s_out));
    }
    // the copies out are joined back into the caller's stream, error or not (the copies in already
    // are: every chunk's kernels waited for them)
    cudaError_t e1 = cudaEventRecord(hp.ev_out, hp.s_out);
    cudaError_t e2 = cudaStreamWaitEvent(cs, hp.ev_out, 0);
    for (cudaError_t e : {e1, e2})
        if (e != cudaSuccess) {
            note_cuda_error((int)e);
            (void)cudaGetLastError();
            if (rc == CLEAR_OK) rc = CLEAR_ERR_CUDA;
        }
    for (clear_plan *sub : hp.sub)
        if (sub) {
            const int r = clear_plan_check(sub, stream);
            if (rc == CLEAR_OK) rc = r;
        }
    if (rc != CLEAR_OK) (void)cudaStreamSynchronize(cs);
    return rc;
}

int clear_plan_info(const clear_plan_t *plan, clear_plan_info_t *info)
{
    if (!plan || !info) return CLEAR_ERR_INVALID_ARG;
    const Shape &s = plan->shape;
    std::memset(info, 0, sizeof(*info));
    info->B = s.B;
    info->H = s.H;
    info->grid_h = s.grid_h;
    info->grid_w = s.grid_w;
    info->n_text = s.n_text;
    info->head_dim = s.head_dim;
    info->dtype = s.dtype;
    info->kernel = plan->kernel;
    info->radius_sq_ceil = (int32_t)plan->sch.thr;
    const bool tc = plan->kernel != CLEAR_KERNEL_SIMT;
    info->tile_h = tc ? kTileH : 0;
    info->tile_w = tc ? kTileW : 0;
    info->n_work_items = plan->kernel == CLEAR_KERNEL_TCGEN05_WS ? (int32_t)plan->sch.pair_items.size()
                                                                  : (int32_t)plan->sch.items.size();
    info->n_text_splits = plan->sch.n_text_splits;
    info->max_item_tiles = plan->sch.max_item_tiles;
    info->sum_mask = plan->sch.sum_mask;
    info->executed_pairs = tc ? plan->sch.executed_pairs : plan->sch.sum_mask;
    info->workspace_bytes = plan->workspace_bytes;
    info->flops = 4.0 * (double)plan->sch.sum_mask * s.head_dim * s.H * s.B;
    return CLEAR_OK;
}

int clear_plan_check(clear_plan_t *plan, void *stream)
{
    if (!plan) return CLEAR_ERR_INVALID_ARG;
    if (plan->host_only) return CLEAR_ERR_PLAN_MISMATCH;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    int words[kStatusWords] = {0, 0, 0, 0};
    CLEAR_CUDA_TRY(cudaMemcpyAsync(words, plan->d_status, sizeof(words), cudaMemcpyDeviceToHost, cs));
    CLEAR_CUDA_TRY(cudaStreamSynchronize(cs));
    const int status = words[3] != 0 ? words[3] : words[0];
    if (status != 0) {
        g_last_device_status = status;
        // a block that gave up may have left the work queue of the persistent kernel mid-way
        CLEAR_CUDA_TRY(cudaMemsetAsync(plan->d_status, 0, kStatusWords * sizeof(int), cs));
        CLEAR_CUDA_TRY(cudaStreamSynchronize(cs));
        return CLEAR_ERR_DEVICE_TIMEOUT;
    }
    return CLEAR_OK;
}

int clear_cache_check(void *stream)
{
    int dev = -1;
    CLEAR_CUDA_TRY(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    int rc = CLEAR_OK;
    for (CacheEntry &e : g_cache) {
        if (e.device != dev) continue;
        // the plan's last launch may have been made on another stream than the one given
        if (e.plan->has_last && cudaEventSynchronize(e.plan->ev_last) != cudaSuccess) {
            (void)cudaGetLastError();
            if (rc == CLEAR_OK) rc = CLEAR_ERR_CUDA;
        }
        const int r = clear_plan_check(e.plan, stream);
        if (r != CLEAR_OK && rc == CLEAR_OK) rc = r;
    }
    return rc;
}

int clear_plan_trim(clear_plan_t *plan)
{
    if (!plan) return CLEAR_ERR_INVALID_ARG;
    if (plan->host_only) return CLEAR_OK;
    int prev = -1;
    if (cudaGetDevice(&prev) == cudaSuccess && prev != plan->device) (void)cudaSetDevice(plan->device);
    int rc = CLEAR_OK;
    if (cudaDeviceSynchronize() != cudaSuccess) {
        (void)cudaGetLastError();
        rc = CLEAR_ERR_CUDA;
    }
    destroy_host_pipe(plan);
    plan->pipe_decided = false;
    for (void *&st : plan->d_stage) {
        if (st && cudaFree(st) != cudaSuccess) {
            (void)cudaGetLastError();
            rc = CLEAR_ERR_CUDA;
        }
        st = nullptr;
    }
    if (prev >= 0 && prev != plan->device) (void)cudaSetDevice(prev);
    return rc;
}

int clear_plan_destroy(clear_plan_t *plan)
{
    if (!plan) return CLEAR_OK;
    int rc = CLEAR_OK;
    if (!plan->host_only) {
        int prev = -1;
        if (cudaGetDevice(&prev) == cudaSuccess && prev != plan->device) (void)cudaSetDevice(plan->device);
        destroy_host_pipe(plan);
        rc = free_device_parts(plan);
        if (prev >= 0 && prev != plan->device) (void)cudaSetDevice(prev);
    }
    delete plan;
    return rc;
}

int clear_cache_clear(void)
{
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    int rc = CLEAR_OK;
    if (!g_cache.empty()) {
        if (cudaDeviceSynchronize() != cudaSuccess) {
            (void)cudaGetLastError();
            rc = CLEAR_ERR_CUDA;
        }
    }
    for (CacheEntry &e : g_cache) {
        int r = clear_plan_destroy(e.plan);
        if (r != CLEAR_OK) rc = r;
    }
    g_cache.clear();
    return rc;
}

const char *clear_status_string(int status)
{
    switch (status) {
        case CLEAR_OK: return "ok";
        case CLEAR_ERR_INVALID_ARG: return "invalid argument";
        case CLEAR_ERR_UNSUPPORTED: return "unsupported shape, dtype or kernel";
        case CLEAR_ERR_MISALIGNED: return "tensor pointer is not 16-byte aligned";
        case CLEAR_ERR_PLAN_MISMATCH: return "plan does not match this call (device, host-only plan)";
        case CLEAR_ERR_CUDA: return "CUDA call failed";
        case CLEAR_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel expired";
        case CLEAR_ERR_NO_MEMORY: return "out of memory";
        case CLEAR_ERR_TOO_LARGE: return "shape exceeds a fixed capacity of the no-allocation entry point";
        default: return "unknown status";
    }
}

int clear_last_cuda_error(void) { return g_last_cuda_error; }

int clear_last_device_status(void) { return g_last_device_status; }

}  // extern "C"
