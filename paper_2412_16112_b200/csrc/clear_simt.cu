// CLEAR attention forward on the CUDA cores: one warp per query, fp32 arithmetic throughout.
//
// This is the exact-order path: it serves fp32 tensors (where tensor-core input rounding would
// break a 1e-5 agreement), head sizes the tensor-core kernel does not take, and non-positive
// scales.  Each warp walks the keys its query may see under Eq. 3 -- the text tokens, then for
// every grid row within reach the run of columns [x - m(dy), x + m(dy)] clipped to the grid --
// and keeps an online softmax (Eq. 1) over blocks of 8 keys.  Lanes split the head dimension.
// The two comparison masks of the appendix that are no window around the query run here too: the
// shifted window grid (a rectangle of keys per query) and the strided mask (every r-th row and column).
#include <cuda_bf16.h>

#include "clear_internal.hpp"

namespace clear {
namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kKeyBlock = 8;

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f32(float *p, float x) { *p = x; }
__device__ __forceinline__ void from_f32(__nv_bfloat16 *p, float x) { *p = __float2bfloat16_rn(x); }

template <typename T, int EPL>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
clear_simt_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v, T *__restrict__ out,
                  int grid_h, int grid_w, int n_text, int d, const int32_t *__restrict__ half_width, int n_half_width,
                  int mask_kind, int mask_size, int mask_param, float scale)
{
    const int lane = threadIdx.x & 31;
    const int64_t N = (int64_t)n_text + (int64_t)grid_h * grid_w;
    const int64_t i = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (i >= N) return;  // whole warp leaves together
    const int64_t base = (int64_t)blockIdx.y * N * d;

    float qv[EPL], acc[EPL];
#pragma unroll
    for (int t = 0; t < EPL; ++t) {
        const int e = lane + 32 * t;
        qv[t] = e < d ? to_f32(q[base + i * d + e]) * scale : 0.f;
        acc[t] = 0.f;
    }
    float m = -INFINITY, l = 0.f;

    // online softmax over the tokens j0, j0 + step, ... below j1
    auto run = [&](int64_t j0, int64_t j1, int64_t step) {
        for (int64_t j = j0; j < j1; j += kKeyBlock * step) {
            float s[kKeyBlock];
#pragma unroll
            for (int u = 0; u < kKeyBlock; ++u) {
                const int64_t jj = j + u * step;
                float part = 0.f;
                if (jj < j1) {
#pragma unroll
                    for (int t = 0; t < EPL; ++t) {
                        const int e = lane + 32 * t;
                        if (e < d) part = fmaf(qv[t], to_f32(k[base + jj * d + e]), part);
                    }
                }
                s[u] = part;
            }
#pragma unroll
            for (int u = 0; u < kKeyBlock; ++u) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) s[u] += __shfl_xor_sync(0xffffffffu, s[u], o);
                if (j + u * step >= j1) s[u] = -INFINITY;
            }
            float m_new = m;
#pragma unroll
            for (int u = 0; u < kKeyBlock; ++u) m_new = fmaxf(m_new, s[u]);
            const float alpha = expf(m - m_new);  // m = -inf on the first block: alpha = 0
            l *= alpha;
#pragma unroll
            for (int t = 0; t < EPL; ++t) acc[t] *= alpha;
#pragma unroll
            for (int u = 0; u < kKeyBlock; ++u) {
                const int64_t jj = j + u * step;
                if (jj < j1) {
                    const float p = expf(s[u] - m_new);
                    l += p;
#pragma unroll
                    for (int t = 0; t < EPL; ++t) {
                        const int e = lane + 32 * t;
                        if (e < d) acc[t] = fmaf(p, to_f32(v[base + jj * d + e]), acc[t]);
                    }
                }
            }
            m = m_new;
        }
    };

    if (i < n_text) {
        run(0, N, 1);  // a text query sees every token
    } else {
        run(0, n_text, 1);  // every image query sees all text keys
        const int64_t pix = i - n_text;
        const int y = (int)(pix / grid_w), x = (int)(pix % grid_w);
        if (mask_kind == CLEAR_MASK_WINDOWS) {
            // the w x w window of the shifted window grid that holds (y, x), clipped to the grid
            const int w = mask_size, sh = mask_param;
            const int y_lo = max(((y + sh) / w) * w - sh, 0), y_hi = min(((y + sh) / w + 1) * w - sh, grid_h);
            const int x_lo = max(((x + sh) / w) * w - sh, 0), x_hi = min(((x + sh) / w + 1) * w - sh, grid_w);
            for (int yy = y_lo; yy < y_hi; ++yy) {
                const int64_t row0 = (int64_t)n_text + (int64_t)yy * grid_w;
                run(row0 + x_lo, row0 + x_hi, 1);
            }
        } else if (mask_kind == CLEAR_MASK_STRIDED) {
            // rows congruent to y + (l div r), columns congruent to x + (l mod r), modulo the stride r
            const int r = mask_size;
            const int y0 = (y + (mask_param / r) % r) % r, x0 = (x + mask_param % r) % r;
            for (int yy = y0; yy < grid_h; yy += r) {
                const int64_t row0 = (int64_t)n_text + (int64_t)yy * grid_w;
                run(row0 + x0, row0 + grid_w, r);
            }
        } else {
            const int R = n_half_width - 1;
            for (int dy = -R; dy <= R; ++dy) {
                const int yy = y + dy;
                if (yy < 0 || yy >= grid_h) continue;
                const int hw = half_width[dy < 0 ? -dy : dy];
                const int lo = max(x - hw, 0), hi = min(x + hw, grid_w - 1);
                const int64_t row0 = (int64_t)n_text + (int64_t)yy * grid_w;
                run(row0 + lo, row0 + hi + 1, 1);
            }
        }
    }

    // l > 0: an image query sees itself under the disc, the square and the windows, and the text keys always;
    // under the strided mask with no text a query may see nothing: its output is 0
    const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
    for (int t = 0; t < EPL; ++t) {
        const int e = lane + 32 * t;
        if (e < d) from_f32(&out[base + i * d + e], acc[t] * inv);
    }
}

template <typename T>
int launch_typed(const clear_plan &p, const void *q, const void *k, const void *v, void *out, float scale,
                 cudaStream_t stream)
{
    const Shape &s = p.shape;
    const int64_t N = (int64_t)s.n_text + (int64_t)s.grid_h * s.grid_w;
    dim3 grid((unsigned)((N + kWarpsPerBlock - 1) / kWarpsPerBlock), (unsigned)(s.B * s.H));
    dim3 block(kWarpsPerBlock * 32);
    const int n_hw = (int)p.sch.half_width.size();
    const int epl = (s.head_dim + 31) / 32;
#define CLEAR_SIMT_CASE(E)                                                                                      \
    case E:                                                                                                     \
        clear_simt_kernel<T, E><<<grid, block, 0, stream>>>((const T *)q, (const T *)k, (const T *)v, (T *)out, \
                                                            s.grid_h, s.grid_w, s.n_text, s.head_dim,           \
                                                            p.d_half_width, n_hw, s.mask_kind, (int)s.radius,   \
                                                            s.mask_param, scale);                               \
        break;
    switch (epl) {
        CLEAR_SIMT_CASE(1)
        CLEAR_SIMT_CASE(2)
        CLEAR_SIMT_CASE(3)
        CLEAR_SIMT_CASE(4)
        CLEAR_SIMT_CASE(5)
        CLEAR_SIMT_CASE(6)
        CLEAR_SIMT_CASE(7)
        CLEAR_SIMT_CASE(8)
        default:
            return CLEAR_ERR_UNSUPPORTED;
    }
#undef CLEAR_SIMT_CASE
    CLEAR_CUDA_TRY(cudaGetLastError());
    return CLEAR_OK;
}

}  // namespace

int launch_simt(const clear_plan &p, const void *q, const void *k, const void *v, void *out, float scale,
                cudaStream_t stream)
{
    if (p.shape.dtype == CLEAR_F32) return launch_typed<float>(p, q, k, v, out, scale, stream);
    return launch_typed<__nv_bfloat16>(p, q, k, v, out, scale, stream);
}

}  // namespace clear
