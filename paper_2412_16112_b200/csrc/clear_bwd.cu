// Backward pass of the CLEAR attention operator on the CUDA cores, fp32 throughout: dQ, dK, dV for an
// upstream gradient dO of  O = softmax(scale Q K^T + log M) V  (Eq. 1 under the mask of Eq. 3), the step
// through which the distillation losses of Sec. 3.3 (Eq. 4-6) reach the attention parameters.
//
// Two kernels, one warp per token, lanes split the head dimension, tokens walked as in the forward CUDA-core
// kernel (the text tokens, then per grid row within reach the clipped run of columns):
//   query kernel: sweep 1 over the query's keys: online softmax -> row maximum m, row sum l, the un-normalised
//       output, hence delta = dO . O; the three row statistics are kept for the second kernel;
//       sweep 2: p = exp(s - m) / l, dP = dO . v, dS = p (dP - delta), dQ += scale dS k;
//   key kernel: the mask is symmetric (M_ij = M_ji), so the queries that see key j are the tokens query j sees:
//       for each of them p_ij and dS_ij again from that query's statistics, dK_j += scale dS q_i, dV_j += p dO_i.
// Every output element has one writer and a fixed order of summation: results are the same from run to run.
// Each allowed pair costs four dot products of d channels instead of two, and no atomic operation.
#include <cuda_bf16.h>

#include "clear_internal.hpp"

namespace clear {
namespace {

constexpr int kWarpsPerBlock = 8;

__device__ __forceinline__ float ldf(const float *p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float *p, float x) { *p = x; }
__device__ __forceinline__ void stf(__nv_bfloat16 *p, float x) { *p = __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

template <typename T, int EPL>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
clear_bwd_query_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
                       const T *__restrict__ d_out, T *__restrict__ dq, float *__restrict__ stats, int grid_h,
                       int grid_w, int n_text, int d, const int32_t *__restrict__ half_width, int n_half_width, float scale)
{
    const int lane = threadIdx.x & 31;
    const int64_t N = (int64_t)n_text + (int64_t)grid_h * grid_w;
    const int64_t i = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (i >= N) return;  // whole warp leaves together
    const int64_t base = (int64_t)blockIdx.y * N * d;

    float qv[EPL], gv[EPL], acc[EPL];
#pragma unroll
    for (int t = 0; t < EPL; ++t) {
        const int e = lane + 32 * t;
        qv[t] = e < d ? ldf(q + base + i * d + e) : 0.f;
        gv[t] = e < d ? ldf(d_out + base + i * d + e) : 0.f;
        acc[t] = 0.f;
    }
    auto dot_row = [&](const float (&a)[EPL], const T *__restrict__ rows, int64_t j) {
        float part = 0.f;
#pragma unroll
        for (int t = 0; t < EPL; ++t) {
            const int e = lane + 32 * t;
            if (e < d) part = fmaf(a[t], ldf(rows + base + j * d + e), part);
        }
        return warp_sum(part);
    };
    // the keys Eq. 3 allows this query, as runs of consecutive tokens
    auto for_each_run = [&](auto &&body) {
        if (i < n_text) {
            body((int64_t)0, N);
            return;
        }
        body((int64_t)0, (int64_t)n_text);
        const int64_t pix = i - n_text;
        const int y = (int)(pix / grid_w), x = (int)(pix % grid_w);
        const int R = n_half_width - 1;
        for (int dy = -R; dy <= R; ++dy) {
            const int yy = y + dy;
            if (yy < 0 || yy >= grid_h) continue;
            const int hw = half_width[dy < 0 ? -dy : dy];
            const int lo = max(x - hw, 0), hi = min(x + hw, grid_w - 1);
            const int64_t row0 = (int64_t)n_text + (int64_t)yy * grid_w;
            body(row0 + lo, row0 + hi + 1);
        }
    };

    // ---- sweep 1: m, l and the un-normalised output ------------------------------------------------
    float m = -INFINITY, l = 0.f;
    for_each_run([&](int64_t j0, int64_t j1) {
        for (int64_t j = j0; j < j1; ++j) {
            const float s = scale * dot_row(qv, k, j);
            const float m_new = fmaxf(m, s);
            const float alpha = expf(m - m_new);  // m = -inf at the first key: alpha = 0
            const float p = expf(s - m_new);
            l = l * alpha + p;
#pragma unroll
            for (int t = 0; t < EPL; ++t) {
                const int e = lane + 32 * t;
                if (e < d) acc[t] = fmaf(p, ldf(v + base + j * d + e), acc[t] * alpha);
            }
            m = m_new;
        }
    });
    const float inv_l = 1.f / l;  // l >= 1: the query itself (image) or any token (text) is always allowed
    float part = 0.f;
#pragma unroll
    for (int t = 0; t < EPL; ++t) part = fmaf(gv[t], acc[t], part);
    const float delta = warp_sum(part) * inv_l;  // dO . O = sum_j p_ij dP_ij
    if (lane == 0) {
        float *st = stats + ((int64_t)blockIdx.y * N + i) * 3;
        st[0] = m;
        st[1] = inv_l;
        st[2] = delta;
    }

    // ---- sweep 2: the gradients --------------------------------------------------------------------
    float gq[EPL];
#pragma unroll
    for (int t = 0; t < EPL; ++t) gq[t] = 0.f;
    for_each_run([&](int64_t j0, int64_t j1) {
        for (int64_t j = j0; j < j1; ++j) {
            const float p = expf(scale * dot_row(qv, k, j) - m) * inv_l;
            const float ds = p * (dot_row(gv, v, j) - delta) * scale;
#pragma unroll
            for (int t = 0; t < EPL; ++t) {
                const int e = lane + 32 * t;
                if (e < d) gq[t] = fmaf(ds, ldf(k + base + j * d + e), gq[t]);
            }
        }
    });
#pragma unroll
    for (int t = 0; t < EPL; ++t) {
        const int e = lane + 32 * t;
        if (e < d) stf(dq + base + i * d + e, gq[t]);
    }
}

// dK_j, dV_j: one warp per key j; the tokens that see key j are the tokens query j sees (symmetric mask).
template <typename T, int EPL>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
clear_bwd_key_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
                     const T *__restrict__ d_out, const float *__restrict__ stats, T *__restrict__ dk,
                     T *__restrict__ dv, int grid_h, int grid_w, int n_text, int d,
                     const int32_t *__restrict__ half_width, int n_half_width, float scale)
{
    const int lane = threadIdx.x & 31;
    const int64_t N = (int64_t)n_text + (int64_t)grid_h * grid_w;
    const int64_t j = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (j >= N) return;  // whole warp leaves together
    const int64_t base = (int64_t)blockIdx.y * N * d;
    const float *st = stats + (int64_t)blockIdx.y * N * 3;

    float kv[EPL], vv[EPL], gk[EPL], gv[EPL];
#pragma unroll
    for (int t = 0; t < EPL; ++t) {
        const int e = lane + 32 * t;
        kv[t] = e < d ? ldf(k + base + j * d + e) : 0.f;
        vv[t] = e < d ? ldf(v + base + j * d + e) : 0.f;
        gk[t] = gv[t] = 0.f;
    }
    auto dot_row = [&](const float (&a)[EPL], const T *__restrict__ rows, int64_t i) {
        float part = 0.f;
#pragma unroll
        for (int t = 0; t < EPL; ++t) {
            const int e = lane + 32 * t;
            if (e < d) part = fmaf(a[t], ldf(rows + base + i * d + e), part);
        }
        return warp_sum(part);
    };
    auto run = [&](int64_t i0, int64_t i1) {
        for (int64_t i = i0; i < i1; ++i) {
            const float m = st[i * 3], inv_l = st[i * 3 + 1], delta = st[i * 3 + 2];
            const float p = expf(scale * dot_row(kv, q, i) - m) * inv_l;
            const float ds = p * (dot_row(vv, d_out, i) - delta) * scale;
#pragma unroll
            for (int t = 0; t < EPL; ++t) {
                const int e = lane + 32 * t;
                if (e < d) {
                    gk[t] = fmaf(ds, ldf(q + base + i * d + e), gk[t]);
                    gv[t] = fmaf(p, ldf(d_out + base + i * d + e), gv[t]);
                }
            }
        }
    };
    if (j < n_text) {
        run(0, N);  // every query sees a text key
    } else {
        run(0, n_text);  // every text query sees every image key
        const int64_t pix = j - n_text;
        const int y = (int)(pix / grid_w), x = (int)(pix % grid_w);
        const int R = n_half_width - 1;
        for (int dy = -R; dy <= R; ++dy) {
            const int yy = y + dy;
            if (yy < 0 || yy >= grid_h) continue;
            const int hw = half_width[dy < 0 ? -dy : dy];
            const int lo = max(x - hw, 0), hi = min(x + hw, grid_w - 1);
            const int64_t row0 = (int64_t)n_text + (int64_t)yy * grid_w;
            run(row0 + lo, row0 + hi + 1);
        }
    }
#pragma unroll
    for (int t = 0; t < EPL; ++t) {
        const int e = lane + 32 * t;
        if (e < d) {
            stf(dk + base + j * d + e, gk[t]);
            stf(dv + base + j * d + e, gv[t]);
        }
    }
}

template <typename T>
int launch_bwd_typed(const clear_plan &p, const void *q, const void *k, const void *v, const void *d_out, void *dq,
                     void *dk, void *dv, float scale, cudaStream_t stream)
{
    const Shape &s = p.shape;
    const int64_t N = (int64_t)s.n_text + (int64_t)s.grid_h * s.grid_w;
    // row statistics (m, 1 / l, delta) of every query: owned by the plan, allocated on its first backward call
    // (calls of one plan are ordered on the device, so one buffer serves them all)
    if (!p.d_bwd_stats) {
        cudaError_t e = cudaMalloc((void **)&p.d_bwd_stats, (size_t)s.B * s.H * N * 3 * sizeof(float));
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            return e == cudaErrorMemoryAllocation ? CLEAR_ERR_NO_MEMORY : CLEAR_ERR_CUDA;
        }
    }
    dim3 grid((unsigned)((N + kWarpsPerBlock - 1) / kWarpsPerBlock), (unsigned)(s.B * s.H));
    dim3 block(kWarpsPerBlock * 32);
    const int n_hw = (int)p.sch.half_width.size();
    const int epl = (s.head_dim + 31) / 32;
#define CLEAR_BWD_CASE(E)                                                                                               \
    case E:                                                                                                             \
        clear_bwd_query_kernel<T, E><<<grid, block, 0, stream>>>((const T *)q, (const T *)k, (const T *)v,             \
                                                                 (const T *)d_out, (T *)dq, p.d_bwd_stats, s.grid_h,    \
                                                                 s.grid_w, s.n_text, s.head_dim, p.d_half_width, n_hw,  \
                                                                 scale);                                                \
        clear_bwd_key_kernel<T, E><<<grid, block, 0, stream>>>((const T *)q, (const T *)k, (const T *)v,               \
                                                               (const T *)d_out, p.d_bwd_stats, (T *)dk, (T *)dv,       \
                                                               s.grid_h, s.grid_w, s.n_text, s.head_dim,                \
                                                               p.d_half_width, n_hw, scale);                            \
        break;
    switch (epl) {
        CLEAR_BWD_CASE(1)
        CLEAR_BWD_CASE(2)
        CLEAR_BWD_CASE(3)
        CLEAR_BWD_CASE(4)
        CLEAR_BWD_CASE(5)
        CLEAR_BWD_CASE(6)
        CLEAR_BWD_CASE(7)
        CLEAR_BWD_CASE(8)
        default:
            return CLEAR_ERR_UNSUPPORTED;
    }
#undef CLEAR_BWD_CASE
    CLEAR_CUDA_TRY(cudaGetLastError());
    return CLEAR_OK;
}

}  // namespace

int launch_bwd(const clear_plan &p, const void *q, const void *k, const void *v, const void *d_out, void *dq, void *dk,
               void *dv, float scale, cudaStream_t stream)
{
    if (p.shape.dtype == CLEAR_F32) return launch_bwd_typed<float>(p, q, k, v, d_out, dq, dk, dv, scale, stream);
    return launch_bwd_typed<__nv_bfloat16>(p, q, k, v, d_out, dq, dk, dv, scale, stream);
}

}  // namespace clear
