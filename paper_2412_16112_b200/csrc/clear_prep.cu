// Q/K preparation in one pass over HBM: RMS normalisation over the head's channels (with a gain), rotary
// position embedding on the two axes of the feature map (Sec. 3.1) with an NTK factor on its base, and a
// constant factor folded into Q (the log-scale attention factor of Sec. 4.3's high-resolution recipe).
//
// The work is elementwise with one reduction per row of d channels, so HBM bounds it: every element of Q and
// K is read once and written once (4 * B * H * N * d * sizeof(element) bytes per call).  One warp owns one
// token position and walks over all (batch, head) rows of that token: the angles depend on the position
// only, so their sines and cosines are computed once per token and reused for 2 * B * H rows; a lane holds
// d / 32 consecutive channels of a row (whole rotary pairs), so a row is one coalesced d-element access.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>

#include "clear_internal.hpp"

namespace clear {
namespace {

constexpr int kPrepThreads = 256;
constexpr int kPrepWarps = kPrepThreads / 32;
constexpr int kMaxPairs = 64;  // head_dim <= 128

struct PrepParams {
    const void *q_in, *k_in;
    void *q_out, *k_out;
    const float *gain_q, *gain_k;  // [d] or null
    int n_bh, n_text, grid_w;
    long long n_tokens;
    float eps, q_factor;
    float freq[kMaxPairs];         // angular frequency of rotary pair p (channels 2p, 2p+1)
    uint8_t axis[kMaxPairs];       // which coordinate of the token's position turns pair p: 0 none, 1 y, 2 x
};

template <typename T, int EPL> struct RowIo;
template <> struct RowIo<__nv_bfloat16, 4> {
    static __device__ __forceinline__ void load(const void *base, long long elem, float (&x)[4])
    {
        const uint2 u = *reinterpret_cast<const uint2 *>(static_cast<const __nv_bfloat16 *>(base) + elem);
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&u.x));
        const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&u.y));
        x[0] = a.x; x[1] = a.y; x[2] = b.x; x[3] = b.y;
    }
    static __device__ __forceinline__ void store(void *base, long long elem, const float (&x)[4])
    {
        uint2 u;
        *reinterpret_cast<__nv_bfloat162 *>(&u.x) = __floats2bfloat162_rn(x[0], x[1]);
        *reinterpret_cast<__nv_bfloat162 *>(&u.y) = __floats2bfloat162_rn(x[2], x[3]);
        *reinterpret_cast<uint2 *>(static_cast<__nv_bfloat16 *>(base) + elem) = u;
    }
};
template <> struct RowIo<__nv_bfloat16, 2> {
    static __device__ __forceinline__ void load(const void *base, long long elem, float (&x)[2])
    {
        const uint32_t u = *reinterpret_cast<const uint32_t *>(static_cast<const __nv_bfloat16 *>(base) + elem);
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&u));
        x[0] = a.x; x[1] = a.y;
    }
    static __device__ __forceinline__ void store(void *base, long long elem, const float (&x)[2])
    {
        uint32_t u;
        *reinterpret_cast<__nv_bfloat162 *>(&u) = __floats2bfloat162_rn(x[0], x[1]);
        *reinterpret_cast<uint32_t *>(static_cast<__nv_bfloat16 *>(base) + elem) = u;
    }
};
template <> struct RowIo<float, 4> {
    static __device__ __forceinline__ void load(const void *base, long long elem, float (&x)[4])
    {
        const float4 v = *reinterpret_cast<const float4 *>(static_cast<const float *>(base) + elem);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    }
    static __device__ __forceinline__ void store(void *base, long long elem, const float (&x)[4])
    {
        *reinterpret_cast<float4 *>(static_cast<float *>(base) + elem) = make_float4(x[0], x[1], x[2], x[3]);
    }
};
template <> struct RowIo<float, 2> {
    static __device__ __forceinline__ void load(const void *base, long long elem, float (&x)[2])
    {
        const float2 v = *reinterpret_cast<const float2 *>(static_cast<const float *>(base) + elem);
        x[0] = v.x; x[1] = v.y;
    }
    static __device__ __forceinline__ void store(void *base, long long elem, const float (&x)[2])
    {
        *reinterpret_cast<float2 *>(static_cast<float *>(base) + elem) = make_float2(x[0], x[1]);
    }
};

// One row: x -> x / sqrt(mean(x^2) + eps) * gain, every pair turned by its angle, times `factor`.
template <int EPL, int D>
__device__ __forceinline__ void prep_row(float (&x)[EPL], const float (&g)[EPL], const float (&cs)[EPL / 2][2], float eps,
                                         float factor)
{
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < EPL; ++i) ss = fmaf(x[i], x[i], ss);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    const float inv = factor / sqrtf(ss * (1.f / D) + eps);
#pragma unroll
    for (int p = 0; p < EPL / 2; ++p) {
        const float a = x[2 * p] * g[2 * p] * inv, b = x[2 * p + 1] * g[2 * p + 1] * inv;
        x[2 * p] = a * cs[p][0] - b * cs[p][1];
        x[2 * p + 1] = a * cs[p][1] + b * cs[p][0];
    }
}

template <typename T, int D>
__global__ void __launch_bounds__(kPrepThreads, 3) clear_qk_prep_kernel(const __grid_constant__ PrepParams prm)
{
    constexpr int EPL = D / 32;  // channels per lane
    constexpr int kRows = 4;     // rows in flight per lane and tensor
    using Io = RowIo<T, EPL>;
    const int lane = threadIdx.x & 31;
    const long long warp0 = (long long)blockIdx.x * kPrepWarps + (threadIdx.x >> 5);
    const long long n_warps = (long long)gridDim.x * kPrepWarps;
    const int c0 = lane * EPL;

    float gq[EPL], gk[EPL], freq[EPL / 2];
    int axis[EPL / 2];
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
        gq[i] = prm.gain_q ? __ldg(prm.gain_q + c0 + i) : 1.f;
        gk[i] = prm.gain_k ? __ldg(prm.gain_k + c0 + i) : 1.f;
    }
#pragma unroll
    for (int p = 0; p < EPL / 2; ++p) {
        freq[p] = prm.freq[c0 / 2 + p];
        axis[p] = prm.axis[c0 / 2 + p];
    }

    for (long long n = warp0; n < prm.n_tokens; n += n_warps) {
        // position of the token: text tokens at the origin, image token p at (y, x) = (p / grid_w, p % grid_w)
        int pos_y = 0, pos_x = 0;
        if (n >= prm.n_text) {
            const long long p = n - prm.n_text;
            pos_y = (int)(p / prm.grid_w);
            pos_x = (int)(p - (long long)pos_y * prm.grid_w);
        }
        float cs[EPL / 2][2];
#pragma unroll
        for (int p = 0; p < EPL / 2; ++p) {
            const int pos = axis[p] == 1 ? pos_y : (axis[p] == 2 ? pos_x : 0);
            sincosf((float)pos * freq[p], &cs[p][1], &cs[p][0]);
        }
        long long elem = n * D + c0;
        const long long row_stride = prm.n_tokens * D;
        int bh = 0;
        for (; bh + kRows <= prm.n_bh; bh += kRows) {
            float xq[kRows][EPL], xk[kRows][EPL];
#pragma unroll
            for (int j = 0; j < kRows; ++j) {
                Io::load(prm.q_in, elem + j * row_stride, xq[j]);
                Io::load(prm.k_in, elem + j * row_stride, xk[j]);
            }
#pragma unroll
            for (int j = 0; j < kRows; ++j) {
                prep_row<EPL, D>(xq[j], gq, cs, prm.eps, prm.q_factor);
                prep_row<EPL, D>(xk[j], gk, cs, prm.eps, 1.f);
                Io::store(prm.q_out, elem + j * row_stride, xq[j]);
                Io::store(prm.k_out, elem + j * row_stride, xk[j]);
            }
            elem += kRows * row_stride;
        }
        for (; bh < prm.n_bh; ++bh) {
            float xq[EPL], xk[EPL];
            Io::load(prm.q_in, elem, xq);
            Io::load(prm.k_in, elem, xk);
            prep_row<EPL, D>(xq, gq, cs, prm.eps, prm.q_factor);
            prep_row<EPL, D>(xk, gk, cs, prm.eps, 1.f);
            Io::store(prm.q_out, elem, xq);
            Io::store(prm.k_out, elem, xk);
            elem += row_stride;
        }
    }
}

}  // namespace

int launch_qk_prep(const void *q_in, const void *k_in, void *q_out, void *k_out, const float *gain_q, const float *gain_k,
                   int n_bh, int grid_h, int grid_w, int n_text, int head_dim, int dtype, const int axes_dim[3],
                   double theta, double ntk_factor, float eps, float q_factor, cudaStream_t stream)
{
    PrepParams prm{};
    prm.q_in = q_in;
    prm.k_in = k_in;
    prm.q_out = q_out;
    prm.k_out = k_out;
    prm.gain_q = gain_q;
    prm.gain_k = gain_k;
    prm.n_bh = n_bh;
    prm.n_text = n_text;
    prm.grid_w = grid_w;
    prm.n_tokens = (long long)n_text + (long long)grid_h * grid_w;
    prm.eps = eps;
    prm.q_factor = q_factor;
    // frequencies in double on the host: w_k = base'^(-2k/dim), base' = theta * ntk^(dim/(dim-2))
    int pair = 0;
    for (int a = 0; a < 3; ++a) {
        const int dim = axes_dim[a];
        double base = theta;
        if (dim > 2) base *= std::pow(ntk_factor, (double)dim / (double)(dim - 2));
        for (int k = 0; k < dim / 2; ++k, ++pair) {
            prm.freq[pair] = (float)std::pow(base, -2.0 * (double)k / (double)dim);
            prm.axis[pair] = (uint8_t)a;
        }
    }
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return CLEAR_ERR_CUDA;
    if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return CLEAR_ERR_CUDA;
    // whole waves of resident blocks, never more warps than tokens
    auto launch = [&](auto kernel) -> int {
        int per_sm = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kPrepThreads, 0) != cudaSuccess || per_sm < 1)
            return CLEAR_ERR_CUDA;
        long long blocks = (long long)n_sm * per_sm;
        const long long need = (prm.n_tokens + kPrepWarps - 1) / kPrepWarps;
        if (blocks > need) blocks = need;
        kernel<<<dim3((unsigned)blocks), dim3(kPrepThreads), 0, stream>>>(prm);
        return CLEAR_OK;
    };
    int rc;
    if (dtype == CLEAR_BF16)
        rc = head_dim == 128 ? launch(clear_qk_prep_kernel<__nv_bfloat16, 128>) : launch(clear_qk_prep_kernel<__nv_bfloat16, 64>);
    else
        rc = head_dim == 128 ? launch(clear_qk_prep_kernel<float, 128>) : launch(clear_qk_prep_kernel<float, 64>);
    if (rc != CLEAR_OK) return rc;
    return cudaGetLastError() == cudaSuccess ? CLEAR_OK : CLEAR_ERR_CUDA;
}

}  // namespace clear
