// Q/K preparation in one pass over HBM: RMS normalisation over the head's channels (with a gain), rotary
// position embedding on the two axes of the feature map (Sec. 3.1) with an NTK factor on its base, and a
// constant factor folded into Q (the log-scale attention factor of Sec. 4.3's high-resolution recipe).
//
// The work is elementwise with one reduction per row of d channels, so HBM bounds it: every element of Q and
// K is read once and written once (4 * B * H * N * d * sizeof(element) bytes per call).  One warp owns a
// few token positions (32 / (d / 8) of them) and walks over all (batch, head) rows of those tokens: the angles
// depend on the position only, so their sines and cosines are computed once per token and reused for
// 2 * B * H rows; a lane holds 8 consecutive channels of a row (whole rotary pairs), so a row is one
// coalesced access of 16 bytes per lane for bf16.
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

// Eight consecutive channels of a row (four rotary pairs) per lane: one 16-byte access for bf16, two for fp32.
template <typename T> struct RowIo;
template <> struct RowIo<__nv_bfloat16> {
    static __device__ __forceinline__ void load(const void *base, long long elem, float (&x)[8])
    {
        const uint4 u = *reinterpret_cast<const uint4 *>(static_cast<const __nv_bfloat16 *>(base) + elem);
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);            // a bf16 is the upper half of an fp32
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ void store(void *base, long long elem, const float (&x)[8])
    {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) *reinterpret_cast<__nv_bfloat162 *>(&w[i]) = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
        *reinterpret_cast<uint4 *>(static_cast<__nv_bfloat16 *>(base) + elem) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};
template <> struct RowIo<float> {
    static __device__ __forceinline__ void load(const void *base, long long elem, float (&x)[8])
    {
        const float4 a = *reinterpret_cast<const float4 *>(static_cast<const float *>(base) + elem);
        const float4 b = *reinterpret_cast<const float4 *>(static_cast<const float *>(base) + elem + 4);
        x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
        x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
    }
    static __device__ __forceinline__ void store(void *base, long long elem, const float (&x)[8])
    {
        *reinterpret_cast<float4 *>(static_cast<float *>(base) + elem) = make_float4(x[0], x[1], x[2], x[3]);
        *reinterpret_cast<float4 *>(static_cast<float *>(base) + elem + 4) = make_float4(x[4], x[5], x[6], x[7]);
    }
};

constexpr int kEpl = 8;  // channels per lane

// One row: x -> x / sqrt(mean(x^2) + eps) * gain, every pair turned by its angle, times `factor`.  The lanes
// that share the row exchange their partial sums of squares; `gcs` holds, per pair, the products of the two
// channels' gains with the pair's cosine and sine (they do not change from row to row of a token).
template <int D>
__device__ __forceinline__ void prep_row(float (&x)[kEpl], const float (&gcs)[kEpl / 2][4], float eps, float factor)
{
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < kEpl; ++i) ss = fmaf(x[i], x[i], ss);
#pragma unroll
    for (int off = D / kEpl / 2; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    const float inv = factor * rsqrtf(fmaf(ss, 1.f / D, eps));
#pragma unroll
    for (int p = 0; p < kEpl / 2; ++p) {
        const float a = x[2 * p], b = x[2 * p + 1];
        x[2 * p] = (a * gcs[p][0] - b * gcs[p][1]) * inv;      // g_a a cos - g_b b sin
        x[2 * p + 1] = (a * gcs[p][2] + b * gcs[p][3]) * inv;  // g_a a sin + g_b b cos
    }
}

template <typename T, int D>
__global__ void __launch_bounds__(kPrepThreads, 2) clear_qk_prep_kernel(const __grid_constant__ PrepParams prm)
{
    constexpr int kLanesPerRow = D / kEpl;           // 16 or 8 lanes share a row
    constexpr int kTokensPerWarp = 32 / kLanesPerRow;
    constexpr int kRows = 4;                         // rows in flight per lane and tensor
    using Io = RowIo<T>;
    const int lane = threadIdx.x & 31;
    const int sub = lane / kLanesPerRow;             // which of the warp's tokens
    const int c0 = (lane % kLanesPerRow) * kEpl;
    const long long group0 = (long long)blockIdx.x * kPrepWarps + (threadIdx.x >> 5);
    const long long n_groups = (long long)gridDim.x * kPrepWarps;

    float gq[kEpl], gk[kEpl], freq[kEpl / 2];
    int axis[kEpl / 2];
#pragma unroll
    for (int i = 0; i < kEpl; ++i) {
        gq[i] = prm.gain_q ? __ldg(prm.gain_q + c0 + i) : 1.f;
        gk[i] = prm.gain_k ? __ldg(prm.gain_k + c0 + i) : 1.f;
    }
#pragma unroll
    for (int p = 0; p < kEpl / 2; ++p) {
        freq[p] = prm.freq[c0 / 2 + p];
        axis[p] = prm.axis[c0 / 2 + p];
    }

    const long long row_stride = prm.n_tokens * D;
    for (long long grp = group0; grp * kTokensPerWarp < prm.n_tokens; grp += n_groups) {
        // the lanes of a token beyond the last one follow the last token and store nothing (the row's lanes
        // stay together for the shuffles)
        const long long n_raw = grp * kTokensPerWarp + sub;
        const bool live = n_raw < prm.n_tokens;
        const long long n = live ? n_raw : prm.n_tokens - 1;
        // position of the token: text tokens at the origin, image token p at (y, x) = (p / grid_w, p % grid_w)
        int pos_y = 0, pos_x = 0;
        if (n >= prm.n_text) {
            const long long p = n - prm.n_text;
            pos_y = (int)(p / prm.grid_w);
            pos_x = (int)(p - (long long)pos_y * prm.grid_w);
        }
        float gcs_q[kEpl / 2][4], gcs_k[kEpl / 2][4];
#pragma unroll
        for (int p = 0; p < kEpl / 2; ++p) {
            const int pos = axis[p] == 1 ? pos_y : (axis[p] == 2 ? pos_x : 0);
            float sn, cs;
            sincosf((float)pos * freq[p], &sn, &cs);
            gcs_q[p][0] = gq[2 * p] * cs; gcs_q[p][1] = gq[2 * p + 1] * sn;
            gcs_q[p][2] = gq[2 * p] * sn; gcs_q[p][3] = gq[2 * p + 1] * cs;
            gcs_k[p][0] = gk[2 * p] * cs; gcs_k[p][1] = gk[2 * p + 1] * sn;
            gcs_k[p][2] = gk[2 * p] * sn; gcs_k[p][3] = gk[2 * p + 1] * cs;
        }
        long long elem = n * D + c0;
        int bh = 0;
        for (; bh + kRows <= prm.n_bh; bh += kRows) {
            float xq[kRows][kEpl], xk[kRows][kEpl];
#pragma unroll
            for (int j = 0; j < kRows; ++j) {
                Io::load(prm.q_in, elem + j * row_stride, xq[j]);
                Io::load(prm.k_in, elem + j * row_stride, xk[j]);
            }
#pragma unroll
            for (int j = 0; j < kRows; ++j) {
                prep_row<D>(xq[j], gcs_q, prm.eps, prm.q_factor);
                prep_row<D>(xk[j], gcs_k, prm.eps, 1.f);
                if (live) {
                    Io::store(prm.q_out, elem + j * row_stride, xq[j]);
                    Io::store(prm.k_out, elem + j * row_stride, xk[j]);
                }
            }
            elem += kRows * row_stride;
        }
        for (; bh < prm.n_bh; ++bh) {
            float xq[kEpl], xk[kEpl];
            Io::load(prm.q_in, elem, xq);
            Io::load(prm.k_in, elem, xk);
            prep_row<D>(xq, gcs_q, prm.eps, prm.q_factor);
            prep_row<D>(xk, gcs_k, prm.eps, 1.f);
            if (live) {
                Io::store(prm.q_out, elem, xq);
                Io::store(prm.k_out, elem, xk);
            }
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
        const long long tokens_per_block = (long long)kPrepWarps * (32 / (head_dim / kEpl));
        const long long need = (prm.n_tokens + tokens_per_block - 1) / tokens_per_block;
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
