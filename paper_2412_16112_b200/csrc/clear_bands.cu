// Row-band parallel form of the operator (Sec. 3.4): the pieces besides the attention kernel itself.
//
// Each GPU owns a band of image rows and holds the text tokens.  Image queries of a band need keys of at most
// `reach` rows beyond it (the halo the neighbours send); a text query needs every key, so each GPU leaves, per
// text row, the un-normalised result over ITS keys with the row's maximum and sum, and the merge over GPUs is
// the merge of a split softmax: exact, and as cheap to exchange as the patch-wise average of Eq. 7, which is
// here as the second mode of the same merge kernel.
//   clear_text_export_kernel  partial results of the key splits of one GPU -> one (O, m, l) record per text row
//   clear_text_merge_kernel   records of all GPUs -> bf16 text rows (exact merge, or Eq. 7's average)
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>

#include "clear_internal.hpp"

namespace clear {
namespace {

// One block per (text row, bh), one thread per channel.  Record layout: D values of O (relative to m), then m
// (log2 units, scale included), then l.
template <int D>
__global__ void __launch_bounds__(D)
clear_text_export_kernel(const float *__restrict__ partial_o, const float *__restrict__ partial_ml,
                         float *__restrict__ records, int n_text, int n_splits, int n_slots)
{
    const int row = blockIdx.x, bh = blockIdx.y, e = threadIdx.x;
    const int tq = row >> 7, rr = row & 127;
    const int64_t slot0 = ((int64_t)bh * n_slots + (int64_t)tq * n_splits) * 128 + rr;
    float m = -INFINITY;
    for (int s = 0; s < n_splits; ++s) m = fmaxf(m, partial_ml[(slot0 + (int64_t)s * 128) * 2]);
    float num = 0.f, den = 0.f;
    for (int s = 0; s < n_splits; ++s) {
        const int64_t rowi = slot0 + (int64_t)s * 128;
        const float ms = partial_ml[rowi * 2];
        const float w = ms == -INFINITY ? 0.f : exp2f(ms - m);
        den = fmaf(w, partial_ml[rowi * 2 + 1], den);
        num = fmaf(w, partial_o[rowi * D + e], num);
    }
    float *rec = records + ((int64_t)bh * n_text + row) * (D + 2);
    rec[e] = num;
    if (e == 0) {
        rec[D] = m;
        rec[D + 1] = den;
    }
}

// records: [n_parts][BH][n_text][D + 2].  mode CLEAR_TEXT_MERGE_EXACT: sum_p w_p O_p / sum_p w_p l_p with
// w_p = 2^(m_p - max m); CLEAR_TEXT_MERGE_AVERAGE (Eq. 7): (1 / n_parts) sum_p O_p / l_p.
template <int D>
__global__ void __launch_bounds__(D)
clear_text_merge_kernel(const float *__restrict__ records, __nv_bfloat16 *__restrict__ out, int n_parts, int n_text,
                        int64_t out_tokens, int mode)
{
    const int row = blockIdx.x, bh = blockIdx.y, e = threadIdx.x;
    const int64_t part_stride = (int64_t)gridDim.y * n_text * (D + 2);
    const float *rec0 = records + ((int64_t)bh * n_text + row) * (D + 2);
    float result;
    if (mode == CLEAR_TEXT_MERGE_EXACT) {
        float m = -INFINITY;
        for (int p = 0; p < n_parts; ++p) m = fmaxf(m, rec0[p * part_stride + D]);
        float num = 0.f, den = 0.f;
        for (int p = 0; p < n_parts; ++p) {
            const float *rec = rec0 + p * part_stride;
            const float w = rec[D] == -INFINITY ? 0.f : exp2f(rec[D] - m);
            den = fmaf(w, rec[D + 1], den);
            num = fmaf(w, rec[e], num);
        }
        result = den > 0.f ? num / den : 0.f;
    } else {
        float acc = 0.f;
        for (int p = 0; p < n_parts; ++p) {
            const float *rec = rec0 + p * part_stride;
            acc += rec[D + 1] > 0.f ? rec[e] / rec[D + 1] : 0.f;
        }
        result = acc / (float)n_parts;
    }
    out[((int64_t)bh * out_tokens + row) * D + e] = __float2bfloat16_rn(result);
}

}  // namespace

int launch_text_export(const clear_plan &p, void *records, cudaStream_t stream)
{
    const Shape &s = p.shape;
    if (p.sch.n_partial_slots <= 0 || s.n_text <= 0) return CLEAR_ERR_PLAN_MISMATCH;
    dim3 grid((unsigned)s.n_text, (unsigned)(s.B * s.H));
    if (s.head_dim == 128)
        clear_text_export_kernel<128><<<grid, 128, 0, stream>>>(p.d_partial_o, p.d_partial_ml, static_cast<float *>(records),
                                                                 s.n_text, p.sch.n_text_splits, p.sch.n_partial_slots);
    else if (s.head_dim == 64)
        clear_text_export_kernel<64><<<grid, 64, 0, stream>>>(p.d_partial_o, p.d_partial_ml, static_cast<float *>(records),
                                                               s.n_text, p.sch.n_text_splits, p.sch.n_partial_slots);
    else
        return CLEAR_ERR_UNSUPPORTED;
    return cudaGetLastError() == cudaSuccess ? CLEAR_OK : CLEAR_ERR_CUDA;
}

int launch_text_merge(const float *records, int n_parts, int n_bh, int n_text, int head_dim, int mode, void *out,
                      long long out_tokens, cudaStream_t stream)
{
    dim3 grid((unsigned)n_text, (unsigned)n_bh);
    if (head_dim == 128)
        clear_text_merge_kernel<128><<<grid, 128, 0, stream>>>(records, static_cast<__nv_bfloat16 *>(out), n_parts, n_text,
                                                                out_tokens, mode);
    else if (head_dim == 64)
        clear_text_merge_kernel<64><<<grid, 64, 0, stream>>>(records, static_cast<__nv_bfloat16 *>(out), n_parts, n_text,
                                                              out_tokens, mode);
    else
        return CLEAR_ERR_UNSUPPORTED;
    return cudaGetLastError() == cudaSuccess ? CLEAR_OK : CLEAR_ERR_CUDA;
}

}  // namespace clear
