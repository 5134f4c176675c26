/*
 * Backward pass of the CLEAR attention operator: plain, slow, fp64 CPU statement.
 *
 * TEST INFRASTRUCTURE ONLY.  The yardstick of the CUDA backward kernel; it is never part of the
 * product path, shares no code, header, table or constant with the CUDA library and includes
 * nothing from it.  Only the tests load it.
 *
 * Why it exists: the paper fine-tunes the attention layers by distillation (Sec. 3.3, Eq. 4-6: a
 * flow-matching loss, a prediction loss and an attention-output loss); each of these back-propagates
 * through  O = softmax(scale Q K^T + log M) V  (Eq. 1 under the mask of Eq. 3).  The paper prints no
 * formula for that step; it is the calculus of Eq. 1, written out here per query i over its allowed
 * keys A_i = { j : M_ij = 1 }:
 *     s_ij  = scale q_i . k_j                       p_ij = exp(s_ij) / sum_{j' in A_i} exp(s_ij')
 *     dP_ij = dO_i . v_j                            dS_ij = p_ij (dP_ij - sum_{j'} p_ij' dP_ij')
 *     dQ_i  = scale sum_j dS_ij k_j      dK_j = scale sum_i dS_ij q_i      dV_j = sum_i p_ij dO_i
 * Same readings of Eq. 3 as the forward oracle (strict "<", window clipped at the border, text
 * tokens first, row-major grid, threshold ceil(r^2)); they are restated below, not shared.
 *
 * Two sweeps, so that every output element is written by one thread only: over the queries (row
 * maxima, row sums, the sums  delta_i = sum_j p_ij dP_ij , and dQ), then over the keys (dK, dV),
 * where the mask entry of every (i, j) pair is evaluated again.
 *
 * q, k, v may be bf16 bit patterns, fp32 or fp64 (widened exactly); dO and the three gradients are
 * double.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { BWD_BF16 = 0, BWD_F32 = 1, BWD_F64 = 2 };

static double widen(const void *base, int dtype, int64_t idx)
{
    if (dtype == BWD_F64) return ((const double *)base)[idx];
    if (dtype == BWD_F32) return (double)((const float *)base)[idx];
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16; /* bf16 = top half of an fp32 */
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* Eq. 3, one entry (tokens 0..n_text-1 are text, then the image tokens row by row). */
static int allowed(int64_t i, int64_t j, int grid_w, int n_text, int64_t thr)
{
    if (i < n_text || j < n_text) return 1;
    int64_t pi = i - n_text, pj = j - n_text;
    int64_t dy = pj / grid_w - pi / grid_w, dx = pj % grid_w - pi % grid_w;
    return dx * dx + dy * dy < thr;
}

static double dot(const void *a, int dtype, int64_t ia, const void *b, int dtype_b, int64_t ib, int d)
{
    double acc = 0.0;
    for (int c = 0; c < d; ++c) acc += widen(a, dtype, ia + c) * widen(b, dtype_b, ib + c);
    return acc;
}

/* dq, dk, dv: [B, H, N, d] doubles, fully written.  Returns 0, -1 on a bad argument, -2 out of memory. */
int clear_oracle_attn_bwd(const void *q, const void *k, const void *v, int dtype, const double *d_out,
                          int B, int H, int grid_h, int grid_w, int n_text, int d, double radius,
                          double scale, double *dq, double *dk, double *dv)
{
    if (B <= 0 || H <= 0 || grid_h <= 0 || grid_w <= 0 || n_text < 0 || d <= 0) return -1;
    if (!(radius > 0.0) || !isfinite(radius) || !isfinite(scale)) return -1;
    if (dtype < BWD_BF16 || dtype > BWD_F64) return -1;
    const int64_t N = (int64_t)n_text + (int64_t)grid_h * grid_w;
    const int64_t thr = (int64_t)ceil(radius * radius);
    const int64_t rows = (int64_t)B * H * N;
    double *row_max = (double *)malloc(sizeof(double) * (size_t)rows);
    double *row_sum = (double *)malloc(sizeof(double) * (size_t)rows);
    double *delta = (double *)malloc(sizeof(double) * (size_t)rows);
    if (!row_max || !row_sum || !delta) {
        free(row_max);
        free(row_sum);
        free(delta);
        return -2;
    }

    /* sweep over the queries */
#pragma omp parallel for schedule(dynamic, 8)
    for (int64_t t = 0; t < rows; ++t) {
        const int64_t bh = t / N, i = t % N, base = bh * N * d;
        double m = -INFINITY;
        for (int64_t j = 0; j < N; ++j)
            if (allowed(i, j, grid_w, n_text, thr)) {
                const double s = scale * dot(q, dtype, base + i * d, k, dtype, base + j * d, d);
                if (s > m) m = s;
            }
        double l = 0.0, pdp = 0.0;
        for (int64_t j = 0; j < N; ++j)
            if (allowed(i, j, grid_w, n_text, thr)) {
                const double e = exp(scale * dot(q, dtype, base + i * d, k, dtype, base + j * d, d) - m);
                l += e;
                pdp += e * dot(d_out, BWD_F64, base + i * d, v, dtype, base + j * d, d);
            }
        row_max[t] = m;
        row_sum[t] = l;
        delta[t] = pdp / l; /* sum_j p_ij dP_ij */
        for (int c = 0; c < d; ++c) dq[base + i * d + c] = 0.0;
        for (int64_t j = 0; j < N; ++j)
            if (allowed(i, j, grid_w, n_text, thr)) {
                const double p = exp(scale * dot(q, dtype, base + i * d, k, dtype, base + j * d, d) - m) / l;
                const double ds = p * (dot(d_out, BWD_F64, base + i * d, v, dtype, base + j * d, d) - delta[t]);
                for (int c = 0; c < d; ++c) dq[base + i * d + c] += scale * ds * widen(k, dtype, base + j * d + c);
            }
    }

    /* sweep over the keys */
#pragma omp parallel for schedule(dynamic, 8)
    for (int64_t t = 0; t < rows; ++t) {
        const int64_t bh = t / N, j = t % N, base = bh * N * d;
        for (int c = 0; c < d; ++c) dk[base + j * d + c] = dv[base + j * d + c] = 0.0;
        for (int64_t i = 0; i < N; ++i)
            if (allowed(i, j, grid_w, n_text, thr)) {
                const int64_t r = bh * N + i;
                const double p = exp(scale * dot(q, dtype, base + i * d, k, dtype, base + j * d, d) - row_max[r]) / row_sum[r];
                const double ds = p * (dot(d_out, BWD_F64, base + i * d, v, dtype, base + j * d, d) - delta[r]);
                for (int c = 0; c < d; ++c) {
                    dk[base + j * d + c] += scale * ds * widen(q, dtype, base + i * d + c);
                    dv[base + j * d + c] += p * d_out[base + i * d + c];
                }
            }
    }
    free(row_max);
    free(row_sum);
    free(delta);
    return 0;
}
