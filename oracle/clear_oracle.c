/*
 * CLEAR attention oracle: plain, slow, fp64 CPU statement of the operator.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the yardstick the CUDA path is
 * checked against; it is never part of the product path.  It shares no code,
 * header, table or constant with the CUDA library and includes nothing from
 * it.  Only the tests, the smoke check and the bench's cpu-baseline leg load it.
 *
 * What it computes (one query at a time, no tiling, no online softmax):
 *   - the 0/1 mask row M[i, :] exactly as Eq. 3 writes it: a pair (i, j) is
 *     allowed when i is a text token, or j is a text token, or the squared
 *     Euclidean distance between the two image tokens' grid positions is
 *     strictly below r^2  (Sec. 3.2, Eq. 3; text tokens come first);
 *   - the masked softmax attention of Eq. 1 over the allowed keys,
 *       out_i = sum_j softmax_j(scale * q_i . k_j) v_j ,
 *     with a max-subtracted natural exponential, everything in double.
 *
 * Readings of points the paper leaves open (each is pinned by a CPU test):
 *   - strict "<" at distance r (Eq. 3 and the prose of Sec. 3.2);
 *   - the window is clipped at the grid border: no wrap-around, no shifting;
 *     both are fixed by the FLOP figures the paper prints (Fig. 2 caption's
 *     4 * sum(M) * c formula against Tab. 1 and the appendix efficiency table);
 *   - image token p sits at row y = p / grid_w, column x = p % grid_w
 *     (row-major; a convention of the interface, the paper is silent:
 *     parity on non-square grids is pinned by this convention only);
 *   - tensors are [B, H, N, d] contiguous, N = n_text + grid_h * grid_w, and
 *     the mask is the same for every batch entry and head;
 *   - a real radius r is used through the integer threshold ceil(r^2): for
 *     integer squared distances  d2 < r^2  <=>  d2 < ceil(r^2).
 *
 * Inputs may be given as bf16 bit patterns, fp32 or fp64; they are widened
 * exactly to double before any arithmetic.  Output is always double.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_BF16 = 0, ORACLE_F32 = 1, ORACLE_F64 = 2 };

static double widen(const void *base, int dtype, int64_t idx)
{
    if (dtype == ORACLE_F64) return ((const double *)base)[idx];
    if (dtype == ORACLE_F32) return (double)((const float *)base)[idx];
    /* bf16: the 16 stored bits are the top half of an IEEE fp32 */
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* ceil(r^2) as an integer threshold for integer squared distances (reading of
 * Eq. 3 for real r).  r*r is formed in double. */
static int64_t radius_threshold(double radius)
{
    return (int64_t)ceil(radius * radius);
}

/* Eq. 3, one entry.  Tokens 0..n_text-1 are text (the paper's 1-based
 * "i <= n_text"), the rest are image tokens in row-major grid order. */
static int mask_entry(int64_t i, int64_t j, int grid_w, int n_text, int64_t thr)
{
    if (i < n_text || j < n_text) return 1;
    int64_t pi = i - n_text, pj = j - n_text;
    int64_t yi = pi / grid_w, xi = pi % grid_w;
    int64_t yj = pj / grid_w, xj = pj % grid_w;
    int64_t dx = xj - xi, dy = yj - yi;
    return (dx * dx + dy * dy < thr) ? 1 : 0;
}

/* Fill row[0..N) with M[i, j] for all j.  Returns the number of ones. */
int64_t clear_oracle_mask_row(int64_t i, int grid_h, int grid_w, int n_text,
                              double radius, uint8_t *row)
{
    int64_t N = (int64_t)n_text + (int64_t)grid_h * grid_w;
    int64_t thr = radius_threshold(radius);
    int64_t cnt = 0;
    for (int64_t j = 0; j < N; ++j) {
        int m = mask_entry(i, j, grid_w, n_text, thr);
        row[j] = (uint8_t)m;
        cnt += m;
    }
    return cnt;
}

/* Per-query count of allowed keys, counts[i] = sum_j M[i, j], by visiting every
 * (i, j) pair.  Returns sum(M).  (The FLOP figure of Fig. 2's caption is
 * 4 * sum(M) * c.) */
int64_t clear_oracle_mask_counts(int grid_h, int grid_w, int n_text,
                                 double radius, int64_t *counts /* may be NULL */)
{
    int64_t n = (int64_t)grid_h * grid_w;
    int64_t N = (int64_t)n_text + n;
    int64_t thr = radius_threshold(radius);
    int64_t total = 0;
#pragma omp parallel for schedule(static) reduction(+ : total)
    for (int64_t i = 0; i < N; ++i) {
        int64_t c = 0;
        if (i < n_text) {
            for (int64_t j = 0; j < N; ++j) c += mask_entry(i, j, grid_w, n_text, thr);
        } else {
            /* same predicate, written over (yj, xj) so the compiler can
             * vectorise the inner loop; text keys are always allowed */
            int64_t pi = i - n_text;
            int yi = (int)(pi / grid_w), xi = (int)(pi % grid_w);
            c = n_text;
            for (int yj = 0; yj < grid_h; ++yj) {
                int64_t dy2 = (int64_t)(yj - yi) * (yj - yi);
                int64_t cr = 0;
                for (int xj = 0; xj < grid_w; ++xj) {
                    int64_t dx = xj - xi;
                    cr += (dx * dx + dy2 < thr);
                }
                c += cr;
            }
        }
        if (counts) counts[i] = c;
        total += c;
    }
    return total;
}

/* One query row of Eq. 1 restricted by Eq. 3.  s and row are scratch of
 * length N.  out_row has d doubles. */
static void attend_one(const void *q, const void *k, const void *v, int dtype,
                       int64_t bh, int64_t i, int grid_h, int grid_w,
                       int n_text, int d, int64_t thr, double scale,
                       double *s, uint8_t *row, double *qrow, double *out_row)
{
    int64_t N = (int64_t)n_text + (int64_t)grid_h * grid_w;
    int64_t base = bh * N * d;
    for (int c = 0; c < d; ++c) qrow[c] = widen(q, dtype, base + i * d + c);

    /* materialise the mask row */
    for (int64_t j = 0; j < N; ++j) row[j] = (uint8_t)mask_entry(i, j, grid_w, n_text, thr);

    /* logits on the allowed keys and their maximum */
    double m = -INFINITY;
    for (int64_t j = 0; j < N; ++j) {
        if (!row[j]) continue;
        double acc = 0.0;
        for (int c = 0; c < d; ++c) acc += qrow[c] * widen(k, dtype, base + j * d + c);
        s[j] = scale * acc;
        if (s[j] > m) m = s[j];
    }
    /* softmax weights */
    double l = 0.0;
    for (int64_t j = 0; j < N; ++j) {
        if (!row[j]) continue;
        s[j] = exp(s[j] - m);
        l += s[j];
    }
    /* weighted sum of the value rows */
    for (int c = 0; c < d; ++c) out_row[c] = 0.0;
    for (int64_t j = 0; j < N; ++j) {
        if (!row[j]) continue;
        double p = s[j] / l;
        for (int c = 0; c < d; ++c) out_row[c] += p * widen(v, dtype, base + j * d + c);
    }
}

static int check_args(int B, int H, int grid_h, int grid_w, int n_text, int d,
                      double radius, double scale, int dtype)
{
    if (B <= 0 || H <= 0 || grid_h <= 0 || grid_w <= 0 || n_text < 0 || d <= 0) return -1;
    if (!(radius > 0.0) || !isfinite(radius) || !isfinite(scale)) return -1;
    if (dtype < ORACLE_BF16 || dtype > ORACLE_F64) return -1;
    return 0;
}

/* Selected query rows.  rows[3*t + {0,1,2}] = (b, h, i); out is [n_rows, d]
 * doubles.  Returns 0, or -1 on a bad argument. */
int clear_oracle_attn_rows(const void *q, const void *k, const void *v, int dtype,
                           int B, int H, int grid_h, int grid_w, int n_text, int d,
                           double radius, double scale,
                           const int64_t *rows, int64_t n_rows, double *out)
{
    if (check_args(B, H, grid_h, grid_w, n_text, d, radius, scale, dtype)) return -1;
    int64_t N = (int64_t)n_text + (int64_t)grid_h * grid_w;
    int64_t thr = radius_threshold(radius);
    for (int64_t t = 0; t < n_rows; ++t) {
        if (rows[3 * t] < 0 || rows[3 * t] >= B || rows[3 * t + 1] < 0 ||
            rows[3 * t + 1] >= H || rows[3 * t + 2] < 0 || rows[3 * t + 2] >= N)
            return -1;
    }
    int bad = 0;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)N);
        uint8_t *row = (uint8_t *)malloc((size_t)N);
        double *qrow = (double *)malloc(sizeof(double) * (size_t)d);
        if (!s || !row || !qrow) {
#pragma omp atomic write
            bad = 1;
        }
#pragma omp barrier
        if (!bad) {
#pragma omp for schedule(dynamic, 1)
            for (int64_t t = 0; t < n_rows; ++t) {
                int64_t bh = rows[3 * t] * H + rows[3 * t + 1];
                attend_one(q, k, v, dtype, bh, rows[3 * t + 2], grid_h, grid_w,
                           n_text, d, thr, scale, s, row, qrow, out + t * d);
            }
        }
        free(s);
        free(row);
        free(qrow);
    }
    return bad ? -2 : 0;
}

/* Every query: out is [B, H, N, d] doubles. */
int clear_oracle_attn(const void *q, const void *k, const void *v, int dtype,
                      int B, int H, int grid_h, int grid_w, int n_text, int d,
                      double radius, double scale, double *out)
{
    if (check_args(B, H, grid_h, grid_w, n_text, d, radius, scale, dtype)) return -1;
    int64_t N = (int64_t)n_text + (int64_t)grid_h * grid_w;
    int64_t thr = radius_threshold(radius);
    int64_t total = (int64_t)B * H * N;
    int bad = 0;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)N);
        uint8_t *row = (uint8_t *)malloc((size_t)N);
        double *qrow = (double *)malloc(sizeof(double) * (size_t)d);
        if (!s || !row || !qrow) {
#pragma omp atomic write
            bad = 1;
        }
#pragma omp barrier
        if (!bad) {
#pragma omp for schedule(dynamic, 16)
            for (int64_t t = 0; t < total; ++t) {
                int64_t bh = t / N, i = t % N;
                attend_one(q, k, v, dtype, bh, i, grid_h, grid_w, n_text, d, thr,
                           scale, s, row, qrow, out + t * d);
            }
        }
        free(s);
        free(row);
        free(qrow);
    }
    return bad ? -2 : 0;
}

/* Threads the parallel loops above will use. */
int clear_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
