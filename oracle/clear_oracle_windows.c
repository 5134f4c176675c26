/*
 * Attention under the other image-to-image masks the paper discusses, as plain fp64 CPU loops.
 *
 * TEST INFRASTRUCTURE ONLY (the yardstick of the CUDA library's window kinds; never on the product
 * path; shares no code, header, table or constant with the CUDA library, nor with the other oracle
 * files: what it needs of them is restated here).
 *
 * Every mask keeps the joint text-image rule of Eq. 3 -- a pair is allowed when either token is a
 * text token (text tokens come first) -- and differs in the image-to-image part, with image token p
 * at row p / grid_w, column p % grid_w:
 *   kind 0  disc      dx^2 + dy^2 < r^2                                   (Eq. 3, CLEAR; a = r)
 *   kind 1  square    max(|dx|, |dy|) < r: the square sliding window of Neighborhood Attention that
 *                     Sec. 3.2 sets the disc against ("about pi / 4 times" its cost)    (a = r)
 *   kind 2  windows   both tokens in the same w x w window of the grid shifted by s: the Swin
 *                     baseline of the appendix (w = 16, s = 8 in odd layers); no wrap-around
 *                                                                          (a = w, b = s)
 *   kind 3  strided   (xj - xi) mod r == l mod r  and  (yj - yi) mod r == l div r, non-negative
 *                     remainders: the strided baseline of the appendix at layer l     (a = r, b = l)
 * The attention itself is Eq. 1 over the allowed keys, one query at a time, max-subtracted natural
 * exponential, everything in double; inputs bf16 bit patterns, fp32 or fp64, widened exactly.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { W_BF16 = 0, W_F32 = 1, W_F64 = 2 };
enum { W_DISC = 0, W_SQUARE = 1, W_WINDOWS = 2, W_STRIDED = 3 };

static double widen(const void *base, int dtype, int64_t idx)
{
    if (dtype == W_F64) return ((const double *)base)[idx];
    if (dtype == W_F32) return (double)((const float *)base)[idx];
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

static int64_t floor_div(int64_t a, int64_t b) { return a >= 0 ? a / b : -((-a + b - 1) / b); }
static int64_t pos_mod(int64_t a, int64_t b) { return ((a % b) + b) % b; }

static int allowed(int kind, double a, double b, int64_t i, int64_t j, int grid_w, int n_text)
{
    if (i < n_text || j < n_text) return 1;
    const int64_t pi = i - n_text, pj = j - n_text;
    const int64_t yi = pi / grid_w, xi = pi % grid_w, yj = pj / grid_w, xj = pj % grid_w;
    const int64_t dx = xj - xi, dy = yj - yi;
    switch (kind) {
        case W_DISC: return (double)(dx * dx + dy * dy) < a * a;
        case W_SQUARE: return (double)(dx < 0 ? -dx : dx) < a && (double)(dy < 0 ? -dy : dy) < a;
        case W_WINDOWS: {
            const int64_t w = (int64_t)a, s = (int64_t)b;
            return floor_div(xi + s, w) == floor_div(xj + s, w) && floor_div(yi + s, w) == floor_div(yj + s, w);
        }
        case W_STRIDED: {
            const int64_t r = (int64_t)a, l = (int64_t)b;
            return pos_mod(dx, r) == l % r && pos_mod(dy, r) == (l / r) % r;
        }
        default: return 0;
    }
}

static int bad_kind(int kind, double a, double b)
{
    if (kind < W_DISC || kind > W_STRIDED || !isfinite(a) || !isfinite(b)) return 1;
    if ((kind == W_DISC || kind == W_SQUARE) && !(a > 0.0)) return 1;
    if ((kind == W_WINDOWS || kind == W_STRIDED) && (a < 1.0 || b < 0.0)) return 1;
    return 0;
}

/* row[j] = M[i, j]; returns the number of ones, -1 on a bad argument. */
int64_t clear_oracle_window_row(int kind, double a, double b, int64_t i, int grid_h, int grid_w, int n_text, uint8_t *row)
{
    if (bad_kind(kind, a, b) || grid_h <= 0 || grid_w <= 0 || n_text < 0) return -1;
    const int64_t N = (int64_t)n_text + (int64_t)grid_h * grid_w;
    int64_t cnt = 0;
    for (int64_t j = 0; j < N; ++j) {
        row[j] = (uint8_t)allowed(kind, a, b, i, j, grid_w, n_text);
        cnt += row[j];
    }
    return cnt;
}

/* counts[i] = sum_j M[i, j] by visiting every pair; returns sum(M), -1 on a bad argument. */
int64_t clear_oracle_window_counts(int kind, double a, double b, int grid_h, int grid_w, int n_text, int64_t *counts)
{
    if (bad_kind(kind, a, b) || grid_h <= 0 || grid_w <= 0 || n_text < 0) return -1;
    const int64_t N = (int64_t)n_text + (int64_t)grid_h * grid_w;
    int64_t total = 0;
#pragma omp parallel for schedule(static) reduction(+ : total)
    for (int64_t i = 0; i < N; ++i) {
        int64_t c = 0;
        for (int64_t j = 0; j < N; ++j) c += allowed(kind, a, b, i, j, grid_w, n_text);
        if (counts) counts[i] = c;
        total += c;
    }
    return total;
}

/* out: [B, H, N, d] doubles.  Returns 0, -1 on a bad argument, -2 out of memory. */
int clear_oracle_window_attn(const void *q, const void *k, const void *v, int dtype, int B, int H, int grid_h, int grid_w,
                             int n_text, int d, int kind, double a, double b, double scale, double *out)
{
    if (bad_kind(kind, a, b) || B <= 0 || H <= 0 || grid_h <= 0 || grid_w <= 0 || n_text < 0 || d <= 0) return -1;
    if (!isfinite(scale) || dtype < W_BF16 || dtype > W_F64) return -1;
    const int64_t N = (int64_t)n_text + (int64_t)grid_h * grid_w;
    const int64_t rows = (int64_t)B * H * N;
    int failed = 0;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)N);
        uint8_t *row = (uint8_t *)malloc((size_t)N);
        if (!s || !row) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp barrier
        if (!failed) {
#pragma omp for schedule(dynamic, 16)
            for (int64_t t = 0; t < rows; ++t) {
                const int64_t bh = t / N, i = t % N, base = bh * N * d;
                double m = -INFINITY;
                for (int64_t j = 0; j < N; ++j) {
                    row[j] = (uint8_t)allowed(kind, a, b, i, j, grid_w, n_text);
                    if (!row[j]) continue;
                    double acc = 0.0;
                    for (int c = 0; c < d; ++c) acc += widen(q, dtype, base + i * d + c) * widen(k, dtype, base + j * d + c);
                    s[j] = scale * acc;
                    if (s[j] > m) m = s[j];
                }
                double l = 0.0;
                for (int64_t j = 0; j < N; ++j)
                    if (row[j]) {
                        s[j] = exp(s[j] - m);
                        l += s[j];
                    }
                for (int c = 0; c < d; ++c) out[t * d + c] = 0.0;
                for (int64_t j = 0; j < N; ++j)
                    if (row[j])
                        for (int c = 0; c < d; ++c) out[t * d + c] += s[j] / l * widen(v, dtype, base + j * d + c);
            }
        }
        free(s);
        free(row);
    }
    return failed ? -2 : 0;
}
