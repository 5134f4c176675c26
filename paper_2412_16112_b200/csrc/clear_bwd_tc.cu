// Backward pass of the CLEAR attention operator on the sm_100a tensor cores (bf16 tensors, fp32 accumulation): dQ, dK,
// dV for an upstream gradient dO of  O = softmax(scale Q K^T + log M) V  (Eq. 1 under the mask of Eq. 3), the step
// through which the distillation losses of Sec. 3.3 (Eq. 4-6) reach the attention parameters.
//
// One kernel, two roles; a CTA runs one work item of the forward tile schedule: a STATIONARY tile of 128 tokens (an
// 8 x 16 patch of the grid, or 128 text tokens) against the list of 128-token tiles the schedule gives it.  Eq. 3's
// mask is symmetric, so the list of key tiles a query tile sees is also the list of query tiles that see it as keys.
//   query role  stationary Q_i, dO_i; streamed K_j, V_j.  Per streamed tile, on tcgen05.mma into tensor memory:
//               S = Q K^T and dP = dO V^T.  Sweep 1 over the list: row maximum m, row sum l and
//               delta = sum_j p_ij dP_ij / l (= dO . O) by an online softmax; the three go to global memory for the
//               key role.  Sweep 2: P = exp2(c S - m) / l, dS = P (dP - delta) as bf16 into tensor memory over S,
//               dQ += dS K (dS the tensor-memory operand, K read MN-major from the same shared-memory tile).
//   key role    stationary K_j, V_j; streamed Q_i, dO_i with the statistics of the queries i.  S^T = K Q^T,
//               dP^T = V dO^T; P^T and dS^T as bf16 over them; dV += P^T dO, dK += dS^T Q.
// 256 threads: two per row of the stationary tile, each with half of the columns of a streamed tile (the halves of
// a row merge their softmax statistics once, after sweep 1); one more warp issues every TMA load and every MMA.  The
// streamed tiles go through two stages, so the next pair travels while this one computes; the MMAs and the
// elementwise step of a CTA still take turns: a first tensor-core version of the backward pass, far above the
// CUDA-core one, not yet a tuned one.
// Every wait is bounded: on expiry the CTA raises the plan's status word and leaves.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstring>

#include "clear_internal.hpp"
#include "ptx.cuh"

namespace clear {
namespace {

constexpr int kRowThreads = 256;         // two threads per row of the stationary tile: one per half of the columns
constexpr int kControlWarp = 8;
constexpr int kBwdThreads = 288;         // 8 row warps + 1 control warp (TMA + MMA issue)
constexpr uint32_t kBwdTmemCols = 512;   // T1 | T2 | ACC1 | ACC2, 128 columns each
constexpr uint32_t kBwdSpinLimit = 1u << 22;

struct BwdParams {
    const clear_work_item_t *items;
    const clear_kv_tile_t *tiles;
    const int32_t *half_width;
    int n_half_width;
    int grid_h, grid_w, n_text;
    long long n_tokens;
    float scale, scale_log2;   // scale, scale * log2(e)
    float4 *stats;             // [bh][token]: m (log2 units, scale included), 1 / l, delta, unused
    __nv_bfloat16 *out1, *out2;  // query role: dq, -; key role: dv, dk
    int *status;
};

struct BwdCtrl {
    uint64_t a_full, b_full[2], t_full, p_ready, o_done, x_done;
    uint64_t s_ready;
    float4 part[2][128];   // query role: the two halves' row statistics after sweep 1
    float4 col[2][128];    // key role: statistics of the streamed tile's 128 columns, two stages
    uint32_t tmem_base;
    int abort_flag;
};

__device__ __forceinline__ bool bwd_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, int code)
{
    if (*abort_flag) return false;
    for (uint32_t it = 0; it < kBwdSpinLimit; ++it) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if (it > 64) __nanosleep(it > 4096 ? 256 : 32);
        if ((it & 1023u) == 1023u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicExch(status, code);
    return false;
}
__device__ __forceinline__ void bwd_drain(uint32_t bar, uint32_t parity)
{
    for (uint32_t it = 0; it < kBwdSpinLimit; ++it) {
        if (ptx::mbar_try_wait(bar, parity)) return;
        if (it > 64) __nanosleep(256);
    }
}

template <int D, bool KEY_ROLE>
__global__ void __launch_bounds__(kBwdThreads, 1)
clear_bwd_tc_kernel(const __grid_constant__ CUtensorMap tm_a1_img, const __grid_constant__ CUtensorMap tm_a1_txt,
                    const __grid_constant__ CUtensorMap tm_a2_img, const __grid_constant__ CUtensorMap tm_a2_txt,
                    const __grid_constant__ CUtensorMap tm_b1_img, const __grid_constant__ CUtensorMap tm_b1_lin,
                    const __grid_constant__ CUtensorMap tm_b2_img, const __grid_constant__ CUtensorMap tm_b2_lin,
                    const BwdParams prm)
{
    constexpr int kHalves = D / 64;                 // 64-channel (128-byte) column blocks of a tile
    constexpr uint32_t kHalfBytes = 128 * 128;      // 128 rows x 128 B
    constexpr uint32_t kTileBytes = kHalves * kHalfBytes;
    constexpr uint32_t kIdescT = ptx::idesc_bf16(128, false);   // [128 rows] x [128 columns], both operands K-major
    constexpr uint32_t kIdescAcc = ptx::idesc_bf16(D, true);    // [128 rows] x [D channels], B read MN-major
    constexpr int kSweeps = KEY_ROLE ? 1 : 2;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    // two stationary tiles, then two stages of the two streamed tiles
    const uint32_t sA1 = smem_base, sA2 = sA1 + kTileBytes, sB = sA2 + kTileBytes;
    BwdCtrl *ctrl = reinterpret_cast<BwdCtrl *>(smem_gen + 6 * kTileBytes);
    volatile int *abort_flag = &ctrl->abort_flag;
    const uint32_t b_a = ptx::smem_u32(&ctrl->a_full), b_b0 = ptx::smem_u32(&ctrl->b_full[0]),
                   b_b1 = ptx::smem_u32(&ctrl->b_full[1]), b_t = ptx::smem_u32(&ctrl->t_full), b_p = ptx::smem_u32(&ctrl->p_ready),
                   b_o = ptx::smem_u32(&ctrl->o_done), b_x = ptx::smem_u32(&ctrl->x_done),
                   b_s = ptx::smem_u32(&ctrl->s_ready);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.y;
    const clear_work_item_t item = prm.items[blockIdx.x];
    const clear_kv_tile_t *tiles = prm.tiles + item.tile_begin;
    const int n_tiles = item.tile_count;
    const bool is_text = item.kind == 1;

    // once any CTA of this plan has given up, the rest of the grid leaves at once
    __shared__ int s_skip;
    if (tid == 0) s_skip = *reinterpret_cast<volatile int *>(prm.status);
    __syncthreads();
    if (s_skip != 0) return;

    if (tid == 0) {
        ctrl->abort_flag = 0;
        ptx::mbar_init(b_a, 1);
        ptx::mbar_init(b_b0, 1);
        ptx::mbar_init(b_b1, 1);
        ptx::mbar_init(b_t, 1);
        ptx::mbar_init(b_p, kRowThreads);
        ptx::mbar_init(b_o, 1);
        ptx::mbar_init(b_x, kRowThreads);
        ptx::mbar_init(b_s, 128);
        ptx::fence_mbar_init();
    }
    if (warp == kControlWarp) {
        ptx::tmem_alloc(ptx::smem_u32(&ctrl->tmem_base), kBwdTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = ctrl->tmem_base;
    const uint32_t tmem_T1 = tmem, tmem_T2 = tmem + 128, tmem_A1 = tmem + 256, tmem_A2 = tmem + 384;

    if (warp == kControlWarp) {
        // ================= control warp: one lane issues every TMA load and every MMA ====================
        if (lane == 0) {
            int b_issued = 0, b_seen = 0;
            bool a_seen = false, mma_pending = false;
            auto load_tile = [&](uint32_t dst, uint32_t bar, const CUtensorMap *tm_img, const CUtensorMap *tm_lin, bool linear,
                                 int x, int y) {
#pragma unroll
                for (int h = 0; h < kHalves; ++h) {
                    if (linear)
                        ptx::tma_load_3d(dst + h * kHalfBytes, tm_lin, bar, h * 64, x, bh);
                    else
                        ptx::tma_load_4d(dst + h * kHalfBytes, tm_img, bar, h * 64, x, y, bh);
                }
            };
            // streamed tiles go through two stages: the tiles of iteration it + 1 travel while iteration it computes
            const int n_iters = kSweeps * n_tiles;
            auto load_streamed = [&](int it) {
                const clear_kv_tile_t t = tiles[it % n_tiles];
                const uint32_t bar = (it & 1) ? b_b1 : b_b0, dst = sB + (uint32_t)(it & 1) * 2 * kTileBytes;
                ptx::mbar_expect_tx(bar, 2 * kTileBytes);
                const bool lin = (t.flags & CLEAR_TILE_LINEAR) != 0;
                load_tile(dst, bar, &tm_b1_img, &tm_b1_lin, lin, t.x, t.y);
                load_tile(dst + kTileBytes, bar, &tm_b2_img, &tm_b2_lin, lin, t.x, t.y);
                ++b_issued;
            };
            ptx::mbar_expect_tx(b_a, 2 * kTileBytes);
            load_tile(sA1, b_a, &tm_a1_img, &tm_a1_txt, is_text, item.qx, item.qy);
            load_tile(sA2, b_a, &tm_a2_img, &tm_a2_txt, is_text, item.qx, item.qy);
            load_streamed(0);
            if (n_iters > 1) load_streamed(1);
            a_seen = bwd_wait(b_a, 0, abort_flag, prm.status, 1);

            // T1 = A1 B1^T, T2 = A2 B2^T of iteration it: D/16 MMAs of 16 channels each
            auto issue_t = [&](int it) -> bool {
                const uint32_t ph = (uint32_t)(it & 1);
                const uint32_t sB1 = sB + ph * 2 * kTileBytes, sB2 = sB1 + kTileBytes;
                if (!bwd_wait(ph ? b_b1 : b_b0, (uint32_t)((it >> 1) & 1), abort_flag, prm.status, 2)) return false;
                ++b_seen;
                ptx::tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
                    ptx::mma_ss(tmem_T1, ptx::smem_desc_sw128(sA1 + off, 16, 1024), ptx::smem_desc_sw128(sB1 + off, 16, 1024),
                                kIdescT, kk > 0);
                }
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
                    ptx::mma_ss(tmem_T2, ptx::smem_desc_sw128(sA2 + off, 16, 1024), ptx::smem_desc_sw128(sB2 + off, 16, 1024),
                                kIdescT, kk > 0);
                }
                ptx::tc_commit(b_t);
                mma_pending = true;
                return true;
            };

            int n_grad = 0;
            bool ok = a_seen && issue_t(0);
            for (int it = 0; it < n_iters && ok; ++it) {
                const bool grad = KEY_ROLE || it >= n_tiles;
                const uint32_t ph = (uint32_t)(it & 1);
                const uint32_t sB1 = sB + ph * 2 * kTileBytes, sB2 = sB1 + kTileBytes;
                // the rows have read T1, T2 (and, in a gradient sweep, put P / dS over them)
                if (!(ok = bwd_wait(b_p, ph, abort_flag, prm.status, 3))) break;
                mma_pending = false;
                if (grad) {
                    ptx::tc_fence_after();
                    // ---- the accumulators: 8 MMAs over 16 streamed tokens each, B read MN-major -------------
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint32_t acc = (n_grad > 0 || kk > 0) ? 1u : 0u;
                        if (KEY_ROLE) {
                            ptx::mma_ts(tmem_A1, tmem_T1 + (kk >> 2) * 64 + (kk & 3) * 8, ptx::smem_desc_sw128(sB2 + kk * 2048, kHalfBytes, 1024),
                                        kIdescAcc, acc);   // dV += P^T dO
                            ptx::mma_ts(tmem_A2, tmem_T2 + (kk >> 2) * 64 + (kk & 3) * 8, ptx::smem_desc_sw128(sB1 + kk * 2048, kHalfBytes, 1024),
                                        kIdescAcc, acc);   // dK += dS^T Q
                        } else {
                            ptx::mma_ts(tmem_A1, tmem_T1 + (kk >> 2) * 64 + (kk & 3) * 8, ptx::smem_desc_sw128(sB1 + kk * 2048, kHalfBytes, 1024),
                                        kIdescAcc, acc);   // dQ += dS K
                        }
                    }
                    ptx::tc_commit(b_o);
                    mma_pending = true;
                }
                // the next tile's T1, T2 go behind these MMAs on the same pipe: they overwrite P / dS only after the
                // accumulations have read them, and run while this warp waits below
                if (it + 1 < n_iters && !(ok = issue_t(it + 1))) break;
                if (grad) {
                    if (!(ok = bwd_wait(b_o, (uint32_t)(n_grad & 1), abort_flag, prm.status, 4))) break;
                    if (it + 1 >= n_iters) mma_pending = false;
                    ++n_grad;
                }
                // this iteration's stage is free (its MMAs have retired): the tiles of iteration it + 2 may land in it
                if (it + 2 < n_iters) load_streamed(it + 2);
            }
            if (*abort_flag) {
                // leave nothing in flight: copies that were issued must land, MMAs must retire
                if (!a_seen) bwd_drain(b_a, 0);
                // at most two loads are in flight: iterations b_seen and b_seen + 1
                for (int it = b_seen; it < b_issued; ++it) bwd_drain((it & 1) ? b_b1 : b_b0, (uint32_t)((it >> 1) & 1));
                if (mma_pending) __nanosleep(100000);
            }
        }
        __syncwarp();
    } else {
        // ================= row warps: thread (g, r) owns row r of the stationary tile and the columns
        // [64 g, 64 g + 64) of every streamed tile (two warps per tensor-memory lane quadrant) =================
        const int g = warp >> 2;                 // column half
        const int r = (warp & 3) * 32 + lane;    // row of the tile
        const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t col0 = 64u * (uint32_t)g;  // first fp32 column of this thread's half; its bf16 results go there too
        const float c = prm.scale_log2;
        int q_y = 0, q_x = 0;
        bool row_valid;
        long long row_token;
        if (is_text) {
            row_valid = r < item.n_rows;
            row_token = (long long)item.qx + r;
        } else {
            q_y = item.qy + (r >> 4);
            q_x = item.qx + (r & 15);
            row_valid = q_y < prm.grid_h && q_x < prm.grid_w;
            row_token = (long long)prm.n_text + (long long)q_y * prm.grid_w + q_x;
        }
        float4 *stats = prm.stats + (long long)bh * prm.n_tokens;
        // query role: statistics of the row; in sweep 1 running values over THIS thread's columns only (m in log2
        // units, scale included), merged with the other half's at the end of the sweep
        float m_row = -INFINITY, l_row = 0.f, d_row = 0.f, il_row = 0.f;
        bool alive = true;
        int iter = 0, n_grad = 0;

        for (int sweep = 0; sweep < kSweeps && alive; ++sweep) {
            const bool grad = KEY_ROLE || sweep == 1;
            for (int i = 0; i < n_tiles; ++i, ++iter) {
                const uint32_t ph = (uint32_t)(iter & 1);
                const clear_kv_tile_t t = tiles[i];
                // ---- mask bits of this row for its 64 columns (bit j of word w = column 64 g + 32 w + j allowed; the
                // mask is symmetric, so the row's token plays the query whichever role the kernel runs in) ----------
                uint32_t mw[2] = {0xffffffffu, 0xffffffffu};
                if (t.flags & CLEAR_TILE_MASKED) {
                    if (t.flags & CLEAR_TILE_LINEAR) {
#pragma unroll
                        for (int w = 0; w < 2; ++w) {
                            const int n = min(max(t.n_valid - 64 * g - 32 * w, 0), 32);
                            mw[w] = n == 32 ? 0xffffffffu : ((1u << n) - 1u);
                        }
                    } else {
                        mw[0] = mw[1] = 0u;
#pragma unroll
                        for (int rr = 0; rr < 4; ++rr) {
                            const int ky = t.y + 4 * g + rr;
                            const int ady = abs(ky - q_y);
                            uint32_t bits = 0u;
                            if (row_valid && ky >= 0 && ky < prm.grid_h && ady < prm.n_half_width) {
                                const int hw = __ldg(prm.half_width + ady);
                                const int lo = max(max(q_x - hw, 0), t.x);
                                const int hi = min(min(q_x + hw, prm.grid_w - 1), t.x + 15);
                                if (lo <= hi) bits = ((1u << (hi - lo + 1)) - 1u) << (lo - t.x);
                            }
                            mw[rr >> 1] |= bits << (16 * (rr & 1));
                        }
                    }
                }

                // key role: the statistics of the tile's 128 columns go to shared memory once, fetched by the first
                // half's threads while the MMAs run (a column that does not exist is masked; its address stays inside
                // the buffer, which is padded by one tile)
                if (KEY_ROLE && g == 0) {
                    const float4 *src;
                    if (t.flags & CLEAR_TILE_LINEAR)
                        src = stats + t.x + r;
                    else
                        src = stats + prm.n_text + (long long)min(t.y + (r >> 4), prm.grid_h - 1) * prm.grid_w + t.x + (r & 15);
                    ctrl->col[ph][r] = __ldg(src);
                    ptx::mbar_arrive(b_s);
                }

                // warp-uniform outcome: the tcgen05.ld / st below need the whole warp
                if (!__all_sync(0xffffffffu, bwd_wait(b_t, ph, abort_flag, prm.status, 5))) { alive = false; break; }
                if (KEY_ROLE && !__all_sync(0xffffffffu, bwd_wait(b_s, ph, abort_flag, prm.status, 8))) { alive = false; break; }
                ptx::tc_fence_after();

                if (!grad) {
                    // ---- sweep 1 of the query role: online softmax statistics and delta over this half ----------
                    float mx = -INFINITY;
#pragma unroll
                    for (int w = 0; w < 2; ++w) {
                        uint32_t s[32];
                        ptx::tmem_ld32(tmem_T1 + lane_off + col0 + 32 * w, s);
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if ((mw[w] >> j) & 1u) mx = fmaxf(mx, __uint_as_float(s[j]));
                    }
                    const float m_new = fmaxf(m_row, mx * c);
                    const float alpha = (m_new == -INFINITY) ? 1.f : ptx::ex2(m_row - m_new);  // m_row = -inf: 0
                    l_row *= alpha;
                    d_row *= alpha;
                    const float mc = (m_new == -INFINITY) ? 0.f : m_new;
#pragma unroll
                    for (int w = 0; w < 2; ++w) {
                        uint32_t s[32], gg[32];
                        ptx::tmem_ld32(tmem_T1 + lane_off + col0 + 32 * w, s);
                        ptx::tmem_ld32(tmem_T2 + lane_off + col0 + 32 * w, gg);
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float p = ((mw[w] >> j) & 1u) ? ptx::ex2(fmaf(__uint_as_float(s[j]), c, -mc)) : 0.f;
                            l_row += p;
                            d_row = fmaf(p, __uint_as_float(gg[j]), d_row);
                        }
                    }
                    m_row = m_new;
                    ptx::tc_fence_before();
                    ptx::mbar_arrive(b_p);
                    continue;
                }

                // ---- gradient sweep: P = exp2(c T1 - m) / l, dS = P (T2 - delta), bf16 over T1 / T2 -------------
#pragma unroll
                for (int w = 0; w < 2; ++w) {
                    uint32_t s[32], gg[32], pk[16], dk[16];
                    ptx::tmem_ld32(tmem_T1 + lane_off + col0 + 32 * w, s);
                    ptx::tmem_ld32(tmem_T2 + lane_off + col0 + 32 * w, gg);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        float p[2], ds[2];
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            float m_c, il_c, d_c;
                            if (KEY_ROLE) {
                                const float4 st = ctrl->col[ph][64 * g + 32 * w + j + u];
                                m_c = st.x;
                                il_c = st.y;
                                d_c = st.z;
                            } else {
                                m_c = m_row;
                                il_c = il_row;
                                d_c = d_row;
                            }
                            const bool on = ((mw[w] >> (j + u)) & 1u) != 0u;
                            p[u] = on ? ptx::ex2(fmaf(__uint_as_float(s[j + u]), c, -m_c)) * il_c : 0.f;
                            ds[u] = p[u] * (__uint_as_float(gg[j + u]) - d_c);
                        }
                        pk[j >> 1] = ptx::pack_bf16(p[0], p[1]);
                        dk[j >> 1] = ptx::pack_bf16(ds[0], ds[1]);
                    }
                    // the half's 32 bf16 columns sit at the start of its own fp32 columns, all of which this thread
                    // has in registers before it writes (chunk 0 covers them)
                    if (KEY_ROLE) {
                        ptx::tmem_st16(tmem_T1 + lane_off + col0 + 16 * w, pk);
                        ptx::tmem_st16(tmem_T2 + lane_off + col0 + 16 * w, dk);
                    } else {
                        ptx::tmem_st16(tmem_T1 + lane_off + col0 + 16 * w, dk);
                    }
                }
                ptx::tmem_wait_st();
                ptx::tc_fence_before();
                ptx::mbar_arrive(b_p);
                ++n_grad;
            }
            if (!KEY_ROLE && sweep == 0 && alive) {
                // the two halves of a row merge their statistics (a split softmax); kept for sweep 2, and left in
                // global memory for the key role
                ctrl->part[g][r] = make_float4(m_row, l_row, d_row, 0.f);
                ptx::mbar_arrive(b_x);
                if (!__all_sync(0xffffffffu, bwd_wait(b_x, 0, abort_flag, prm.status, 7))) { alive = false; break; }
                const float4 o = ctrl->part[g ^ 1][r];
                const float m = fmaxf(m_row, o.x);
                const float a0 = (m_row == -INFINITY) ? 0.f : ptx::ex2(m_row - m), a1 = (o.x == -INFINITY) ? 0.f : ptx::ex2(o.x - m);
                const float l = l_row * a0 + o.y * a1;
                il_row = l > 0.f ? 1.f / l : 0.f;
                d_row = (d_row * a0 + o.z * a1) * il_row;
                m_row = (m == -INFINITY) ? 0.f : m;  // a row without any key: P = 0 through il = 0
                if (row_valid && g == 0) stats[row_token] = make_float4(m_row, il_row, d_row, 0.f);
            }
        }

        // ---- epilogue: wait for the last accumulation, then store the rows (each half its share of the channels) ----
        if (alive && n_grad > 0)
            alive = __all_sync(0xffffffffu, bwd_wait(b_o, (uint32_t)((n_grad - 1) & 1), abort_flag, prm.status, 6));
        if (alive) {
            ptx::tc_fence_after();
            auto store_rows = [&](uint32_t tmem_acc, __nv_bfloat16 *dst_base, float factor) {
                __nv_bfloat16 *dst = dst_base + ((long long)bh * prm.n_tokens + row_token) * D;
#pragma unroll
                for (int ww = 0; ww < D / 64; ++ww) {
                    const int w = g * (D / 64) + ww;  // 32-channel chunk
                    uint32_t o[32];
                    ptx::tmem_ld32(tmem_acc + lane_off + 32 * w, o);
                    ptx::tmem_wait_ld();
                    if (row_valid) {
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) {
                            uint4 val;
                            val.x = ptx::pack_bf16(__uint_as_float(o[8 * cc + 0]) * factor, __uint_as_float(o[8 * cc + 1]) * factor);
                            val.y = ptx::pack_bf16(__uint_as_float(o[8 * cc + 2]) * factor, __uint_as_float(o[8 * cc + 3]) * factor);
                            val.z = ptx::pack_bf16(__uint_as_float(o[8 * cc + 4]) * factor, __uint_as_float(o[8 * cc + 5]) * factor);
                            val.w = ptx::pack_bf16(__uint_as_float(o[8 * cc + 6]) * factor, __uint_as_float(o[8 * cc + 7]) * factor);
                            *reinterpret_cast<uint4 *>(dst + 32 * w + 8 * cc) = val;
                        }
                    }
                }
            };
            if (KEY_ROLE) {
                store_rows(tmem_A1, prm.out1, 1.f);         // dV
                store_rows(tmem_A2, prm.out2, prm.scale);   // dK
            } else {
                store_rows(tmem_A1, prm.out1, prm.scale);   // dQ
            }
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == kControlWarp) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, kBwdTmemCols);
    }
}

}  // namespace

int launch_bwd_tc(const clear_plan &p, const void *q, const void *k, const void *v, const void *d_out, void *dq, void *dk,
                  void *dv, float scale, cudaStream_t stream)
{
    const Shape &s = p.shape;
    if (!(scale > 0.f)) return CLEAR_ERR_UNSUPPORTED;
    if (s.head_dim != 64 && s.head_dim != 128) return CLEAR_ERR_UNSUPPORTED;
    const uint64_t d = (uint64_t)s.head_dim, gw = (uint64_t)s.grid_w, gh = (uint64_t)s.grid_h, T = (uint64_t)s.n_text;
    const uint64_t N = T + gw * gh, BH = (uint64_t)s.B * s.H;
    if (!p.d_bwd_stats) {
        // one tile of padding: the statistics of columns past the end are read (and masked), never used
        cudaError_t e = cudaMalloc((void **)&p.d_bwd_stats, ((size_t)BH * N + kTileTokens) * sizeof(float4));
        if (e == cudaSuccess) e = cudaMemsetAsync(p.d_bwd_stats, 0, ((size_t)BH * N + kTileTokens) * sizeof(float4), stream);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            return e == cudaErrorMemoryAllocation ? CLEAR_ERR_NO_MEMORY : CLEAR_ERR_CUDA;
        }
    }
    // Per tensor three views: the image part as [BH][grid_h][grid_w][d] (8 x 16 patches), the token sequence
    // [BH][N][d] (128 consecutive tokens), and its text prefix [BH][n_text][d] (rows past the text read as zero).
    const uint64_t row_b = d * 2;
    const uint64_t dims4[4] = {d, gw, gh, BH};
    const uint64_t str4[3] = {row_b, gw * row_b, N * row_b};
    const uint32_t box4[4] = {64, (uint32_t)kTileW, (uint32_t)kTileH, 1};
    const uint64_t dims3[3] = {d, N, BH};
    const uint64_t dims3t[3] = {d, T > 0 ? T : 1, BH};
    const uint64_t str3[2] = {row_b, N * row_b};
    const uint32_t box3[3] = {64, (uint32_t)kTileTokens, 1};
    struct Views {
        CUtensorMap img, lin, txt;
    };
    auto make = [&](const void *base, Views &out) {
        const char *img = static_cast<const char *>(base) + T * row_b;
        return encode_bf16_map(&out.img, img, 4, dims4, str4, box4) && encode_bf16_map(&out.lin, base, 3, dims3, str3, box3) &&
               encode_bf16_map(&out.txt, base, 3, dims3t, str3, box3);
    };
    Views vq, vk, vv, vg;
    if (!make(q, vq) || !make(k, vk) || !make(v, vv) || !make(d_out, vg)) return CLEAR_ERR_CUDA;

    BwdParams prm{};
    prm.items = p.d_items;
    prm.tiles = p.d_tiles;
    prm.half_width = p.d_half_width;
    prm.n_half_width = (int)p.sch.half_width.size();
    prm.grid_h = s.grid_h;
    prm.grid_w = s.grid_w;
    prm.n_text = s.n_text;
    prm.n_tokens = (long long)N;
    prm.scale = scale;
    prm.scale_log2 = scale * 1.4426950408889634f;
    prm.stats = reinterpret_cast<float4 *>(p.d_bwd_stats);
    prm.status = p.d_status;

    const dim3 grid((unsigned)p.sch.items.size(), (unsigned)BH), block(kBwdThreads);
    auto run = [&](auto kernel_q, auto kernel_k, size_t smem) -> int {
        CLEAR_CUDA_TRY(cudaFuncSetAttribute(kernel_q, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        CLEAR_CUDA_TRY(cudaFuncSetAttribute(kernel_k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        BwdParams pq = prm;
        pq.out1 = static_cast<__nv_bfloat16 *>(dq);
        kernel_q<<<grid, block, smem, stream>>>(vq.img, vq.txt, vg.img, vg.txt, vk.img, vk.lin, vv.img, vv.lin, pq);
        CLEAR_CUDA_TRY(cudaGetLastError());
        BwdParams pk = prm;
        pk.out1 = static_cast<__nv_bfloat16 *>(dv);
        pk.out2 = static_cast<__nv_bfloat16 *>(dk);
        kernel_k<<<grid, block, smem, stream>>>(vk.img, vk.txt, vv.img, vv.txt, vq.img, vq.lin, vg.img, vg.lin, pk);
        CLEAR_CUDA_TRY(cudaGetLastError());
        return CLEAR_OK;
    };
    if (s.head_dim == 128)
        return run(clear_bwd_tc_kernel<128, false>, clear_bwd_tc_kernel<128, true>, 6 * 32768 + 1024 + sizeof(BwdCtrl));
    return run(clear_bwd_tc_kernel<64, false>, clear_bwd_tc_kernel<64, true>, 6 * 16384 + 1024 + sizeof(BwdCtrl));
}

}  // namespace clear
