// CLEAR attention forward on the sm_100a tensor cores: block-sparse flash-style kernel.
//
// One CTA runs one work item of the plan: 128 queries (an 8 x 16 patch of the latent grid, or 128
// consecutive text tokens) against a list of 128-key tiles (2-D key patches that meet the query
// patch's radius-r dilation, and linear tiles of the token sequence).  Per key tile:
//   TMA stages K and V (bf16, 128-byte swizzle) in shared memory;
//   S = Q K^T on tcgen05.mma into tensor memory (fp32);
//   128 softmax threads (one query row each) read S with tcgen05.ld, apply the Eq. 3 mask where
//   the plan says the tile needs it, keep the online-softmax state of Eq. 1, and put P (bf16)
//   back into tensor memory over S;
//   O += P V on tcgen05.mma with P as the tensor-memory operand and V as an MN-major shared one.
// The CTA keeps one K and one V buffer: K(i+1) is fetched while the softmax of tile i runs and
// V(i+1) while QK(i+1) and its softmax run; two CTAs per SM (256 tensor-memory columns each)
// overlap one CTA's softmax with the other's MMAs.
// Text-query items whose key range was split write un-normalised partial results; a small kernel
// merges them.  Every wait is bounded: on expiry the CTA raises the plan's status word and leaves.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstring>

#include "clear_internal.hpp"
#include "ptx.cuh"

namespace clear {
namespace {

constexpr int kSoftmaxThreads = 128;
constexpr int kThreads = 160;           // 4 softmax warps + 1 control warp (TMA + MMA issue)
constexpr uint32_t kTmemCols = 256;     // S/P: columns [0, 128), O: columns [128, 128 + D)
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr float kRescaleThreshold = 8.f;  // log2 units: O is rescaled only when the row max grows by more

struct TcParams {
    const clear_work_item_t *items;
    const clear_kv_tile_t *tiles;
    const int32_t *half_width;
    int n_half_width;
    int grid_h, grid_w, n_text;
    float scale_log2;  // scale * log2(e)
    float *partial_o;
    float *partial_ml;
    int n_partial_slots;
    int *status;
};

struct Ctrl {
    uint64_t q_full, k_full, v_full, s_full, p_ready, o_done, staged;
    uint32_t tmem_base;
    int abort_flag;
};

// Bounded wait on an mbarrier phase.  Returns false once the CTA has given up.
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, int code)
{
    if (*abort_flag) return false;
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if (it > 64) __nanosleep(it > 4096 ? 256 : 32);
        if ((it & 1023u) == 1023u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicExch(status, code);
    return false;
}
// Drain: wait for a phase regardless of the abort flag (used before leaving with copies in flight).
__device__ __forceinline__ void drain_bar(uint32_t bar, uint32_t parity)
{
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (ptx::mbar_try_wait(bar, parity)) return;
        if (it > 64) __nanosleep(256);
    }
}

template <int D>
__global__ void __launch_bounds__(kThreads, 2)
clear_tc_kernel(const __grid_constant__ CUtensorMap tm_q_img, const __grid_constant__ CUtensorMap tm_k_img,
                const __grid_constant__ CUtensorMap tm_v_img, const __grid_constant__ CUtensorMap tm_o_img,
                const __grid_constant__ CUtensorMap tm_q_txt, const __grid_constant__ CUtensorMap tm_k_lin,
                const __grid_constant__ CUtensorMap tm_v_lin, const __grid_constant__ CUtensorMap tm_o_txt,
                const TcParams prm)
{
    constexpr int kHalves = D / 64;                 // 64-channel (128-byte) column blocks of a tile
    constexpr uint32_t kHalfBytes = 128 * 128;      // 128 rows x 128 B
    constexpr uint32_t kTileBytes = kHalves * kHalfBytes;
    constexpr uint32_t kIdescQK = ptx::idesc_bf16(128, false);
    constexpr uint32_t kIdescPV = ptx::idesc_bf16(D, true);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const uint32_t sQ = smem_base, sK = sQ + kTileBytes, sV = sK + kTileBytes;
    constexpr uint32_t kCtrlOff = 3 * kTileBytes;
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(smem_gen + kCtrlOff);
    volatile int *abort_flag = &ctrl->abort_flag;

    const uint32_t b_q = ptx::smem_u32(&ctrl->q_full), b_k = ptx::smem_u32(&ctrl->k_full),
                   b_v = ptx::smem_u32(&ctrl->v_full), b_s = ptx::smem_u32(&ctrl->s_full),
                   b_p = ptx::smem_u32(&ctrl->p_ready), b_o = ptx::smem_u32(&ctrl->o_done),
                   b_st = ptx::smem_u32(&ctrl->staged);

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
        ptx::mbar_init(b_q, 1);
        ptx::mbar_init(b_k, 1);
        ptx::mbar_init(b_v, 1);
        ptx::mbar_init(b_s, 1);
        ptx::mbar_init(b_p, kSoftmaxThreads);
        ptx::mbar_init(b_o, 1);
        ptx::mbar_init(b_st, kSoftmaxThreads);
        ptx::fence_mbar_init();
    }
    if (warp == 4) {
        ptx::tmem_alloc(ptx::smem_u32(&ctrl->tmem_base), kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = ctrl->tmem_base;
    const uint32_t tmem_S = tmem, tmem_O = tmem + 128;

    if (warp == 4) {
        // ================= control warp: one elected lane issues every TMA load and every MMA =========
        if (lane == 0) {
            int k_issued = 0, v_issued = 0, k_seen = 0, v_seen = 0;  // loads issued / waited for
            bool q_seen = false;
            auto load_kv = [&](uint32_t dst, uint32_t bar, const CUtensorMap *tm_img, const CUtensorMap *tm_lin,
                               const clear_kv_tile_t &t) {
                ptx::mbar_expect_tx(bar, kTileBytes);
#pragma unroll
                for (int h = 0; h < kHalves; ++h) {
                    if (t.flags & CLEAR_TILE_LINEAR)
                        ptx::tma_load_3d(dst + h * kHalfBytes, tm_lin, bar, h * 64, t.x, bh);
                    else
                        ptx::tma_load_4d(dst + h * kHalfBytes, tm_img, bar, h * 64, t.x, t.y, bh);
                }
            };
            ptx::mbar_expect_tx(b_q, kTileBytes);
#pragma unroll
            for (int h = 0; h < kHalves; ++h) {
                if (is_text)
                    ptx::tma_load_3d(sQ + h * kHalfBytes, &tm_q_txt, b_q, h * 64, item.qx, bh);
                else
                    ptx::tma_load_4d(sQ + h * kHalfBytes, &tm_q_img, b_q, h * 64, item.qx, item.qy, bh);
            }
            clear_kv_tile_t t_next = tiles[0];
            load_kv(sK, b_k, &tm_k_img, &tm_k_lin, t_next);
            ++k_issued;
            load_kv(sV, b_v, &tm_v_img, &tm_v_lin, t_next);
            ++v_issued;
            q_seen = wait_bar(b_q, 0, abort_flag, prm.status, 1);

            bool mma_pending = false;
            for (int i = 0; i < n_tiles; ++i) {
                const uint32_t ph = (uint32_t)(i & 1);
                if (!wait_bar(b_k, ph, abort_flag, prm.status, 2)) break;
                ++k_seen;
                ptx::tc_fence_after();
                // ---- S = Q K^T : D/16 MMAs of K = 16 -------------------------------------------------
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
                    ptx::mma_ss(tmem_S, ptx::smem_desc_sw128(sQ + off, 16, 1024),
                                ptx::smem_desc_sw128(sK + off, 16, 1024), kIdescQK, kk > 0);
                }
                ptx::tc_commit(b_s);
                mma_pending = true;
                if (i + 1 < n_tiles) t_next = tiles[i + 1];
                // K buffer is free once QK(i) has run: fetch K(i+1) under the softmax of tile i
                if (!wait_bar(b_s, ph, abort_flag, prm.status, 3)) break;
                mma_pending = false;
                if (i + 1 < n_tiles) {
                    load_kv(sK, b_k, &tm_k_img, &tm_k_lin, t_next);
                    ++k_issued;
                }
                if (!wait_bar(b_v, ph, abort_flag, prm.status, 4)) break;
                ++v_seen;
                if (!wait_bar(b_p, ph, abort_flag, prm.status, 5)) break;
                ptx::tc_fence_after();
                // ---- O += P V : 8 MMAs over 16 keys each --------------------------------------------
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint64_t bdesc = ptx::smem_desc_sw128(sV + kk * 2048, kHalfBytes, 1024);
                    const uint32_t acc = (i > 0 || kk > 0) ? 1u : 0u;
                    ptx::mma_ts(tmem_O, tmem_S + kk * 8, bdesc, kIdescPV, acc);
                }
                ptx::tc_commit(b_o);
                mma_pending = true;
                // V buffer and the S/P columns are free once PV(i) has run
                if (!wait_bar(b_o, ph, abort_flag, prm.status, 6)) break;
                mma_pending = false;
                if (i + 1 < n_tiles) {
                    load_kv(sV, b_v, &tm_v_img, &tm_v_lin, t_next);
                    ++v_issued;
                }
            }
            if (*abort_flag) {
                // leave nothing in flight: copies that were issued must land, MMAs must retire
                if (!q_seen) drain_bar(b_q, 0);
                if (k_issued > k_seen) drain_bar(b_k, (uint32_t)(k_seen & 1));
                if (v_issued > v_seen) drain_bar(b_v, (uint32_t)(v_seen & 1));
                if (mma_pending) __nanosleep(100000);
            }
        }
        __syncwarp();
    } else {
        // ================= softmax warps: thread r owns query row r of the tile =========================
        const int r = tid;
        const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
        const float c = prm.scale_log2;
        int q_y = 0, q_x = 0;
        bool q_valid;
        if (is_text) {
            q_valid = r < item.n_rows;
        } else {
            q_y = item.qy + (r >> 4);
            q_x = item.qx + (r & 15);
            q_valid = q_y < prm.grid_h && q_x < prm.grid_w;
        }
        float m_used = -INFINITY, l = 0.f;
        bool alive = true;

        for (int i = 0; i < n_tiles; ++i) {
            const uint32_t ph = (uint32_t)(i & 1);
            const clear_kv_tile_t t = tiles[i];
            // ---- mask bits of this row for the tile (bit j = key j allowed) ---------------------------
            uint32_t mw[4] = {0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu};
            if (t.flags & CLEAR_TILE_MASKED) {
                if (t.flags & CLEAR_TILE_LINEAR) {
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        const int n = min(max(t.n_valid - 32 * w, 0), 32);
                        mw[w] = n == 32 ? 0xffffffffu : ((1u << n) - 1u);
                    }
                } else {
#pragma unroll
                    for (int w = 0; w < 4; ++w) mw[w] = 0u;
#pragma unroll
                    for (int rr = 0; rr < 8; ++rr) {
                        const int ky = t.y + rr;
                        const int ady = abs(ky - q_y);
                        uint32_t bits = 0u;
                        if (q_valid && ky >= 0 && ky < prm.grid_h && ady < prm.n_half_width) {
                            const int hw = __ldg(prm.half_width + ady);
                            const int lo = max(max(q_x - hw, 0), t.x);
                            const int hi = min(min(q_x + hw, prm.grid_w - 1), t.x + 15);
                            if (lo <= hi) bits = ((1u << (hi - lo + 1)) - 1u) << (lo - t.x);
                        }
                        mw[rr >> 1] |= bits << (16 * (rr & 1));
                    }
                }
            }

            // warp-uniform outcome: the tcgen05.ld / st below need the whole warp
            if (!__all_sync(0xffffffffu, wait_bar(b_s, ph, abort_flag, prm.status, 7))) { alive = false; break; }
            ptx::tc_fence_after();
            uint32_t s[4][32];
#pragma unroll
            for (int w = 0; w < 4; ++w) ptx::tmem_ld32(tmem_S + lane_off + 32 * w, s[w]);
            ptx::tmem_wait_ld();

            float mx = -INFINITY;
            if (t.flags & CLEAR_TILE_MASKED) {
#pragma unroll
                for (int w = 0; w < 4; ++w)
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float val = ((mw[w] >> j) & 1u) ? __uint_as_float(s[w][j]) : -INFINITY;
                        s[w][j] = __float_as_uint(val);
                        mx = fmaxf(mx, val);
                    }
            } else {
#pragma unroll
                for (int w = 0; w < 4; ++w)
#pragma unroll
                    for (int j = 0; j < 32; ++j) mx = fmaxf(mx, __uint_as_float(s[w][j]));
            }

            // ---- running maximum; O is rescaled only when it grew by more than the threshold ---------
            const float m_new = fmaxf(m_used, mx);
            if (i == 0) {
                m_used = m_new;
            } else {
                const bool need = (m_new - m_used) * c > kRescaleThreshold;  // false for NaN (-inf minus -inf)
                if (__any_sync(0xffffffffu, need)) {
                    float alpha = 1.f;
                    if (need) {
                        alpha = ptx::ex2((m_used - m_new) * c);
                        m_used = m_new;
                        l *= alpha;
                    }
#pragma unroll
                    for (int w = 0; w < D / 32; ++w) {
                        uint32_t o[32];
                        ptx::tmem_ld32(tmem_O + lane_off + 32 * w, o);
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
                        ptx::tmem_st32(tmem_O + lane_off + 32 * w, o);
                    }
                }
            }
            const float mc = (m_used == -INFINITY) ? 0.f : m_used * c;

            // ---- P = exp2(S * c - m * c), row sum, bf16 pairs -----------------------------------------
            uint32_t pk[2][32];
#pragma unroll
            for (int w = 0; w < 4; ++w)
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    const float p0 = ptx::ex2(fmaf(__uint_as_float(s[w][j]), c, -mc));
                    const float p1 = ptx::ex2(fmaf(__uint_as_float(s[w][j + 1]), c, -mc));
                    l += p0 + p1;
                    pk[w >> 1][(w & 1) * 16 + (j >> 1)] = ptx::pack_bf16(p0, p1);
                }
            ptx::tmem_st32(tmem_S + lane_off, pk[0]);
            ptx::tmem_st32(tmem_S + lane_off + 32, pk[1]);
            ptx::tmem_wait_st();
            ptx::tc_fence_before();
            ptx::mbar_arrive(b_p);
        }

        // ---- epilogue: wait for the last PV, then normalise and store ---------------------------------
        if (alive) alive = __all_sync(0xffffffffu, wait_bar(b_o, (uint32_t)((n_tiles - 1) & 1), abort_flag, prm.status, 8));
        if (alive) {
            ptx::tc_fence_after();
            if (item.partial_slot >= 0) {
                // split text-query tile: un-normalised fp32 row, its maximum (log2 units) and its sum
                const int64_t row = ((int64_t)bh * prm.n_partial_slots + item.partial_slot) * 128 + r;
                float *dst = prm.partial_o + row * D;
#pragma unroll
                for (int w = 0; w < D / 32; ++w) {
                    uint32_t o[32];
                    ptx::tmem_ld32(tmem_O + lane_off + 32 * w, o);
                    ptx::tmem_wait_ld();
                    if (q_valid) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            *reinterpret_cast<uint4 *>(dst + 32 * w + j) = make_uint4(o[j], o[j + 1], o[j + 2], o[j + 3]);
                    }
                }
                if (q_valid) {
                    prm.partial_ml[row * 2] = m_used * c;
                    prm.partial_ml[row * 2 + 1] = l;
                }
            } else {
                const float inv = l > 0.f ? 1.f / l : 0.f;
                uint8_t *o_gen = smem_gen;  // the Q buffer: every QK^T has retired
#pragma unroll
                for (int w = 0; w < D / 32; ++w) {
                    uint32_t o[32];
                    ptx::tmem_ld32(tmem_O + lane_off + 32 * w, o);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        uint4 val;
                        val.x = ptx::pack_bf16(__uint_as_float(o[8 * cc + 0]) * inv, __uint_as_float(o[8 * cc + 1]) * inv);
                        val.y = ptx::pack_bf16(__uint_as_float(o[8 * cc + 2]) * inv, __uint_as_float(o[8 * cc + 3]) * inv);
                        val.z = ptx::pack_bf16(__uint_as_float(o[8 * cc + 4]) * inv, __uint_as_float(o[8 * cc + 5]) * inv);
                        val.w = ptx::pack_bf16(__uint_as_float(o[8 * cc + 6]) * inv, __uint_as_float(o[8 * cc + 7]) * inv);
                        const int ch = (w & 1) * 4 + cc;  // 16-byte chunk within the 128-byte row of half w / 2
                        *reinterpret_cast<uint4 *>(o_gen + (w >> 1) * kHalfBytes + r * 128 + ((ch ^ (r & 7)) << 4)) = val;
                    }
                }
                ptx::fence_proxy_async_smem();
                ptx::mbar_arrive(b_st);
                if (tid == 0 && wait_bar(b_st, 0, abort_flag, prm.status, 9)) {
#pragma unroll
                    for (int h = 0; h < kHalves; ++h) {
                        if (is_text)
                            ptx::tma_store_3d(&tm_o_txt, sQ + h * kHalfBytes, h * 64, item.qx, bh);
                        else
                            ptx::tma_store_4d(&tm_o_img, sQ + h * kHalfBytes, h * 64, item.qx, item.qy, bh);
                    }
                    ptx::bulk_commit_group();
                    ptx::bulk_wait_group0();
                }
            }
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, kTmemCols);
    }
}

// Merge the split-KV partial results of the text-query rows: out = sum_s w_s O_s / sum_s w_s l_s,
// w_s = 2^(m_s - max_s m_s).  One block per (text row, bh), one thread per channel.
template <int D>
__global__ void __launch_bounds__(D)
clear_tc_combine_kernel(const float *__restrict__ partial_o, const float *__restrict__ partial_ml,
                        __nv_bfloat16 *__restrict__ out, int n_text, int64_t n_tokens, int n_splits, int n_slots)
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
    out[((int64_t)bh * n_tokens + row) * D + e] = __float2bfloat16_rn(den > 0.f ? num / den : 0.f);
}

// ---- host side: tensor maps and launch ---------------------------------------------------------
int build_maps(const clear_plan &p, const void *q, const void *k, const void *v, void *out)
{
    const Shape &s = p.shape;
    const uint64_t d = (uint64_t)s.head_dim, gw = (uint64_t)s.grid_w, gh = (uint64_t)s.grid_h, T = (uint64_t)s.n_text;
    const uint64_t N = T + gw * gh, BH = (uint64_t)s.B * s.H;
    const uint64_t row_b = d * 2;
    CUtensorMap *tm = reinterpret_cast<CUtensorMap *>(p.tm_storage);
    const void *ptrs[4] = {q, k, v, out};
    // image part as [BH][grid_h][grid_w][d], starting after the text tokens of each (batch, head)
    const uint64_t dims4[4] = {d, gw, gh, BH};
    const uint64_t str4[3] = {row_b, gw * row_b, N * row_b};
    const uint32_t box4[4] = {64, (uint32_t)kTileW, (uint32_t)kTileH, 1};
    for (int t = 0; t < 4; ++t) {
        const char *base = static_cast<const char *>(ptrs[t]) + T * row_b;
        if (!encode_bf16_map(&tm[t], base, 4, dims4, str4, box4)) return CLEAR_ERR_CUDA;
    }
    // token sequence as [BH][N][d] (K, V) and its text prefix [BH][n_text][d] (Q, O of text tiles)
    const uint64_t dims3[3] = {d, N, BH};
    const uint64_t dims3t[3] = {d, T > 0 ? T : 1, BH};
    const uint64_t str3[2] = {row_b, N * row_b};
    const uint32_t box3[3] = {64, (uint32_t)kTileTokens, 1};
    if (!encode_bf16_map(&tm[4], q, 3, dims3t, str3, box3)) return CLEAR_ERR_CUDA;
    if (!encode_bf16_map(&tm[5], k, 3, dims3, str3, box3)) return CLEAR_ERR_CUDA;
    if (!encode_bf16_map(&tm[6], v, 3, dims3, str3, box3)) return CLEAR_ERR_CUDA;
    if (!encode_bf16_map(&tm[7], out, 3, dims3t, str3, box3)) return CLEAR_ERR_CUDA;
    for (int t = 0; t < 4; ++t) p.tm_ptrs[t] = ptrs[t];
    p.tm_valid = true;
    return CLEAR_OK;
}

template <int D>
int launch_variant(const clear_plan &p, const CUtensorMap *tm, const TcParams &prm, void *out, cudaStream_t stream)
{
    const Shape &s = p.shape;
    constexpr size_t kSmem = 1024 + 3 * (size_t)(D / 64) * 16384 + sizeof(Ctrl) + 64;
    static bool configured[64] = {};  // the attribute is set once per device
    if (p.device >= 0 && p.device < 64 && !configured[p.device]) {
        CLEAR_CUDA_TRY(cudaFuncSetAttribute(clear_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)kSmem));
        configured[p.device] = true;
    }
    dim3 grid((unsigned)p.sch.items.size(), (unsigned)(s.B * s.H));
    clear_tc_kernel<D><<<grid, kThreads, kSmem, stream>>>(tm[0], tm[1], tm[2], tm[3], tm[4], tm[5], tm[6], tm[7],
                                                                  prm);
    CLEAR_CUDA_TRY(cudaGetLastError());
    return launch_text_combine(p, out, stream);
}

}  // namespace

int launch_text_combine(const clear_plan &p, void *out, cudaStream_t stream)
{
    const Shape &s = p.shape;
    // the text part of a band leaves records for the merge over all bands instead of finished rows
    if (s.part == CLEAR_PART_BAND_TEXT) return launch_text_export(p, out, stream);
    if (p.sch.n_partial_slots <= 0) return CLEAR_OK;
    const int64_t N = (int64_t)s.n_text + (int64_t)s.grid_h * s.grid_w;
    dim3 cgrid((unsigned)s.n_text, (unsigned)(s.B * s.H));
    if (s.head_dim == 128)
        clear_tc_combine_kernel<128><<<cgrid, 128, 0, stream>>>(p.d_partial_o, p.d_partial_ml, (__nv_bfloat16 *)out,
                                                                s.n_text, N, p.sch.n_text_splits, p.sch.n_partial_slots);
    else if (s.head_dim == 64)
        clear_tc_combine_kernel<64><<<cgrid, 64, 0, stream>>>(p.d_partial_o, p.d_partial_ml, (__nv_bfloat16 *)out,
                                                              s.n_text, N, p.sch.n_text_splits, p.sch.n_partial_slots);
    else
        return CLEAR_ERR_UNSUPPORTED;
    CLEAR_CUDA_TRY(cudaGetLastError());
    return CLEAR_OK;
}

int launch_tc(const clear_plan &p, const void *q, const void *k, const void *v, void *out, float scale,
              cudaStream_t stream)
{
    if (!(scale > 0.f)) return CLEAR_ERR_UNSUPPORTED;
    CUtensorMap tm[8];
    {
        std::lock_guard<std::mutex> lock(p.tm_mutex);
        if (!(p.tm_valid && p.tm_ptrs[0] == q && p.tm_ptrs[1] == k && p.tm_ptrs[2] == v && p.tm_ptrs[3] == out)) {
            int rc = build_maps(p, q, k, v, out);
            if (rc != CLEAR_OK) {
                p.tm_valid = false;
                return rc;
            }
        }
        std::memcpy(tm, p.tm_storage, sizeof(tm));
    }
    TcParams prm;
    prm.items = p.d_items;
    prm.tiles = p.d_tiles;
    prm.half_width = p.d_half_width;
    prm.n_half_width = (int)p.sch.half_width.size();
    prm.grid_h = p.shape.grid_h;
    prm.grid_w = p.shape.grid_w;
    prm.n_text = p.shape.n_text;
    prm.scale_log2 = scale * 1.4426950408889634f;
    prm.partial_o = p.d_partial_o;
    prm.partial_ml = p.d_partial_ml;
    prm.n_partial_slots = p.sch.n_partial_slots;
    prm.status = p.d_status;
    if (p.shape.head_dim == 128) return launch_variant<128>(p, tm, prm, out, stream);
    if (p.shape.head_dim == 64) return launch_variant<64>(p, tm, prm, out, stream);
    return CLEAR_ERR_UNSUPPORTED;
}

}  // namespace clear
