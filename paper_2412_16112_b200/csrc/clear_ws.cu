// CLEAR attention forward on the sm_100a tensor cores: persistent, warp-specialised kernel.
//
// One thread block per SM takes work items from a queue (an atomic counter).  A work item is a PAIR
// of 128-query tiles -- two vertically adjacent 8 x 16 patches of the latent grid, or two tiles of
// text tokens -- and a list of steps; in each step every query tile of the pair meets one 128-key
// tile (Eq. 1 restricted by Eq. 3).  Key tiles both query tiles need are staged once.
//
// Roles (384 threads):
//   warp 0        : takes items from the queue and issues every TMA load (Q tiles, K/V ring);
//   warp 1        : one thread issues every tcgen05.mma, alternating between the two query tiles:
//                   S_t = Q_t K^T, O_t += P_t V; the softmax of one tile runs under the MMAs of the other;
//   warps 4-7     : softmax and epilogue of query tile 0 (thread r owns query row r = tensor-memory
//                   lane r): running maximum, P = exp2(.) on the keys Eq. 3 allows and 0 elsewhere, as
//                   bf16 into tensor memory over S, row sum; at the end of an item O / l -> bf16 ->
//                   global memory (or fp32 partial results of split text rows);
//   warps 8-11    : the same for query tile 1.
// Tensor memory (512 columns): S0 | S1 | O0 | O1, 128 columns each; P_t takes the first 64 columns of
// S_t and is the tensor-memory operand of P_t V, so that P never crosses shared memory: with both MMA
// operands in shared memory a 128 x 128 x 16 MMA reads 8 KB per 64 clocks, all a shared memory can
// deliver, and nothing else (P stores, TMA fills) fits beside it.
// Shared memory: Q0, Q1 and a ring of five key/value stages (K and V tiles take one stage each).
// Every wait is bounded: on expiry the block raises the plan's status word and leaves.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <type_traits>

#include "clear_internal.hpp"
#include "ptx.cuh"

namespace clear {
namespace {

constexpr int kWsThreads = 384;   // 4 control warps + 2 x 4 softmax warps
constexpr int kRing = 5;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr uint32_t kWaitHintNs = 20000;            // one sleep inside try_wait
constexpr uint64_t kWaitLimitNs = 2000000000ull;   // a wait that lasts 2 s has failed
constexpr float kRescaleThreshold = 8.f;  // log2 units: O is rescaled only when the row max grows by more
constexpr float kMaxTileSum = 256.f;      // 2^kRescaleThreshold: a row sum of P up to this needs no look at the maximum
constexpr int kSchedDepth = 2;
// arrivals that free a queue slot: the MMA thread and one lane of each of the 8 softmax warps
constexpr uint32_t kSchedReaders = 9;
// registers per thread of each role: 128 x 80 + 256 x 208 = 63488, within what the block is launched with
// (384 threads x 168); raising a warp's budget only draws on registers other warps of the block gave back
constexpr uint32_t kRegsControl = 80, kRegsSoftmax = 208;
static_assert(128 * kRegsControl + 256 * kRegsSoftmax <= 384 * 168, "a raise beyond the block's registers would wait for ever");

// Optional timeline of the softmax warps (compile with -DCLEAR_WS_TRACE): clocks per phase, summed over the
// launch, printed by block 0.  Off in the product build.
#ifdef CLEAR_WS_TRACE
#define TRACE_DECL unsigned long long tr_acc[10] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0}; long long tr_t = clock64(); unsigned tr_steps = 0;
#define TRACE_MARK(i) { const long long tr_n = clock64(); tr_acc[i] += (unsigned long long)(tr_n - tr_t); tr_t = tr_n; }
#else
#define TRACE_DECL
#define TRACE_MARK(i)
#endif

struct WsParams {
    const clear_pair_item_t *items;
    const clear_pair_step_t *steps;
    const int32_t *half_width;
    const uint32_t *mask_table;  // [entry][128 query rows][4 words]: Eq. 3 per relative patch offset
    int n_half_width;
    int grid_h, grid_w, n_text;
    long long n_tokens;
    int n_items, n_text_items, n_bh;
    float scale_log2;  // scale * log2(e)
    float *partial_o;
    float *partial_ml;
    int n_partial_slots;
    __nv_bfloat16 *out;
    int *status;  // [0] status word of this launch, [1] queue head, [2] finished blocks, [3] status kept for the host
};

struct Ctrl {
    uint64_t q_full[2], q_empty[2];
    uint64_t kv_full[kRing], kv_empty[kRing];
    uint64_t s_full[2], p_ready[2], o_full[2], o_empty[2];
    uint64_t sched_full[kSchedDepth], sched_empty[kSchedDepth];
    uint64_t drain[1];
    int32_t sched_item[kSchedDepth];            // queue position, >= total: no more work
    int32_t sched_bh[kSchedDepth];
    clear_pair_item_t sched_rec[kSchedDepth];   // the item's record, read once from global memory
    uint32_t tmem_base;
    int abort_flag;
    int skip;
};

// Bounded wait on an mbarrier phase.  Returns false once the block has given up.  The polling loop is
// kept to two instructions per try, and roles that can afford it (SLEEP_NS > 0) sleep between tries:
// a busily polling warp takes issue slots and instruction-cache lines from the softmax warps.
template <uint32_t SLEEP_NS>
__device__ __forceinline__ bool wait_bar_slow(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, int code)
{
    const uint64_t t0 = ptx::globaltimer_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 128; ++i) {
            if (ptx::mbar_try_wait_hint(bar, parity, kWaitHintNs)) return true;
            if (SLEEP_NS > 0) __nanosleep(SLEEP_NS);
        }
        if (*abort_flag) return false;
        if (ptx::globaltimer_ns() - t0 > kWaitLimitNs) break;
    }
    *abort_flag = 1;
    atomicCAS(status, 0, code);  // the first wait that expired names the cause
    return false;
}
template <uint32_t SLEEP_NS = 0>
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, int code)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    return wait_bar_slow<SLEEP_NS>(bar, parity, abort_flag, status, code);
}
// One arrival for the whole warp, after every lane has got here (and its earlier writes with it).
__device__ __forceinline__ void warp_arrive(uint32_t bar, int lane)
{
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(bar);
}
// Drain: wait for a phase regardless of the abort flag (used before leaving with copies in flight).
__device__ __forceinline__ void drain_bar(uint32_t bar, uint32_t parity)
{
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (ptx::mbar_try_wait(bar, parity)) return;
        if (it > 64) __nanosleep(256);
    }
}

struct ItemRef {
    int bh;
    int item;
};
// Queue position -> (batch*head, item): every text item of every head first, then the image items.
__device__ __forceinline__ ItemRef decode_item(const WsParams &prm, int g)
{
    ItemRef r;
    const int n_txt_all = prm.n_text_items * prm.n_bh;
    if (g < n_txt_all) {
        r.bh = g / prm.n_text_items;
        r.item = g - r.bh * prm.n_text_items;
    } else {
        const int n_img = prm.n_items - prm.n_text_items;
        const int g2 = g - n_txt_all;
        r.bh = g2 / n_img;
        r.item = prm.n_text_items + (g2 - r.bh * n_img);
    }
    return r;
}

__device__ __forceinline__ clear_pair_step_t load_step(const clear_pair_step_t *p)
{
    const int4 a = __ldg(reinterpret_cast<const int4 *>(p));
    const int4 b = __ldg(reinterpret_cast<const int4 *>(p) + 1);
    clear_pair_step_t s;
    s.x0 = a.x; s.y0 = a.y; s.x1 = a.z; s.y1 = a.w;
    s.flags = b.x; s.n_valid0 = b.y; s.n_valid1 = b.z; s.load_base = b.w;
    return s;
}
__device__ __forceinline__ clear_pair_item_t load_item(const clear_pair_item_t *p)
{
    const int4 a = __ldg(reinterpret_cast<const int4 *>(p));
    const int4 b = __ldg(reinterpret_cast<const int4 *>(p) + 1);
    const int4 c = __ldg(reinterpret_cast<const int4 *>(p) + 2);
    clear_pair_item_t it;
    it.kind = a.x; it.n_sides = a.y; it.qx = a.z; it.qy0 = a.w;
    it.qy1 = b.x; it.n_rows0 = b.y; it.n_rows1 = b.z; it.step_begin = b.w;
    it.step_count = c.x; it.n_loads = c.y; it.partial_slot0 = c.z; it.partial_slot1 = c.w;
    return it;
}
// The part of a step record the softmax of one query tile of the pair needs on every step.
struct SideStep {
    int flags, n_valid;
};
__device__ __forceinline__ SideStep load_side_step(const clear_pair_step_t *p, int side)
{
    const int4 b = __ldg(reinterpret_cast<const int4 *>(p) + 1);
    SideStep s;
    s.flags = b.x;
    s.n_valid = side ? b.z : b.y;
    return s;
}
// Origin of the key patch of that tile (only clipped patches and plans without a mask table need it).
__device__ __forceinline__ int2 load_side_origin(const clear_pair_step_t *p, int side)
{
    const int4 a = __ldg(reinterpret_cast<const int4 *>(p));
    return side ? make_int2(a.z, a.w) : make_int2(a.x, a.y);
}
static_assert(sizeof(clear_pair_step_t) == 32 && sizeof(clear_pair_item_t) == 48, "table records are read as int4");

__device__ __forceinline__ bool step_uses(int flags, int side) { return (flags & (side ? CLEAR_STEP_USE1 : CLEAR_STEP_USE0)) != 0; }
// A step's K tiles, and its V tiles, take one ring position per distinct key tile (tile 0's first):
__device__ __forceinline__ int step_tile_index(int flags, int side)
{
    if (side == 0 || (flags & CLEAR_STEP_SHARED)) return 0;
    return (flags & CLEAR_STEP_USE0) ? 1 : 0;
}

// The last block of a launch to leave: the work queue goes back to zero, and a status some block raised
// moves to the word that stays until the host has read it, so that the next launch starts clean.
__device__ __forceinline__ void close_launch(int *status)
{
    atomicExch(status + 1, 0);
    atomicExch(status + 2, 0);
    const int raised = atomicExch(status, 0);
    if (raised != 0) atomicCAS(status + 3, 0, raised);
}

template <int D>
__global__ void __launch_bounds__(kWsThreads, 1)
clear_ws_kernel(const __grid_constant__ CUtensorMap tm_q_img, const __grid_constant__ CUtensorMap tm_k_img,
                const __grid_constant__ CUtensorMap tm_v_img, const __grid_constant__ CUtensorMap tm_q_txt,
                const __grid_constant__ CUtensorMap tm_k_lin, const __grid_constant__ CUtensorMap tm_v_lin,
                const WsParams prm)
{
    constexpr int kHalves = D / 64;                 // 64-channel (128-byte) column blocks of a tile
    constexpr uint32_t kHalfBytes = 128 * 128;      // 128 rows x 128 B
    constexpr uint32_t kTileBytes = kHalves * kHalfBytes;
    constexpr uint32_t kIdescQK = ptx::idesc_bf16(128, false);
    constexpr uint32_t kIdescPV = ptx::idesc_bf16(D, true);

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t smem_base = ptx::smem_u32(smem_raw);
    // Q0, Q1 | ring of K/V stages | control
    const uint32_t sQ = smem_base, sRing = sQ + 2 * kTileBytes;
    constexpr uint32_t kCtrlOff = (2 + kRing) * kTileBytes;
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(smem_raw + kCtrlOff);
    volatile int *abort_flag = &ctrl->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int total_items = prm.n_items * prm.n_bh;

    // once any block of this launch has given up, the rest of the grid leaves at once; a window that
    // is not 1024-byte aligned (never expected) cannot hold swizzled tiles
    if (tid == 0) {
        int skip = *reinterpret_cast<volatile int *>(prm.status);
        if ((smem_base & 1023u) != 0u) {
            atomicExch(prm.status, 100);
            skip = 1;
        }
        ctrl->skip = skip;
    }
    __syncthreads();
    if (ctrl->skip != 0) {
        if (tid == 0) {
            // keep the finished-block count right so that the queue is reset for the next launch
            const int done = atomicAdd(prm.status + 2, 1);
            if (done == (int)gridDim.x - 1) close_launch(prm.status);
        }
        return;
    }

    if (tid == 0) {
        ctrl->abort_flag = 0;
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->q_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctrl->q_empty[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctrl->s_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctrl->p_ready[i]), 4);  // one arrival per softmax warp of the tile
            ptx::mbar_init(ptx::smem_u32(&ctrl->o_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctrl->o_empty[i]), 4);
        }
        for (int i = 0; i < kRing; ++i) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->kv_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctrl->kv_empty[i]), 1);
        }
        for (int i = 0; i < kSchedDepth; ++i) {
            ptx::mbar_init(ptx::smem_u32(&ctrl->sched_full[i]), 1);
            ptx::mbar_init(ptx::smem_u32(&ctrl->sched_empty[i]), kSchedReaders);
        }
        ptx::mbar_init(ptx::smem_u32(&ctrl->drain[0]), 1);
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&ctrl->tmem_base), kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = ctrl->tmem_base;

    if (warp < 4) {
        ptx::setmaxnreg_dec<kRegsControl>();
        if (warp == 0 && lane == 0) {
            // ================= loader: work queue + every TMA load ====================================
            uint32_t n_loads = 0;    // K/V stages filled so far by this block
            uint32_t n_q[2] = {0, 0};
            for (uint32_t k = 0;; ++k) {
                const uint32_t slot = k % kSchedDepth, use = k / kSchedDepth;
                if (!wait_bar<200>(ptx::smem_u32(&ctrl->sched_empty[slot]), (use & 1u) ^ 1u, abort_flag, prm.status, 1)) break;
                const int g = atomicAdd(prm.status + 1, 1);
                ItemRef ref{0, 0};
                clear_pair_item_t item{};
                if (g < total_items) {
                    ref = decode_item(prm, g);
                    item = load_item(prm.items + ref.item);
                    ctrl->sched_rec[slot] = item;
                    ctrl->sched_bh[slot] = ref.bh;
                }
                ctrl->sched_item[slot] = g;
                ptx::mbar_arrive(ptx::smem_u32(&ctrl->sched_full[slot]));
                if (g >= total_items) break;
                bool ok = true;
                for (int t = 0; t < item.n_sides && ok; ++t) {
                    const uint32_t bar = ptx::smem_u32(&ctrl->q_full[t]);
                    ok = wait_bar<200>(ptx::smem_u32(&ctrl->q_empty[t]), (n_q[t] & 1u) ^ 1u, abort_flag, prm.status, 2);
                    if (!ok) break;
                    ptx::mbar_expect_tx(bar, kTileBytes);
#pragma unroll
                    for (int h = 0; h < kHalves; ++h) {
                        const uint32_t dst = sQ + t * kTileBytes + h * kHalfBytes;
                        if (item.kind == 1)
                            ptx::tma_load_3d(dst, &tm_q_txt, bar, h * 64, item.qx + t * 128, ref.bh);
                        else
                            ptx::tma_load_4d(dst, &tm_q_img, bar, h * 64, item.qx, t ? item.qy1 : item.qy0, ref.bh);
                    }
                    ++n_q[t];
                }
                // K/V stages in the plan's staging order: for every step its K tiles, then its V tiles
                auto stage_tiles = [&](const clear_pair_step_t &st, int kv) {
                    const bool has_a = (st.flags & CLEAR_STEP_USE0) != 0;
                    const bool has_b = (st.flags & CLEAR_STEP_USE1) && !(st.flags & CLEAR_STEP_SHARED);
                    const bool linear = (st.flags & CLEAR_STEP_LINEAR) != 0;
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        if (!ok || (t == 0 ? !has_a : !has_b)) continue;
                        const uint32_t stage = n_loads % kRing, fill = n_loads / kRing;
                        ok = wait_bar<100>(ptx::smem_u32(&ctrl->kv_empty[stage]), (fill & 1u) ^ 1u, abort_flag, prm.status, 3);
                        if (!ok) continue;
                        const uint32_t bar = ptx::smem_u32(&ctrl->kv_full[stage]);
                        const uint32_t dst = sRing + stage * kTileBytes;
                        const int x = t ? st.x1 : st.x0, y = t ? st.y1 : st.y0;
                        ptx::mbar_expect_tx(bar, kTileBytes);
#pragma unroll
                        for (int h = 0; h < kHalves; ++h) {
                            if (linear)
                                ptx::tma_load_3d(dst + h * kHalfBytes, kv ? &tm_v_lin : &tm_k_lin, bar, h * 64, x, ref.bh);
                            else
                                ptx::tma_load_4d(dst + h * kHalfBytes, kv ? &tm_v_img : &tm_k_img, bar, h * 64, x, y, ref.bh);
                        }
                        ++n_loads;
                    }
                };
                const clear_pair_step_t *steps = prm.steps + item.step_begin;
                clear_pair_step_t st = load_step(steps);
                for (int s = 0; s < item.step_count && ok; ++s) {
                    // records are fetched ahead of their use, so their latency is off the critical path
                    clear_pair_step_t st_next = st;
                    if (s + 1 < item.step_count) st_next = load_step(steps + s + 1);
                    stage_tiles(st, 0);
                    stage_tiles(st, 1);
                    st = st_next;
                }
                if (!ok) break;
            }
            if (*abort_flag) {
                // leave no copy in flight: whatever was issued must land before the block exits
                for (int t = 0; t < 2; ++t)
                    if (n_q[t] > 0) drain_bar(ptx::smem_u32(&ctrl->q_full[t]), (n_q[t] - 1) & 1u);
                for (uint32_t j = 0; j < (uint32_t)kRing && j < n_loads; ++j) {
                    const uint32_t idx = n_loads - 1 - j;
                    drain_bar(ptx::smem_u32(&ctrl->kv_full[idx % kRing]), (idx / kRing) & 1u);
                }
            }
        } else if (warp == 1) {
            // ================= MMA issuer: S_t = Q_t K^T, O_t += P_t V for both query tiles ============
            // One thread issues for both tiles in a fixed order -- at every step, for t = 0, 1:
            // P_t V of tile t's previous step (as soon as its softmax warps have put P_t into tensor
            // memory), then S_t = Q_t K^T of this step, which overwrites P_t only after P_t V has read it
            // (same issue order, same pipe).  The tensor core runs the groups in that order, so S_0 is
            // ready half a step before S_1, the two softmax phases settle half a step apart, and each
            // tile's exponentials run under the other tile's MMAs.
            // The whole warp walks the loop in step and one elected lane issues: with warp-uniform control
            // flow and values the descriptor arithmetic stays on the uniform datapath, and an MMA costs few
            // enough issue slots to keep the tensor core fed while the softmax warps of the same scheduler
            // are in their exponential phase (a lone thread in a divergent branch could not: 96 clocks per
            // MMA against 64 of execution).
            constexpr uint32_t kDescHiK = ptx::smem_desc_hi_sw128(1024);  // 8-row groups are 1024 bytes apart
            auto uni = [](int v) { return __shfl_sync(0xffffffffu, v, 0); };  // tells the compiler v is warp-uniform
            uint32_t ring_base = 0;  // K/V stages filled by the items before this one
            uint32_t n_it[2] = {0, 0};   // items in which the query tile existed
            uint32_t n_pv[2] = {0, 0};   // steps whose P V has been issued
            bool ok = true;
            TRACE_DECL
            // Every staged tile is read by this warp: it waits once for the fill of a ring position and
            // frees the stage with an MMA commit behind the last MMA that reads it (a key tile both query
            // tiles share is read by tile 0 first and freed behind tile 1's MMA).
            auto kv_wait = [&](uint32_t pos) {
                if (ok)
                    ok = __all_sync(0xffffffffu, wait_bar(ptx::smem_u32(&ctrl->kv_full[pos % kRing]), (pos / kRing) & 1u, abort_flag, prm.status, 4));
            };
            for (uint32_t k = 0; ok; ++k) {
                const uint32_t slot = k % kSchedDepth, use = k / kSchedDepth;
                if (!__all_sync(0xffffffffu, wait_bar(ptx::smem_u32(&ctrl->sched_full[slot]), use & 1u, abort_flag, prm.status, 5))) break;
                const int g = uni(ctrl->sched_item[slot]);
                const int n_sides = uni(ctrl->sched_rec[slot].n_sides);
                const int step_begin = uni(ctrl->sched_rec[slot].step_begin);
                const int n = uni(ctrl->sched_rec[slot].step_count);
                const int n_loads = uni(ctrl->sched_rec[slot].n_loads);
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->sched_empty[slot]));
                if (g >= total_items) break;
                const clear_pair_step_t *steps = prm.steps + step_begin;
                for (int t = 0; t < n_sides && ok; ++t)
                    ok = __all_sync(0xffffffffu, wait_bar(ptx::smem_u32(&ctrl->q_full[t]), n_it[t] & 1u, abort_flag, prm.status, 6));
                if (!ok) break;

                // One group of MMAs for query tile t: O_t += P_t V of its previous step (if one is pending:
                // pv), then S_t = Q_t K^T of this step (if it takes part: qk).  Everything that does not
                // need P_t -- the fills of the V and K stages, the descriptors -- comes before the wait for
                // P_t, so that between the arrival of P_t and the MMAs lie as few instructions as possible:
                // this warp shares its scheduler with two softmax warps in their exponential phase.
                //   P_t V : P_t (bf16 pairs) in the first 64 columns of S_t, 16 keys = 8 columns; V MN-major,
                //           16 keys are 16 rows of 128 bytes = 2048 bytes;
                //   Q K^T : both operands K-major: 16 contraction channels are 32 bytes along a 128-byte row,
                //           the next 64 channels are the tile's second half.
                auto issue_group = [&](int t, bool pv, int pv_flags, int pv_base, bool first_pv, bool qk, int qk_flags,
                                       int qk_base, bool last) {
                    const bool pv_shared = (pv_flags & CLEAR_STEP_SHARED) != 0, qk_shared = (qk_flags & CLEAR_STEP_SHARED) != 0;
                    const uint32_t pos_v = ring_base + ((uint32_t)pv_base >> 16) + (uint32_t)step_tile_index(pv_flags, t);
                    const uint32_t pos_k = ring_base + ((uint32_t)qk_base & 0xffffu) + (uint32_t)step_tile_index(qk_flags, t);
                    TRACE_MARK(0)
                    if (pv && !(pv_shared && t == 1)) kv_wait(pos_v);
                    if (qk && !(qk_shared && t == 1)) kv_wait(pos_k);
                    // the epilogue must have read the previous item's O_t out of tensor memory
                    if (ok && pv && first_pv)
                        ok = __all_sync(0xffffffffu, wait_bar(ptx::smem_u32(&ctrl->o_empty[t]), (n_it[t] & 1u) ^ 1u, abort_flag, prm.status, 8));
                    TRACE_MARK(1)  // wait for K, V
                    const uint32_t tmem_S = tmem + t * 128, tmem_O = tmem + 256 + t * 128;
                    const uint32_t v_lo = ptx::smem_desc_lo(sRing + (pos_v % kRing) * kTileBytes, kHalfBytes);
                    const uint32_t q_lo = ptx::smem_desc_lo(sQ + t * kTileBytes, 16);
                    const uint32_t k_lo = ptx::smem_desc_lo(sRing + (pos_k % kRing) * kTileBytes, 16);
                    const uint32_t b_vfree = ptx::smem_u32(&ctrl->kv_empty[pos_v % kRing]);
                    const uint32_t b_kfree = ptx::smem_u32(&ctrl->kv_empty[pos_k % kRing]);
                    const bool free_v = !pv_shared || t == 1, free_k = !qk_shared || t == 1;
                    if (ok && pv) ok = __all_sync(0xffffffffu, wait_bar(ptx::smem_u32(&ctrl->p_ready[t]), n_pv[t] & 1u, abort_flag, prm.status, 7));
                    if (!ok) return;
                    TRACE_MARK(4)  // wait for P
                    ptx::tc_fence_after();
                    if (ptx::elect_one()) {
                        if (pv) {
                            ptx::mma_ts(tmem_O, tmem_S, ptx::make_desc(v_lo, kDescHiK), kIdescPV, first_pv ? 0u : 1u);
#pragma unroll
                            for (int kk = 1; kk < 8; ++kk)
                                ptx::mma_ts_c<true>(tmem_O, tmem_S + kk * 8, ptx::make_desc(v_lo + kk * (2048 >> 4), kDescHiK), kIdescPV);
                            if (free_v) ptx::tc_commit(b_vfree);
                        }
                        if (qk) {
                            ptx::mma_ss_c<false>(tmem_S, ptx::make_desc(q_lo, kDescHiK), ptx::make_desc(k_lo, kDescHiK), kIdescQK);
#pragma unroll
                            for (int kk = 1; kk < D / 16; ++kk) {
                                const uint32_t off16 = ((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4;
                                ptx::mma_ss_c<true>(tmem_S, ptx::make_desc(q_lo + off16, kDescHiK),
                                                    ptx::make_desc(k_lo + off16, kDescHiK), kIdescQK);
                            }
                            ptx::tc_commit(ptx::smem_u32(&ctrl->s_full[t]));
                            if (free_k) ptx::tc_commit(b_kfree);
                        }
                        // the item's last group of the tile: its output is complete once these MMAs are
                        if (last) ptx::tc_commit(ptx::smem_u32(&ctrl->o_full[t]));
                    }
                    __syncwarp();
                    if (pv) ++n_pv[t];
                    TRACE_MARK(5)  // issue
                };

                int pend_flags[2] = {0, 0}, pend_base[2] = {0, 0};  // the step whose P_t V is still to be issued
                bool pending[2] = {false, false};
                bool first_pv[2] = {true, true};
                int4 rec = __ldg(reinterpret_cast<const int4 *>(steps) + 1);  // flags, n_valid0, n_valid1, load_base
                for (int s = 0; s < n && ok; ++s) {
                    const int flags = uni(rec.x), load_base = uni(rec.w);
                    if (s + 1 < n) rec = __ldg(reinterpret_cast<const int4 *>(steps + s + 1) + 1);  // one step ahead
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        if (t >= n_sides || !ok) continue;
                        const bool qk = step_uses(flags, t);
                        if (!pending[t] && !qk) continue;
                        issue_group(t, pending[t], pend_flags[t], pend_base[t], first_pv[t], qk, flags, load_base, false);
                        if (pending[t]) first_pv[t] = false;
                        pending[t] = qk;
                        pend_flags[t] = flags;
                        pend_base[t] = load_base;
                    }
                }
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (t >= n_sides || !ok) continue;
                    // every Q_t K^T of the item has been issued: the next item's Q tile may land
                    if (ptx::elect_one()) ptx::tc_commit(ptx::smem_u32(&ctrl->q_empty[t]));
                    __syncwarp();
                    issue_group(t, pending[t], pend_flags[t], pend_base[t], first_pv[t], false, 0, 0, true);
                    ++n_it[t];
                }
                ring_base += (uint32_t)n_loads;
            }
#ifdef CLEAR_WS_TRACE
            TRACE_MARK(0)
            if (blockIdx.x == 0 && lane == 0)
                printf("mma thread: other %llu waitK %llu issueQK %llu waitV %llu waitP %llu issuePV %llu\n", tr_acc[0], tr_acc[1],
                       tr_acc[2], tr_acc[3], tr_acc[4], tr_acc[5]);
#endif
            if (*abort_flag) {
                // MMAs that were issued must retire before tensor memory is given back
                if (lane == 0) {
                    ptx::tc_commit(ptx::smem_u32(&ctrl->drain[0]));
                    drain_bar(ptx::smem_u32(&ctrl->drain[0]), 0);
                }
            }
        }
        __syncwarp();
    } else {
        // ================= softmax warps: thread r owns query row r (tensor-memory lane r) of its tile =====
        // Per step: S_t into registers, row maximum, P = exp2(.) under the Eq. 3 mask as bf16 into tensor
        // memory over S_t, row sum; at the end of an item O_t / l -> bf16 -> global memory (or fp32 partial
        // results of split text rows).
        ptx::setmaxnreg_inc<kRegsSoftmax>();
        TRACE_DECL
        const int t = (warp - 4) >> 2;  // query tile of the pair
        const int q4 = warp & 3;        // tensor-memory lane quadrant
        const int r = q4 * 32 + lane;   // query row of the tile
        const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
        const uint32_t tmem_S = tmem + t * 128, tmem_O = tmem + 256 + t * 128;
        const float c = prm.scale_log2;
        const uint32_t b_s = ptx::smem_u32(&ctrl->s_full[t]), b_pready = ptx::smem_u32(&ctrl->p_ready[t]);
        uint32_t n_s = 0, n_items_seen = 0;
        bool alive = true;
        for (uint32_t k = 0; alive; ++k) {
            const uint32_t slot = k % kSchedDepth, use = k / kSchedDepth;
            if (!__all_sync(0xffffffffu, wait_bar(ptx::smem_u32(&ctrl->sched_full[slot]), use & 1u, abort_flag, prm.status, 9)))
                break;
            const int g = ctrl->sched_item[slot];
            const clear_pair_item_t item = ctrl->sched_rec[slot];
            const int bh = ctrl->sched_bh[slot];
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&ctrl->sched_empty[slot]));
            if (g >= total_items) break;
            if (t >= item.n_sides) continue;
            const clear_pair_step_t *steps = prm.steps + item.step_begin;
            const int step_count = item.step_count;
            const bool is_text = item.kind == 1;
            // grid position of this row's query (image tiles), and whether the row exists
            const int q_y = (t ? item.qy1 : item.qy0) + (r >> 4), q_x = item.qx + (r & 15);
            const bool q_valid = is_text ? r < (t ? item.n_rows1 : item.n_rows0) : (q_y < prm.grid_h && q_x < prm.grid_w);
            float m_used = -INFINITY, l = 0.f;
            bool first = true;

            // Step records are fetched two steps ahead and this row's precomputed mask words one step ahead,
            // so that neither latency is on the critical path.
            const int kMaskedBit = t ? CLEAR_STEP_MASKED1 : CLEAR_STEP_MASKED0;
            auto load_mask_row = [&](const SideStep &q) -> uint4 {
                if (step_uses(q.flags, t) && (q.flags & kMaskedBit) && !(q.flags & CLEAR_STEP_LINEAR) && q.n_valid >= 0)
                    return __ldg(reinterpret_cast<const uint4 *>(prm.mask_table) + ((size_t)q.n_valid * 128 + r));
                return make_uint4(0u, 0u, 0u, 0u);
            };
            SideStep st_next = load_side_step(steps, t);
            SideStep st_next2 = st_next;
            if (step_count > 1) st_next2 = load_side_step(steps + 1, t);
            uint4 mrow_next = load_mask_row(st_next);
            TRACE_MARK(8)  // between items
            for (int s = 0; s < step_count; ++s) {
                const SideStep st = st_next;
                const uint4 mrow = mrow_next;
                st_next = st_next2;  // fetched a step ago: the mask row's address does not wait for it
                if (s + 2 < step_count) st_next2 = load_side_step(steps + s + 2, t);
                if (s + 1 < step_count) mrow_next = load_mask_row(st_next);
                if (!step_uses(st.flags, t)) continue;
                const bool masked = (st.flags & kMaskedBit) != 0;
                // ---- mask bits of this row for the tile (bit j of word w = key 32 w + j allowed) --------
                uint32_t mw[4] = {0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu};
                if (masked) {
                    if (st.flags & CLEAR_STEP_LINEAR) {
#pragma unroll
                        for (int w = 0; w < 4; ++w) {
                            const int nv = min(max(st.n_valid - 32 * w, 0), 32);
                            mw[w] = nv == 32 ? 0xffffffffu : ((1u << nv) - 1u);
                        }
                    } else if (st.n_valid >= 0) {
                        // Eq. 3 from the table; keys of the patch that lie off the grid do not exist
                        mw[0] = mrow.x;
                        mw[1] = mrow.y;
                        mw[2] = mrow.z;
                        mw[3] = mrow.w;
                        if (st.flags & (t ? CLEAR_STEP_CLIP1 : CLEAR_STEP_CLIP0)) {
                            const int2 org = load_side_origin(steps + s, t);
                            const int lo = max(0, -org.x), hi = min(15, prm.grid_w - 1 - org.x);
                            const uint32_t cols = lo <= hi ? (((1u << (hi - lo + 1)) - 1u) << lo) : 0u;
#pragma unroll
                            for (int w = 0; w < 4; ++w) {
                                const int ky0 = org.y + 2 * w, ky1 = ky0 + 1;
                                const uint32_t ok0 = (ky0 >= 0 && ky0 < prm.grid_h) ? cols : 0u;
                                const uint32_t ok1 = (ky1 >= 0 && ky1 < prm.grid_h) ? cols : 0u;
                                mw[w] &= ok0 | (ok1 << 16);
                            }
                        }
                    } else {
                        // no table entry (very large radius): Eq. 3 row by row from the half widths
                        const int2 org = load_side_origin(steps + s, t);
#pragma unroll
                        for (int w = 0; w < 4; ++w) mw[w] = 0u;
#pragma unroll 1
                        for (int rr = 0; rr < 8; ++rr) {
                            const int ky = org.y + rr;
                            const int ady = abs(ky - q_y);
                            uint32_t bits = 0u;
                            if (q_valid && ky >= 0 && ky < prm.grid_h && ady < prm.n_half_width) {
                                const int hw = __ldg(prm.half_width + ady);
                                const int lo = max(max(q_x - hw, 0), org.x);
                                const int hi = min(min(q_x + hw, prm.grid_w - 1), org.x + 15);
                                if (lo <= hi) bits = ((1u << (hi - lo + 1)) - 1u) << (lo - org.x);
                            }
                            bits <<= 16 * (rr & 1);
                            if ((rr >> 1) == 0) mw[0] |= bits;
                            if ((rr >> 1) == 1) mw[1] |= bits;
                            if ((rr >> 1) == 2) mw[2] |= bits;
                            if ((rr >> 1) == 3) mw[3] |= bits;
                        }
                    }
                }

                TRACE_MARK(0)  // step prologue: records, mask words
                // warp-uniform outcome: the tcgen05.ld / st below need the whole warp.  Once S_t of this step
                // is complete, so is P_t V of the step before (same thread, same pipe, issued earlier).
                if (!__all_sync(0xffffffffu, wait_bar(b_s, n_s & 1u, abort_flag, prm.status, 10))) {
                    alive = false;
                    break;
                }
                ++n_s;
                TRACE_MARK(1)  // wait for S
                ptx::tc_fence_after();
                uint32_t sv[4][32];
#pragma unroll
                for (int w = 0; w < 4; ++w) ptx::tmem_ld32(tmem_S + lane_off + 32 * w, sv[w]);
                ptx::tmem_wait_ld();
                TRACE_MARK(2)  // S into registers

                // ---- P = exp2(S * c - m * c) on the allowed keys, 0 elsewhere; row sum; bf16 pairs into
                // tensor memory, 32 keys (16 columns) at a time (two-wide fp32 FMA and ADD; four independent
                // partial sums)
                float tile_sum = 0.f;
                auto exp_pass = [&](auto masked_c, float mc) {
                    constexpr bool kMasked = decltype(masked_c)::value;
                    const uint64_t c2 = ptx::pack2(c, c), nmc2 = ptx::pack2(-mc, -mc);
                    uint64_t lsum[2] = {0ull, 0ull};
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        uint32_t pk[16];
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {
                            const uint64_t x2 =
                                ptx::fma2(ptx::pack2(__uint_as_float(sv[w][j]), __uint_as_float(sv[w][j + 1])), c2, nmc2);
                            float x0, x1;
                            ptx::unpack2(x2, x0, x1);
                            if (kMasked) {
                                x0 = ((mw[w] >> j) & 1u) ? x0 : -INFINITY;
                                x1 = ((mw[w] >> (j + 1)) & 1u) ? x1 : -INFINITY;
                            }
                            const float p0 = ptx::ex2(x0), p1 = ptx::ex2(x1);
                            lsum[(j >> 1) & 1] = ptx::add2(lsum[(j >> 1) & 1], ptx::pack2(p0, p1));
                            pk[j >> 1] = ptx::pack_bf16(p0, p1);
                        }
                        ptx::tmem_st16(tmem_S + lane_off + 16 * w, pk);
                    }
                    float a0, a1, a2, a3;
                    ptx::unpack2(lsum[0], a0, a1);
                    ptx::unpack2(lsum[1], a2, a3);
                    tile_sum = (a0 + a1) + (a2 + a3);
                };
                // The running maximum m of a row moves only when a tile's maximum over the allowed keys
                // exceeds it by more than the threshold, i.e. when some P of the tile would exceed
                // 2^threshold.  So P is formed against the maximum as it stands, and only when a row's sum
                // over the tile exceeds 2^threshold (no single P can otherwise), or the row has no maximum
                // yet, is the tile's maximum taken, m moved by the rule above, O rescaled and P formed again:
                // the same results as with a maximum pass on every tile, which costs a third of the
                // exponentials' time and is needed on the first tile of a row and hardly ever after.
                bool use_mask = masked;
                bool exact = __any_sync(0xffffffffu, first || (m_used == -INFINITY && q_valid));
#pragma unroll 1
                for (;;) {
                    if (exact) {
                        // maximum over the allowed keys (the scores Eq. 3 forbids become -inf in place)
                        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                        if (use_mask) {
#pragma unroll
                            for (int w = 0; w < 4; ++w)
#pragma unroll
                                for (int j = 0; j < 32; j += 2) {
                                    const float v0 = ((mw[w] >> j) & 1u) ? __uint_as_float(sv[w][j]) : -INFINITY;
                                    const float v1 = ((mw[w] >> (j + 1)) & 1u) ? __uint_as_float(sv[w][j + 1]) : -INFINITY;
                                    sv[w][j] = __float_as_uint(v0);
                                    sv[w][j + 1] = __float_as_uint(v1);
                                    mx4[(j >> 1) & 3] = ptx::max3(mx4[(j >> 1) & 3], v0, v1);
                                }
                            use_mask = false;
                        } else {
#pragma unroll
                            for (int w = 0; w < 4; ++w)
#pragma unroll
                                for (int j = 0; j < 32; j += 2)
                                    mx4[(j >> 1) & 3] = ptx::max3(mx4[(j >> 1) & 3], __uint_as_float(sv[w][j]), __uint_as_float(sv[w][j + 1]));
                        }
                        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                        const float m_new = fmaxf(m_used, mx);
                        if (first) {
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
#pragma unroll 1
                                for (int w = 0; w < D / 16; ++w) {
                                    uint32_t o[16];
                                    ptx::tmem_ld16(tmem_O + lane_off + 16 * w, o);
                                    ptx::tmem_wait_ld();
#pragma unroll
                                    for (int j = 0; j < 16; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
                                    ptx::tmem_st16(tmem_O + lane_off + 16 * w, o);
                                }
                            }
                        }
                    }
                    const float mc = (m_used == -INFINITY) ? 0.f : m_used * c;
                    if (use_mask)
                        exp_pass(std::true_type{}, mc);
                    else
                        exp_pass(std::false_type{}, mc);
                    if (exact) break;
                    exact = __any_sync(0xffffffffu, !(tile_sum <= kMaxTileSum));  // also for a NaN
                    if (!exact) break;
                }
                first = false;
                l += tile_sum;
                TRACE_MARK(5)  // exponentials
                // P_t (and a rescaled O_t) must be in tensor memory before the MMA thread is told
                ptx::tmem_wait_st();
                ptx::tc_fence_before();
                warp_arrive(b_pready, lane);
                TRACE_MARK(6)  // arrival
#ifdef CLEAR_WS_TRACE
                ++tr_steps;
#endif
            }
            if (!alive) break;
            TRACE_MARK(0)

            // ---- epilogue: the last P_t V has retired once o_full completes; O_t / l -> global memory -----
            if (!__all_sync(0xffffffffu, wait_bar(ptx::smem_u32(&ctrl->o_full[t]), n_items_seen & 1u, abort_flag, prm.status, 14)))
                break;
            ++n_items_seen;
            ptx::tc_fence_after();
            const int slot_p = t ? item.partial_slot1 : item.partial_slot0;
            if (slot_p >= 0) {
                // split text-query tile: un-normalised fp32 row, its maximum (log2 units) and its sum
                const long long row = ((long long)bh * prm.n_partial_slots + slot_p) * 128 + r;
                float *dst = prm.partial_o + row * D;
#pragma unroll
                for (int w = 0; w < D / 32; ++w) {
                    uint32_t o[32];
                    ptx::tmem_ld32(tmem_O + lane_off + 32 * w, o);
                    ptx::tmem_wait_ld();
                    if (w == D / 32 - 1) {
                        ptx::tc_fence_before();
                        warp_arrive(ptx::smem_u32(&ctrl->o_empty[t]), lane);
                    }
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
                const long long token = is_text ? (long long)(item.qx + t * 128 + r) : prm.n_text + (long long)q_y * prm.grid_w + q_x;
                __nv_bfloat16 *dst = prm.out + ((long long)bh * prm.n_tokens + token) * D;
#pragma unroll
                for (int w = 0; w < D / 32; ++w) {
                    uint32_t o[32];
                    ptx::tmem_ld32(tmem_O + lane_off + 32 * w, o);
                    ptx::tmem_wait_ld();
                    if (w == D / 32 - 1) {
                        ptx::tc_fence_before();
                        warp_arrive(ptx::smem_u32(&ctrl->o_empty[t]), lane);
                    }
                    if (q_valid) {
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) {
                            uint4 val;
                            val.x = ptx::pack_bf16(__uint_as_float(o[8 * cc + 0]) * inv, __uint_as_float(o[8 * cc + 1]) * inv);
                            val.y = ptx::pack_bf16(__uint_as_float(o[8 * cc + 2]) * inv, __uint_as_float(o[8 * cc + 3]) * inv);
                            val.z = ptx::pack_bf16(__uint_as_float(o[8 * cc + 4]) * inv, __uint_as_float(o[8 * cc + 5]) * inv);
                            val.w = ptx::pack_bf16(__uint_as_float(o[8 * cc + 6]) * inv, __uint_as_float(o[8 * cc + 7]) * inv);
                            *reinterpret_cast<uint4 *>(dst + 32 * w + 8 * cc) = val;
                        }
                    }
                }
            }
            TRACE_MARK(7)  // epilogue
        }
#ifdef CLEAR_WS_TRACE
        if (blockIdx.x == 0 && lane == 0)
            printf("tile %d warp %d steps %u: prologue %llu waitS %llu ldS %llu max %llu rescale %llu exp %llu arrive %llu epilogue %llu between items %llu\n",
                   t, q4, tr_steps, tr_acc[0], tr_acc[1], tr_acc[2], tr_acc[3], tr_acc[4], tr_acc[5], tr_acc[6], tr_acc[7], tr_acc[8]);
#endif
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, kTmemCols);
    }
    if (tid == 0) {
        // the last block to finish puts the queue back to zero for the next launch
        const int done = atomicAdd(prm.status + 2, 1);
        if (done == (int)gridDim.x - 1) close_launch(prm.status);
    }
}

// ---- host side: tensor maps and launch ---------------------------------------------------------
// Maps 0..2: image part of q, k, v as [BH][grid_h][grid_w][d]; 3: text prefix of q as [BH][n_text][d];
// 4, 5: k, v as the token sequence [BH][N][d].
int build_maps(const clear_plan &p, const void *q, const void *k, const void *v)
{
    const Shape &s = p.shape;
    const uint64_t d = (uint64_t)s.head_dim, gw = (uint64_t)s.grid_w, gh = (uint64_t)s.grid_h, T = (uint64_t)s.n_text;
    const uint64_t N = T + gw * gh, BH = (uint64_t)s.B * s.H;
    const uint64_t row_b = d * 2;
    CUtensorMap *tm = reinterpret_cast<CUtensorMap *>(p.tm_storage);
    const void *ptrs[3] = {q, k, v};
    const uint64_t dims4[4] = {d, gw, gh, BH};
    const uint64_t str4[3] = {row_b, gw * row_b, N * row_b};
    const uint32_t box4[4] = {64, (uint32_t)kTileW, (uint32_t)kTileH, 1};
    for (int t = 0; t < 3; ++t) {
        const char *base = static_cast<const char *>(ptrs[t]) + T * row_b;
        if (!encode_bf16_map(&tm[t], base, 4, dims4, str4, box4)) return CLEAR_ERR_CUDA;
    }
    const uint64_t dims3[3] = {d, N, BH};
    const uint64_t dims3t[3] = {d, T > 0 ? T : 1, BH};
    const uint64_t str3[2] = {row_b, N * row_b};
    const uint32_t box3[3] = {64, (uint32_t)kTileTokens, 1};
    if (!encode_bf16_map(&tm[3], q, 3, dims3t, str3, box3)) return CLEAR_ERR_CUDA;
    if (!encode_bf16_map(&tm[4], k, 3, dims3, str3, box3)) return CLEAR_ERR_CUDA;
    if (!encode_bf16_map(&tm[5], v, 3, dims3, str3, box3)) return CLEAR_ERR_CUDA;
    for (int t = 0; t < 3; ++t) p.tm_ptrs[t] = ptrs[t];
    p.tm_ptrs[3] = nullptr;
    p.tm_valid = true;
    return CLEAR_OK;
}

struct DeviceInfo {
    bool known = false;
    int n_sm = 0;
    bool configured[2] = {false, false};
};
DeviceInfo g_dev[64];
std::mutex g_dev_mutex;

template <int D>
int launch_variant(const clear_plan &p, const CUtensorMap *tm, const WsParams &prm, cudaStream_t stream)
{
    constexpr size_t kSmem = (size_t)(2 + kRing) * (D / 64) * 16384 + sizeof(Ctrl);
    static_assert(kSmem <= 232448, "shared memory of one block");
    int n_sm = 0;
    {
        std::lock_guard<std::mutex> lock(g_dev_mutex);
        if (p.device < 0 || p.device >= 64) return CLEAR_ERR_UNSUPPORTED;
        DeviceInfo &di = g_dev[p.device];
        if (!di.known) {
            CLEAR_CUDA_TRY(cudaDeviceGetAttribute(&di.n_sm, cudaDevAttrMultiProcessorCount, p.device));
            di.known = true;
        }
        if (!di.configured[D == 128]) {
            CLEAR_CUDA_TRY(cudaFuncSetAttribute(clear_ws_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem));
            di.configured[D == 128] = true;
        }
        n_sm = di.n_sm;
    }
    const long long total = (long long)prm.n_items * prm.n_bh;
    const unsigned grid = (unsigned)std::min<long long>(n_sm, total);
    clear_ws_kernel<D><<<grid, kWsThreads, kSmem, stream>>>(tm[0], tm[1], tm[2], tm[3], tm[4], tm[5], prm);
    CLEAR_CUDA_TRY(cudaGetLastError());
    return launch_text_combine(p, prm.out, stream);
}

}  // namespace

int launch_ws(const clear_plan &p, const void *q, const void *k, const void *v, void *out, float scale,
              cudaStream_t stream)
{
    if (!(scale > 0.f)) return CLEAR_ERR_UNSUPPORTED;
    const long long total = (long long)p.sch.pair_items.size() * p.shape.B * p.shape.H;
    if (total <= 0 || total >= (1ll << 30)) return CLEAR_ERR_UNSUPPORTED;
    CUtensorMap tm[6];
    {
        std::lock_guard<std::mutex> lock(p.tm_mutex);
        if (!(p.tm_valid && p.tm_ptrs[0] == q && p.tm_ptrs[1] == k && p.tm_ptrs[2] == v)) {
            int rc = build_maps(p, q, k, v);
            if (rc != CLEAR_OK) {
                p.tm_valid = false;
                return rc;
            }
        }
        std::memcpy(tm, p.tm_storage, sizeof(tm));
    }
    WsParams prm;
    prm.items = p.d_pair_items;
    prm.steps = p.d_pair_steps;
    prm.half_width = p.d_half_width;
    prm.mask_table = p.d_mask_table;
    prm.n_half_width = (int)p.sch.half_width.size();
    prm.grid_h = p.shape.grid_h;
    prm.grid_w = p.shape.grid_w;
    prm.n_text = p.shape.n_text;
    prm.n_tokens = (long long)p.shape.n_text + (long long)p.shape.grid_h * p.shape.grid_w;
    prm.n_items = (int)p.sch.pair_items.size();
    prm.n_text_items = p.sch.n_text_pair_items;
    prm.n_bh = p.shape.B * p.shape.H;
    prm.scale_log2 = scale * 1.4426950408889634f;
    prm.partial_o = p.d_partial_o;
    prm.partial_ml = p.d_partial_ml;
    prm.n_partial_slots = p.sch.n_partial_slots;
    prm.out = static_cast<__nv_bfloat16 *>(out);
    prm.status = p.d_status;
    if (p.shape.head_dim == 128) return launch_variant<128>(p, tm, prm, stream);
    if (p.shape.head_dim == 64) return launch_variant<64>(p, tm, prm, stream);
    return CLEAR_ERR_UNSUPPORTED;
}

}  // namespace clear
