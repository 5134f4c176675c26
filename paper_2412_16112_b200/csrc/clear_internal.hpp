// Internal plan object and kernel launchers shared by the C-ABI layer and the kernels.
#pragma once

#include <cuda_runtime.h>

#include <mutex>

#include "clear_attn.h"
#include "clear_plan.hpp"

namespace clear {

// The host-tensor entry point cuts the (batch, head) axis into chunks: while chunk c is computed,
// chunk c+1 travels to the device and chunk c-1 travels back.  Each chunk size has a plan of its own
// (B = 1, H = heads of the chunk); streams and events order the three stages.
constexpr int kMaxHostChunks = 16;
struct HostPipe {
    int chunk_heads = 0;              // (b, h) slices per full chunk
    int n_chunks = 0;
    clear_plan *sub[2] = {nullptr, nullptr};  // plan of a full chunk, plan of the shorter last chunk
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_out = nullptr;
    cudaEvent_t ev_in[kMaxHostChunks] = {};
    cudaEvent_t ev_done[kMaxHostChunks] = {};
};

}  // namespace clear

struct clear_plan {
    clear::Shape shape;
    clear::Schedule sch;
    int kernel = CLEAR_KERNEL_SIMT;  // selected kernel (never AUTO)
    bool host_only = false;
    int device = -1;

    // device tables (owned)
    int32_t *d_half_width = nullptr;
    clear_work_item_t *d_items = nullptr;
    clear_kv_tile_t *d_tiles = nullptr;
    clear_pair_item_t *d_pair_items = nullptr;
    clear_pair_step_t *d_pair_steps = nullptr;
    uint32_t *d_mask_table = nullptr;
    // [0] status word of the launch in flight: 0 = fine, set by a kernel whose bounded wait expired (the
    //     rest of that launch's blocks then leave at once); the persistent kernel puts it back to zero when
    //     its last block leaves;
    // [1] work-queue head and [2] finished-block count of the persistent kernel (both back at zero
    //     when a launch ends);
    // [3] the first non-zero status of any launch since the last clear_plan_check (which reads and clears it)
    int *d_status = nullptr;

    // Launches of one plan share its work queue, status words and split-KV workspace, so the library
    // orders them on the device: a launch on another stream than the one before waits for that one's
    // end (an event recorded behind every launch).
    mutable std::mutex launch_mutex;
    mutable cudaEvent_t ev_last = nullptr;
    mutable cudaStream_t last_stream = nullptr;
    mutable bool has_last = false;

    // split-KV workspace of the text-query rows (owned): per (bh, slot) 128 x head_dim fp32
    // un-normalised outputs, and per row the running maximum (log2 units) and the row sum
    float *d_partial_o = nullptr;
    float *d_partial_ml = nullptr;
    // backward pass: (m, 1 / l, delta) per query row, allocated on the plan's first backward call
    mutable float *d_bwd_stats = nullptr;
    int64_t workspace_bytes = 0;

    // staging buffers of the host-tensor entry point (owned, allocated on first use)
    void *d_stage[4] = {nullptr, nullptr, nullptr, nullptr};
    // copy/compute pipeline of the host-tensor entry point (owned, built on first use; null while
    // the whole problem goes through in one piece)
    clear::HostPipe *pipe = nullptr;
    bool pipe_decided = false;

    // tensor maps of the last (q, k, v, out) seen by the tensor-core launcher
    mutable std::mutex tm_mutex;
    mutable const void *tm_ptrs[4] = {nullptr, nullptr, nullptr, nullptr};
    alignas(64) mutable unsigned char tm_storage[8][128];
    mutable bool tm_valid = false;
};

namespace clear {

// Thread-local record of the last failing CUDA call.
void note_cuda_error(int err);

#define CLEAR_CUDA_TRY(expr)                          \
    do {                                              \
        cudaError_t _e = (expr);                      \
        if (_e != cudaSuccess) {                      \
            clear::note_cuda_error((int)_e);          \
            (void)cudaGetLastError();                 \
            return CLEAR_ERR_CUDA;                    \
        }                                             \
    } while (0)

int launch_simt(const clear_plan &p, const void *q, const void *k, const void *v, void *out, float scale,
                cudaStream_t stream);
int launch_tc(const clear_plan &p, const void *q, const void *k, const void *v, void *out, float scale,
              cudaStream_t stream);
int launch_ws(const clear_plan &p, const void *q, const void *k, const void *v, void *out, float scale,
              cudaStream_t stream);
// Backward pass on the CUDA cores (fp32 arithmetic; tensors of the plan's dtype): a query kernel and a key kernel.
int launch_bwd(const clear_plan &p, const void *q, const void *k, const void *v, const void *d_out, void *dq, void *dk,
               void *dv, float scale, cudaStream_t stream);
// Row-band form: one (O, m, l) record per text row from a band-text plan's partial results, and the merge of the
// records of all bands into bf16 text rows.
int launch_text_export(const clear_plan &p, void *records, cudaStream_t stream);
int launch_text_merge(const float *records, int n_parts, int n_bh, int n_text, int head_dim, int mode, void *out,
                      long long out_tokens, cudaStream_t stream);
// Q/K preparation (RMS normalisation, rotary embedding, factor on Q): one elementwise pass, no plan.
int launch_qk_prep(const void *q_in, const void *k_in, void *q_out, void *k_out, const float *gain_q, const float *gain_k,
                   int n_bh, int grid_h, int grid_w, int n_text, int head_dim, int dtype, const int axes_dim[3],
                   double theta, double ntk_factor, float eps, float q_factor, cudaStream_t stream);
// Backward pass on the tensor cores (bf16): a query-role and a key-role launch over the plan's tile schedule, which
// must have been built without text splits.
int launch_bwd_tc(const clear_plan &p, const void *q, const void *k, const void *v, const void *d_out, void *dq, void *dk,
                  void *dv, float scale, cudaStream_t stream);
// Merge of the split-KV partial results of the text-query rows (both tensor-core kernels).
int launch_text_combine(const clear_plan &p, void *out, cudaStream_t stream);

// Tensor map (a CUtensorMap, 128 bytes) of a bf16 tensor of `rank` dims, innermost first, with 128-byte swizzle
// and out-of-bounds elements read as zero; strides in bytes for dims 1..rank-1.  False if the driver refuses.
bool encode_bf16_map(void *tensor_map, const void *base, int rank, const uint64_t *dims, const uint64_t *strides,
                     const uint32_t *box);

constexpr int kStatusWords = 4;

}  // namespace clear
