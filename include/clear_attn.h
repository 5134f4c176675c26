/*
 * clear_attn.h -- C ABI of the CLEAR attention forward library for NVIDIA B200 (sm_100a).
 *
 * The operator (Sec. 3.2 of the CLEAR paper, arXiv 2412.16112):
 *   tokens are [n_text text tokens ; grid_h * grid_w image tokens, row-major on the 2-D latent
 *   grid]; the attention mask of Eq. 3 allows a (query i, key j) pair when i is a text token,
 *   or j is a text token, or both are image tokens whose grid positions are at Euclidean
 *   distance strictly below `radius` (window clipped at the grid border, no wrap-around);
 *   the output is the masked softmax attention of Eq. 1,
 *       out_i = sum_j softmax_j(scale * q_i . k_j) v_j   over the allowed j,
 *   computed independently for every batch entry and head with the same mask.
 *
 * Conventions shared by every entry point
 *   - q, k, v, out are [B, H, N, head_dim] contiguous, N = n_text + grid_h * grid_w; image token
 *     p sits at grid row p / grid_w and column p % grid_w.
 *   - Unless an entry point says "host", tensor pointers are DEVICE pointers on the device that
 *     was current when the plan was created, 16-byte aligned; `out` must not overlap an input.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Forward
 *     calls only enqueue work on it and never synchronise the host.
 *   - Every function returns a clear_status code; nothing throws, aborts or prints.
 *   - The library has no CPU fallback: without a usable CUDA device the calls fail with
 *     CLEAR_ERR_CUDA.
 */
#ifndef CLEAR_ATTN_H_
#define CLEAR_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum clear_status {
    CLEAR_OK = 0,
    CLEAR_ERR_INVALID_ARG = -1,    /* null pointer, non-positive size, radius <= 0, non-finite value */
    CLEAR_ERR_UNSUPPORTED = -2,    /* shape or dtype outside what the requested kernel handles      */
    CLEAR_ERR_MISALIGNED = -3,     /* a tensor pointer is not 16-byte aligned                        */
    CLEAR_ERR_PLAN_MISMATCH = -4,  /* plan used on another device / with a kernel it was not built for */
    CLEAR_ERR_CUDA = -5,           /* a CUDA runtime or driver call failed (see clear_last_cuda_error) */
    CLEAR_ERR_DEVICE_TIMEOUT = -6, /* a bounded wait inside a kernel expired; outputs are invalid    */
    CLEAR_ERR_NO_MEMORY = -7,      /* host or device allocation failed                               */
    CLEAR_ERR_TOO_LARGE = -8       /* shape exceeds a fixed capacity of clear_attn_fwd_static        */
} clear_status;

typedef enum clear_dtype { CLEAR_BF16 = 0, CLEAR_F32 = 1 } clear_dtype;

/* Which kernel a plan drives.
 *   AUTO       : TCGEN05_WS when it applies (bf16, head_dim 64 or 128, scale > 0 at call time), else SIMT.
 *   SIMT       : exact-order fp32 CUDA-core kernel; any head_dim <= 256, bf16 or fp32 tensors.
 *   TCGEN05    : block-sparse flash-style kernel on the 5th-generation tensor cores (TMA + TMEM), one
 *                128-query tile per thread block, two blocks per SM.
 *   TCGEN05_WS : the same mathematics as a persistent, warp-specialised kernel: one block per SM walks a
 *                work queue; each work item is a PAIR of 128-query tiles (two vertically adjacent grid
 *                patches, or two text tiles) that share every key/value tile both of them need. */
typedef enum clear_kernel {
    CLEAR_KERNEL_AUTO = 0,
    CLEAR_KERNEL_SIMT = 1,
    CLEAR_KERNEL_TCGEN05 = 2,
    CLEAR_KERNEL_TCGEN05_WS = 3
} clear_kernel;

typedef struct clear_plan clear_plan_t; /* opaque */

typedef struct clear_plan_info {
    int32_t B, H, grid_h, grid_w, n_text, head_dim;
    int32_t dtype;             /* clear_dtype                                                       */
    int32_t kernel;            /* clear_kernel actually selected (never AUTO)                       */
    int32_t radius_sq_ceil;    /* integer threshold: a pair is allowed when dx^2 + dy^2 < this      */
    int32_t tile_h, tile_w;    /* 2-D query / key patch of the tensor-core kernel (0 for SIMT)      */
    int32_t n_work_items;      /* work items per (batch, head)                                      */
    int32_t n_text_splits;     /* key ranges each text-query tile is split into                     */
    int32_t max_item_tiles;    /* longest key-tile list of any work item                            */
    int64_t sum_mask;          /* sum(M) of Eq. 3 for one (batch, head): allowed (query, key) pairs */
    int64_t executed_pairs;    /* (query, key) pairs the kernel's tiles cover, one (batch, head)    */
    int64_t workspace_bytes;   /* device scratch owned by the plan                                  */
    double flops;              /* 4 * sum_mask * head_dim * H * B  (Fig. 2 caption: 4 * sum(M) * c) */
} clear_plan_info_t;

/* ---- schedule tables (read-only views for inspection and tests) --------------------------- */

/* One key/value tile of 128 keys that a work item visits. */
typedef struct clear_kv_tile {
    int32_t x;       /* image patch: grid column of its first key (may be negative or reach past  */
    int32_t y;       /*   the grid: such keys are masked); linear tile: x = first token, y = 0    */
    int32_t flags;   /* CLEAR_TILE_* bits                                                         */
    int32_t n_valid; /* linear tile: keys [0, n_valid) of the tile exist / are allowed            */
} clear_kv_tile_t;

enum {
    CLEAR_TILE_LINEAR = 1, /* 128 consecutive tokens of the [text; image] sequence, else a 2-D patch */
    CLEAR_TILE_MASKED = 2  /* some (query, key) pair of the tile is not allowed: apply Eq. 3 / n_valid */
};

/* One unit of work of the tensor-core kernel: 128 queries against a list of key tiles. */
typedef struct clear_work_item {
    int32_t kind;         /* 0 = 2-D patch of image queries, 1 = 128 consecutive text queries      */
    int32_t qx, qy;       /* image: grid column / row of the patch origin; text: qx = first token  */
    int32_t n_rows;       /* queries of the tile that exist (text: min(128, n_text - qx))          */
    int32_t tile_begin;   /* first entry of its list in the key-tile table                         */
    int32_t tile_count;   /* length of the list (>= 1)                                             */
    int32_t partial_slot; /* -1: writes final outputs; else index of its split-KV partial result   */
    int32_t reserved;
} clear_work_item_t;

/* ---- schedule tables of the TCGEN05_WS kernel ------------------------------------------------ */

enum {
    CLEAR_STEP_USE0 = 1,    /* query tile 0 of the pair visits its key tile in this step             */
    CLEAR_STEP_USE1 = 2,    /* query tile 1 of the pair visits its key tile in this step             */
    CLEAR_STEP_SHARED = 4,  /* both visit the SAME key tile (x0, y0): it is staged once             */
    CLEAR_STEP_LINEAR = 8,  /* key tiles of this step are 128 consecutive tokens, else 2-D patches  */
    CLEAR_STEP_MASKED0 = 16, /* tile 0 must apply Eq. 3 / n_valid0 to its key tile                  */
    CLEAR_STEP_MASKED1 = 32, /* tile 1 likewise                                                     */
    CLEAR_STEP_CLIP0 = 64,   /* tile 0's 2-D key patch reaches past the grid border: such keys do not exist */
    CLEAR_STEP_CLIP1 = 128   /* tile 1's likewise                                                    */
};

/* One step of a pair item: each query tile of the pair multiplies against one key tile. */
typedef struct clear_pair_step {
    int32_t x0, y0;     /* key tile of query tile 0 (and of tile 1 when SHARED); as clear_kv_tile_t */
    int32_t x1, y1;     /* key tile of query tile 1 when not SHARED                                 */
    int32_t flags;      /* CLEAR_STEP_* bits                                                        */
    int32_t n_valid0;   /* linear tiles: keys [0, n_valid) of the tile exist / are allowed; 2-D patches: */
    int32_t n_valid1;   /*   index of the tile pair's entry in the mask table, or -1 if it has none      */
    int32_t load_base;  /* where this step's tiles sit in the item's staging order, which runs, for every
                           step in turn, its K tiles and then its V tiles.  Low 16 bits: position of the
                           step's first K tile; high 16 bits: position of its first V tile (a step with two
                           distinct key tiles takes two consecutive positions each time, tile 0's first). */
} clear_pair_step_t;

/* One unit of work of the TCGEN05_WS kernel: two 128-query tiles walking one step list. */
typedef struct clear_pair_item {
    int32_t kind;          /* 0 = two vertically adjacent 8 x 16 image patches, 1 = two text tiles   */
    int32_t n_sides;       /* 2, or 1 when the second tile does not exist                            */
    int32_t qx;            /* image: grid column of both patches; text: first token of tile 0        */
    int32_t qy0, qy1;      /* image: grid row of patch 0 / patch 1; text: unused (tile 1 = qx + 128) */
    int32_t n_rows0, n_rows1; /* queries of each tile that exist                                     */
    int32_t step_begin;    /* first entry of its list in the step table                              */
    int32_t step_count;    /* length of the list (>= 1)                                              */
    int32_t n_loads;       /* key and value tiles its steps stage in total                           */
    int32_t partial_slot0; /* -1: tile 0 writes final outputs; else its split-KV partial-result slot */
    int32_t partial_slot1;
} clear_pair_item_t;

/* Eq. 1 under the mask of Eq. 3 for bf16 tensors, fp32 accumulation, bf16 output.
 * A plan for the shape is looked up in (or added to) a process-wide cache, so the first call for
 * a shape allocates and copies small tables; later calls only launch kernels.  The cache keeps the
 * 16 most recently used plans (environment variable CLEAR_CACHE_MAX_PLANS); making room for a new
 * shape synchronises the device.
 * Streams and threads: any.  Calls for one shape share one plan (work queue, status words, split-KV
 * workspace), so the library orders them on the device: a call made on another stream than the call
 * before it for that shape first waits there for that call's kernels (cudaStreamWaitEvent, no host
 * wait).  Calls for different shapes, or on different devices, do not wait for each other.
 * A kernel whose bounded wait expired is found by clear_cache_check, not here.
 * Errors: INVALID_ARG (B, H, grid_h, grid_w, head_dim <= 0; n_text < 0; radius <= 0 or
 * non-finite; scale non-finite; null tensor), MISALIGNED, UNSUPPORTED (head_dim > 256), CUDA. */
int clear_attn_fwd(const void *q, const void *k, const void *v, void *out, int B, int H, int grid_h,
                   int grid_w, int n_text, int head_dim, float radius, float scale, void *stream);

/* The same operator for fp32 tensors on the fp32 CUDA-core kernel (fp32 in, fp32 accumulate,
 * fp32 out; Eq. 1 and Eq. 3 as above).  Same errors. */
int clear_attn_fwd_f32(const void *q, const void *k, const void *v, void *out, int B, int H,
                       int grid_h, int grid_w, int n_text, int head_dim, float radius, float scale,
                       void *stream);

/* Backward pass of the operator for fp32 tensors (the distillation losses of Sec. 3.3, Eq. 4-6, reach the
 * attention parameters through it): given the upstream gradient d_out of the output of clear_attn_fwd_f32,
 *     p_ij  = softmax_j(scale q_i . k_j) over the keys Eq. 3 allows query i (Eq. 1),
 *     dS_ij = p_ij (d_out_i . v_j - sum_j' p_ij' d_out_i . v_j'),
 *     dq_i = scale sum_j dS_ij k_j,   dk_j = scale sum_i dS_ij q_i,   dv_j = sum_i p_ij d_out_i.
 * All seven tensors are device pointers, [B, H, N, head_dim] contiguous fp32, 16-byte aligned; q, k, v,
 * d_out are read, dq, dk, dv fully written.  Two CUDA-core kernels: one warp per query (row statistics, dq), then
 * one warp per key (dk, dv; the mask is symmetric, so the queries that see a key are the tokens that key's own
 * query sees): every output element has one writer and a fixed order of summation, so results repeat bit for
 * bit.  The first call for a shape allocates 12 bytes per token and (b, h) for the row statistics; calls for one
 * shape are ordered on the device like those of clear_attn_fwd.  Nothing but `stream` is synchronised.  Meant for
 * small problems (four dot products per allowed pair on the CUDA cores).
 * Errors: INVALID_ARG, MISALIGNED, UNSUPPORTED (head_dim > 256), CUDA. */
int clear_attn_bwd_f32(const void *q, const void *k, const void *v, const void *d_out, void *dq, void *dk,
                       void *dv, int B, int H, int grid_h, int grid_w, int n_text, int head_dim, float radius,
                       float scale, void *stream);

/* The same backward pass for bf16 tensors (all seven; 16-byte aligned): fp32 arithmetic and statistics as above,
 * gradients rounded to bf16 (nearest even) when stored.  Same kernels, errors and stream rules. */
int clear_attn_bwd_bf16(const void *q, const void *k, const void *v, const void *d_out, void *dq, void *dk,
                        void *dv, int B, int H, int grid_h, int grid_w, int n_text, int head_dim, float radius,
                        float scale, void *stream);

/* What the model does to Q and K between their projections and the attention call, in one pass over memory:
 * RMS normalisation over the head's channels, rotary position embedding on the two axes of the feature map
 * (Sec. 3.1: the model perceives spatial relations through it, by the relative distances on the two axes), with
 * the NTK factor on the rotary base that Sec. 4.3 raises from 1 to 10 beyond the training resolution, and a
 * constant factor on Q (pass clear_log_scale_factor() for the log-scale attention factor of the same recipe, or
 * leave it at 1 and multiply `scale` of the attention call instead).  For every (b, h) and token n with
 * position (0, 0, 0) for text tokens and (0, y, x) for image token p = y * grid_w + x:
 *     z   = x / sqrt(mean_c(x_c^2) + eps) * gain                                  (x = the row q[b,h,n,:] or k[b,h,n,:])
 *     the head's channels form three groups of axis0_dim, axis1_dim, axis2_dim channels (in this order); in
 *     group a of `dim` channels the pair (2j, 2j+1) turns by the angle position[a] * w_j,
 *     w_j = base^(-2j/dim), base = theta * ntk_factor^(dim/(dim-2)) (base = theta when dim = 2):
 *     out_2j = z_2j cos - z_2j+1 sin,   out_2j+1 = z_2j sin + z_2j+1 cos;   q_out is further multiplied by q_factor.
 * q_in, k_in, q_out, k_out: device pointers, [B, H, N, head_dim] contiguous, N = n_text + grid_h * grid_w,
 * bf16 (dtype CLEAR_BF16) or fp32 (CLEAR_F32), 16-byte aligned; arithmetic in fp32, frequencies from fp64 on
 * the host; an output may be the very same pointer as its input (in place), any other overlap is not allowed.
 * gain_q, gain_k: device pointers to head_dim fp32 values, or NULL for a gain of one.  The caller owns all
 * buffers.  One kernel launch on `stream` (a cudaStream_t), no allocation, no host synchronisation.
 * Errors: INVALID_ARG (sizes <= 0, n_text < 0, an odd or negative group size, groups not summing to head_dim,
 * theta or ntk_factor <= 0 or non-finite, eps < 0, a non-finite value, a null tensor, unknown dtype),
 * UNSUPPORTED (head_dim other than 64 or 128), MISALIGNED, CUDA. */
int clear_qk_norm_rope(const void *q_in, const void *k_in, void *q_out, void *k_out, const float *gain_q,
                       const float *gain_k, int B, int H, int grid_h, int grid_w, int n_text, int head_dim, int dtype,
                       int axis0_dim, int axis1_dim, int axis2_dim, float theta, float ntk_factor, float eps,
                       float q_factor, void *stream);

/* sqrt(log n_tokens / log n_train_tokens): the factor on the logits that keeps the entropy of the attention
 * of a longer sequence where it was at the training length (the log-scale attention factor Sec. 4.3 applies
 * beyond the training resolution).  Host arithmetic only; 1 when either count is below 2. */
float clear_log_scale_factor(long long n_tokens, long long n_train_tokens);

/* The backward pass for bf16 tensors on the tensor cores (head_dim 64 or 128, scale > 0): same arguments and
 * results as clear_attn_bwd_bf16, computed with tcgen05 MMAs over the forward pass's tile schedule -- a launch in
 * which every 128-query tile meets its key tiles (row statistics and delta = dO . O in a first sweep, dQ in a second)
 * and a launch in which every 128-key tile meets the query tiles that see it (dK, dV; Eq. 3's mask is symmetric, so
 * these are the same lists).  P and dS enter the MMAs rounded to bf16, as P does in the forward pass: gradients
 * agree with the exact ones to about 1e-2 of the largest gradient of the tensor.  One writer per element: results
 * repeat bit for bit.  The first call for a shape allocates its schedule tables and 16 bytes per token and (b, h).
 * Errors: INVALID_ARG, MISALIGNED, UNSUPPORTED (other head sizes, scale <= 0), CUDA; a kernel whose bounded wait
 * expired is found by clear_cache_check. */
int clear_attn_bwd_bf16_tc(const void *q, const void *k, const void *v, const void *d_out, void *dq, void *dk,
                           void *dv, int B, int H, int grid_h, int grid_w, int n_text, int head_dim, float radius,
                           float scale, void *stream);

/* Window of an image query (text tokens are always allowed, as in Eq. 3). */
enum {
    CLEAR_MASK_DISC = 0,   /* Eq. 3: dx^2 + dy^2 < r^2, the paper's circular window                              */
    CLEAR_MASK_SQUARE = 1, /* max(|dx|, |dy|) < r: the square sliding window of Neighborhood Attention, which
                              Sec. 3.2 sets the circular one against (the circle costs about pi / 4 of it)      */
    CLEAR_MASK_WINDOWS = 2, /* both tokens in the same w x w window of the grid, the window grid shifted by s
                               (floor((x + s) / w) and floor((y + s) / w) agree; no wrap-around): the Swin baseline
                               of the appendix (w = 16, s = 8 in every other layer)                              */
    CLEAR_MASK_STRIDED = 3  /* (xj - xi) mod r == l mod r and (yj - yi) mod r == (l div r) mod r, non-negative
                               remainders: the strided baseline of the appendix at layer l                      */
};

/* Build the schedule for one shape on the current device (Eq. 3 turned into integer geometry):
 * the threshold ceil(radius^2), for every 2-D query patch the list of key patches that meet its
 * radius-r dilation (with a flag telling whether the exact mask is needed) plus the text tiles,
 * text-query tiles split over key ranges, and an order of the work items that evens out the load.
 * The plan owns its device tables and workspace; the caller owns the handle and must destroy it
 * when no call using it is still running.  `*plan` is written only on CLEAR_OK.
 * Errors: INVALID_ARG, UNSUPPORTED (kernel/dtype/head_dim combination), CUDA, NO_MEMORY. */
int clear_plan_create(clear_plan_t **plan, int B, int H, int grid_h, int grid_w, int n_text,
                      int head_dim, float radius, int dtype, int kernel);

/* clear_plan_create with the window kind chosen (CLEAR_MASK_*); every kernel serves both kinds, the schedule
 * and its mask table are built for the window given.  Errors as clear_plan_create, INVALID_ARG for an unknown kind. */
int clear_plan_create_ex(clear_plan_t **plan, int B, int H, int grid_h, int grid_w, int n_text,
                         int head_dim, float radius, int dtype, int kernel, int mask_kind, int host_only);

/* ---- Row-band parallel form (Sec. 3.4) --------------------------------------------------------------------
 * The H x W feature map is cut into bands of rows, one per GPU; every GPU also holds the text tokens.  An image
 * query sees keys at most `reach` rows away (Eq. 3), so a GPU needs, besides its band, `halo_lo` rows above and
 * `halo_hi` rows below it, which its neighbours send ("communication only in the boundary areas").  A GPU's LOCAL
 * tensors are [B, H, n_text + local_rows * grid_w, head_dim] with local_rows = halo_lo + (y1 - y0) + halo_hi: the
 * text tokens, then the rows y0 - halo_lo .. y1 + halo_hi - 1 of the grid, row-major; the band sits at local rows
 * [halo_lo, halo_lo + y1 - y0).  Q and the output need only hold valid data in the text and band rows.
 *   image queries of the band: a CLEAR_PART_BAND_IMAGE plan over the local grid, run by clear_attn_fwd_planned:
 *       exactly the rows of the single-GPU result (the halo holds every key such a query can see, and the local
 *       grid's border is the true border wherever a window reaches it);
 *   text queries: they see every key, so each GPU computes them over ITS keys only -- a CLEAR_PART_BAND_TEXT plan,
 *       run by clear_attn_text_partial, leaves per text row the un-normalised output with the row's maximum and
 *       sum -- and clear_text_merge combines the records of all GPUs: exactly (the merge of a split softmax, Eq. 1
 *       unchanged), or by the patch-wise average of Eq. 7.  Either way one record of head_dim + 2 floats per
 *       text row and (b, h) is all that travels.
 * The exchange itself (halo rows to the neighbours, records to everyone) is the caller's: the Python package does
 * it with torch.distributed send/recv and all-gather into local buffers. */
enum {
    CLEAR_PART_ALL = 0,         /* an ordinary plan: the whole operator on one GPU                                  */
    CLEAR_PART_BAND_IMAGE = 1,  /* the image queries of the band's rows                                             */
    CLEAR_PART_BAND_TEXT = 2    /* the text queries over this GPU's keys, as records for clear_text_merge          */
};
enum {
    CLEAR_TEXT_MERGE_EXACT = 0,   /* sum_p w_p O_p / sum_p w_p l_p, w_p = 2^(m_p - max m): the exact text rows       */
    CLEAR_TEXT_MERGE_AVERAGE = 1  /* Eq. 7: (1 / n_parts) sum_p O_p / l_p                                            */
};

/* Rows [*y0, *y1) of band `band` when grid_h rows are cut into n_bands bands as evenly as possible (the first
 * grid_h % n_bands bands are one row taller), and the halo rows the band needs above and below: the window's
 * reach (largest |dy| with a visible key: dy^2 < ceil(radius^2) for the disc, ceil(radius) - 1 for the square),
 * clipped at the grid's border.  Host arithmetic only; any output pointer may be NULL.
 * Errors: INVALID_ARG (n_bands < 1 or > grid_h, band out of range, radius <= 0 or non-finite, unknown kind). */
int clear_band_geometry(int grid_h, float radius, int mask_kind, int n_bands, int band, int32_t *y0, int32_t *y1,
                        int32_t *halo_lo, int32_t *halo_hi);

/* Plan of one part of a band (bf16, head_dim 64 or 128, the warp-specialised tensor-core kernel) over the LOCAL
 * grid of local_rows x grid_w; the band is local rows [q_row_begin, q_row_end).
 *   CLEAR_PART_BAND_IMAGE: work items for the 8 x 16 query patches that hold rows of the band.  Output rows of those
 *       patches that lie outside the band are written too (with values the caller must ignore); text rows and all
 *       other rows of `out` are left alone.
 *   CLEAR_PART_BAND_TEXT: work items for the text queries over the image tokens of the band's own rows, and over
 *       the text tokens too iff text_keys != 0.  For the exact merge exactly one GPU counts the text keys
 *       (text_keys = 1 on band 0, 0 elsewhere); for Eq. 7 every GPU does.  Needs n_text > 0.
 * clear_plan_info reports the allowed pairs and flops of the part.  Ownership, host_only and errors as
 * clear_plan_create_ex; INVALID_ARG also for an empty or out-of-range band, an unknown part. */
int clear_plan_create_band(clear_plan_t **plan, int B, int H, int local_rows, int grid_w, int n_text, int head_dim,
                           float radius, int mask_kind, int part, int q_row_begin, int q_row_end, int text_keys,
                           int host_only);

/* Text queries over this GPU's keys (a CLEAR_PART_BAND_TEXT plan; q, k, v local tensors as above).  `records`:
 * device pointer, [B * H][n_text][head_dim + 2] fp32, 16-byte aligned, fully written: head_dim values of
 * sum_j 2^(s_ij - m_i) v_j over the keys j this GPU counts (s = scale * log2(e) * q_i . k_j), then m_i, then
 * l_i = sum_j 2^(s_ij - m_i).  Streams, ordering and errors as clear_attn_fwd_planned; PLAN_MISMATCH for any
 * other kind of plan (and clear_attn_fwd_planned returns PLAN_MISMATCH for this kind). */
int clear_attn_text_partial(const clear_plan_t *plan, const void *q, const void *k, const void *v, float *records,
                            float scale, void *stream);

/* Merge of the records of all bands into the text rows: `records` is [n_parts][B * H][n_text][head_dim + 2] fp32
 * on the device (the parts' records one after the other, e.g. as an all-gather leaves them), `out` a bf16
 * [B, H, out_tokens, head_dim] tensor whose first n_text rows per (b, h) are written (16-byte aligned).  mode:
 * CLEAR_TEXT_MERGE_EXACT or CLEAR_TEXT_MERGE_AVERAGE (Eq. 7).  One small kernel on `stream`, no allocation.
 * Errors: INVALID_ARG, UNSUPPORTED (head_dim other than 64 or 128, B * H > 65535), MISALIGNED, CUDA. */
int clear_text_merge(const float *records, int n_parts, int B, int H, int n_text, int head_dim, int mode, void *out,
                     long long out_tokens, void *stream);

/* Plan for any mask kind (bf16 or fp32).  mask_size: r of CLEAR_MASK_DISC / CLEAR_MASK_SQUARE, the window size w
 * of CLEAR_MASK_WINDOWS, the stride r of CLEAR_MASK_STRIDED (the last two whole numbers >= 1); mask_param: the shift
 * s of the window grid, the layer index l of the strided mask, 0 for the other kinds.  The windows and the strided
 * mask are no windows around the query (membership depends on absolute position, or on a residue class), so the
 * tensor-core kernels' tables do not carry them: these two kinds run on the fp32-accumulating CUDA-core kernel,
 * which walks the allowed keys of each query row by row (the kernel is chosen by the library).  They serve to
 * reproduce the appendix's comparison masks; clear_plan_info reports their sum(M) and flops.
 * Run the plan with clear_attn_fwd_planned.  Errors as clear_plan_create_ex; INVALID_ARG for a fractional window
 * size or stride, a negative shift or layer, a non-zero mask_param with the disc or the square. */
int clear_plan_create_mask(clear_plan_t **plan, int B, int H, int grid_h, int grid_w, int n_text, int head_dim, int dtype,
                           int mask_kind, float mask_size, int mask_param, int host_only);

/* The same schedule built on the host only: no CUDA call is made and no device is needed.  The
 * plan can be inspected (clear_plan_info, clear_plan_tables) and destroyed, not executed
 * (forward calls return PLAN_MISMATCH).  Errors: INVALID_ARG, UNSUPPORTED, NO_MEMORY. */
int clear_plan_create_host(clear_plan_t **plan, int B, int H, int grid_h, int grid_w, int n_text,
                           int head_dim, float radius, int dtype, int kernel);

/* Borrow the host copies of the schedule tables (valid until the plan is destroyed).  Any output
 * pointer may be NULL.  `half_width[dy]`, dy in [0, n_half_width), is the largest |dx| allowed at
 * row offset dy.  For SIMT plans the item and tile tables are empty.  Errors: INVALID_ARG. */
int clear_plan_tables(const clear_plan_t *plan, const clear_work_item_t **items, int32_t *n_items,
                      const clear_kv_tile_t **tiles, int32_t *n_tiles, const int32_t **half_width,
                      int32_t *n_half_width);

/* The same for a TCGEN05_WS plan: its pair items (text items first, then image items, longest step
 * lists first) and their steps.  Empty for other plans.  Errors: INVALID_ARG. */
int clear_plan_pair_tables(const clear_plan_t *plan, const clear_pair_item_t **items, int32_t *n_items,
                           const clear_pair_step_t **steps, int32_t *n_steps);

/* Mask table of a TCGEN05_WS plan: Eq. 3 evaluated once per relative position of a key patch to a query
 * patch (the mask depends only on that offset).  Entry e is 128 rows (queries of the patch, row-major)
 * of four 32-bit words; bit j of word w tells whether key 32 w + j of the patch (row-major) lies within
 * the radius of that query.  Grid clipping is not part of it (CLEAR_STEP_CLIP*).  Errors: INVALID_ARG. */
int clear_plan_mask_table(const clear_plan_t *plan, const uint32_t **words, int32_t *n_entries);

/* Forward pass with an explicit plan.  Tensor dtype is the plan's.  Calls on one plan share its
 * workspace and work queue; the library orders them on the device as described at clear_attn_fwd, so
 * they may be made on any streams (two plans of one shape run side by side).
 * Errors: INVALID_ARG, MISALIGNED, PLAN_MISMATCH (current device differs from the plan's),
 * UNSUPPORTED (tensor-core plan called with scale <= 0), CUDA. */
int clear_attn_fwd_planned(const clear_plan_t *plan, const void *q, const void *k, const void *v,
                           void *out, float scale, void *stream);

/* Forward pass on HOST tensors (same layout and dtype as the plan's): copies q, k, v to staging
 * buffers the plan owns (allocated on first use), runs the kernels, copies `out` back, and returns
 * after synchronising `stream`.  A problem of more than one chunk (a chunk = whole (b, h) slices of
 * at least 96 MiB per tensor, at most 16 chunks; the environment variable CLEAR_HOST_CHUNK_BYTES,
 * read at the plan's first call, changes the size) runs as a three-stage pipeline: the copies in,
 * the kernels (on `stream`, with a plan per chunk size that this plan owns) and the copies out each
 * work on a different chunk, on two extra streams the plan creates, so both PCIe directions and
 * the GPU are busy at once; results are identical to the one-piece run.  Only pinned host memory
 * lets the stages overlap.  Eq. 1 and Eq. 3 hold per (b, h) slice, so cutting that axis changes
 * nothing.  Errors as clear_attn_fwd_planned, plus NO_MEMORY and DEVICE_TIMEOUT. */
int clear_attn_fwd_host(clear_plan_t *plan, const void *q_host, const void *k_host,
                        const void *v_host, void *out_host, float scale, void *stream);

/* Fixed capacities of clear_attn_fwd_static (one static device array of about 33.3 MiB in total). */
#define CLEAR_STATIC_SCRATCH_BYTES (32u << 20) /* split-KV partial results of the text-query rows      */
#define CLEAR_STATIC_MAX_ITEMS 8192            /* work items per (batch, head)                          */
#define CLEAR_STATIC_MAX_TILES 65536           /* key-tile list entries per (batch, head)               */
#define CLEAR_STATIC_MAX_HALF_WIDTH 1024       /* rows an image query can reach upwards, plus one       */

/* bf16 forward pass on the tensor-core kernel that never allocates device memory.  (The paper has no
 * counterpart: this is an interface variant, not a step of the method.)
 *
 * Who needs it: code that may not call cudaMalloc at the point where attention runs -- a host running
 * under a fixed, pre-partitioned memory budget, a plug-in whose embedding framework owns every device
 * byte, or a process that has already handed all free memory to a caching allocator, where a driver
 * allocation would fail or stall the other streams.  The planned entry points allocate schedule tables
 * and a split-KV workspace per plan; this one keeps them in one file-scope device array inside the
 * library image, so every GPU that loads the library holds those ~33.3 MiB until the process exits.
 *
 * Same tensors, layout and mathematics as clear_attn_fwd; it runs the one-tile-per-block tensor-core
 * kernel, so its results equal those of a CLEAR_KERNEL_TCGEN05 plan bit for bit and those of
 * clear_attn_fwd (another kernel) within the bf16 tolerance.  head_dim must be 64 or 128 and scale > 0.
 * It calls no cudaMalloc / cudaFree and no allocating library routine; it does enqueue one 4-byte memset
 * on `stream` and, when the shape differs from the previous call's, three small table copies from
 * ordinary host memory (such a copy can make the host wait for the stream).
 * - The first call on a device looks up the array's device address (set-up); make that call with the
 *   device current and before starting any stream capture.
 * - Shapes whose tables or partial results exceed the CLEAR_STATIC_* capacities are rejected with
 *   CLEAR_ERR_TOO_LARGE (the 2048px FLUX shape fits; the 4096px and 8K shapes do not).
 * - All calls on a device share the array, which keeps the last call's contents; the call re-uploads the
 *   tables when the shape changes and clears the status word every time.  Two calls that overlap on the
 *   GPU (different streams without ordering) race on it: order them.
 * - Device-side wait expiries are not reported by this entry point.
 * Errors: INVALID_ARG, UNSUPPORTED, MISALIGNED, TOO_LARGE, NO_MEMORY (host), CUDA. */
int clear_attn_fwd_static(const void *q, const void *k, const void *v, void *out, int B, int H, int grid_h,
                          int grid_w, int n_text, int head_dim, float radius, float scale, void *stream);

/* Fill `info` from the plan (host only, no CUDA call).  Errors: INVALID_ARG. */
int clear_plan_info(const clear_plan_t *plan, clear_plan_info_t *info);

/* Synchronise `stream`, then read and clear the plan's device status words.  Returns
 * CLEAR_ERR_DEVICE_TIMEOUT if any kernel launched with this plan gave up on a bounded wait since
 * the last check, CLEAR_OK otherwise.  A launch whose blocks gave up writes nothing more (its outputs
 * are incomplete); later launches of the plan run normally.  Errors: INVALID_ARG, CUDA. */
int clear_plan_check(clear_plan_t *plan, void *stream);

/* Give back the staging buffers (four tensors' worth of device memory) and the copy pipeline that
 * clear_attn_fwd_host built for this plan; the next such call builds them again.  Synchronises the
 * plan's device.  Errors: INVALID_ARG, CUDA. */
int clear_plan_trim(clear_plan_t *plan);

/* Free the plan's device memory and the handle.  NULL is accepted.  Errors: CUDA. */
int clear_plan_destroy(clear_plan_t *plan);

/* clear_plan_check for every plan the unplanned entry points (clear_attn_fwd, clear_attn_fwd_f32)
 * have cached for the current device: waits for their last launches and for `stream`, returns
 * CLEAR_ERR_DEVICE_TIMEOUT if a kernel of any of them gave up on a bounded wait since the last check
 * (clear_last_device_status names the wait), and clears that record.  Errors: CUDA. */
int clear_cache_check(void *stream);

/* Drop every plan the unplanned entry points cached (synchronises the device first; no call of those
 * entry points runs at the same time: they hold the cache's lock while they launch). */
int clear_cache_clear(void);

/* Static, human-readable name of a status code. */
const char *clear_status_string(int status);

/* cudaError_t value of the most recent CUDA failure seen by the calling thread (0 if none). */
int clear_last_cuda_error(void);

/* Diagnostic detail of the most recent CLEAR_ERR_DEVICE_TIMEOUT returned to the calling thread by
 * clear_plan_check or clear_attn_fwd_host: the non-zero word the kernel left in the plan's status
 * slot, which names the wait that expired (a kernel-internal code, stable only within one build).
 * 0 if there was none. */
int clear_last_device_status(void);

#ifdef __cplusplus
}
#endif
#endif /* CLEAR_ATTN_H_ */
