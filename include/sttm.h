/*
 * sttm.h - C ABI of the STTM token-merging library for NVIDIA B200 (sm_100a).
 *
 * STTM ("Multi-Granular Spatio-Temporal Token Merging", Section 3) reduces a video's
 * visual tokens Z_V [T, H, W, D] to a packed multi-granular set Z_ST [N_ST, D]:
 *   1. spatial stage (Section 3.2): per frame, 2x2 average pooling builds a quadtree up
 *      to a coarsest map of at most lv1 x lv1 nodes; a coarse-to-fine search keeps the
 *      coarsest node whose children all have cosine similarity > tau_s to it;
 *   2. temporal stage (Section 3.3): every kept node of frame t is compared with the
 *      kept nodes of frame t-1 that overlap its region and is linked to one whose
 *      similarity is > tau_t (priority to the top-left one); links are followed to the
 *      common root in the earliest frame and all nodes of a chain are averaged into it;
 *   3. reordering (Section 3.4): surviving tokens are ordered by frame, then by their
 *      top-left coordinate (row-major), and receive position ids.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer owned by the caller unless its comment says
 *     "host".  The library never frees or keeps caller memory.
 *   - Except sttm_merge / sttm_merge_host (which keep one cached workspace per device)
 *     the library allocates nothing: the caller provides `ws` of at least
 *     sttm_workspace_bytes(params) bytes, 256-byte aligned.
 *   - Calls are asynchronous on `stream` and do not synchronise (sttm_merge_host does).
 *   - Host-detectable errors are returned with no work enqueued.  Conditions found on
 *     the device are OR-ed as (1 << status) bits into *device_status; kernels never trap:
 *       1 << STTM_ERR_CAPACITY       more rows than out_capacity_rows (the rows that fit are valid),
 *       1 << STTM_ERR_NOT_CONVERGED  the root search hit its round limit,
 *       1 << STTM_ERR_TIMEOUT        a wait between the stages of a pipelined kernel (on a
 *                                    shared-memory barrier) was given up after 2 seconds; the
 *                                    kernel then ended early and its outputs are not valid.
 *   - The library keeps per-device tables but no per-call global state; calls on different
 *     host threads are independent as long as they use different workspaces and streams.
 *     The benchmark knobs (sttm_set_tuning, sttm_set_ring_split, sttm_set_stage_events) are
 *     process-wide or per-thread test hooks and are not meant to be changed while calls run.
 *   - Layout: feats is [B, T, H, W, D] contiguous, D fastest; D must be a multiple of 4
 *     and the base pointer 16-byte aligned.  A token's cell id inside its video is
 *     c = t*H*W + y*W + x.  A quadtree node is named by the cell id of its top-left
 *     (anchor) cell.  Quadtrees of up to 3 levels (coarsest node at most 4 cells wide) run on
 *     the tuned kernels; deeper ones (up to 8 levels) only through sttm_merge_ex / sttm_merge /
 *     sttm_merge_host, on plain general kernels (same results, a row's members added in index
 *     order, several times slower); the stage calls and the budget mode report them as
 *     STTM_ERR_UNSUPPORTED.  On every path the output bits do not depend on scheduling.
 */
#ifndef STTM_H
#define STTM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    STTM_OK = 0,
    STTM_ERR_ARG = 1,            /* null pointer, non-positive size, misalignment      */
    STTM_ERR_UNSUPPORTED = 2,    /* shape outside what the kernels cover                */
    STTM_ERR_WORKSPACE = 3,      /* ws_bytes smaller than sttm_workspace_bytes()        */
    STTM_ERR_CAPACITY = 4,       /* more output rows than out_capacity_rows (device)    */
    STTM_ERR_NOT_CONVERGED = 5,  /* root search hit its round limit (device)            */
    STTM_ERR_CUDA = 6,           /* a CUDA runtime call failed                          */
    STTM_ERR_TIMEOUT = 7         /* a bounded wait inside a kernel ran out (device)     */
} sttm_status;

typedef enum { STTM_BF16 = 0, STTM_F32 = 1 } sttm_dtype;
/* Section 3.4: keep the surviving token's original position, or renumber 0..N_ST-1. */
typedef enum { STTM_POS_SURVIVED = 0, STTM_POS_REASSIGNED = 1 } sttm_pos_mode;
/* Averaging weights inside a chain (the paper does not fix them): one per node, or the
 * number of grid cells the node covers. */
typedef enum { STTM_W_NODE = 0, STTM_W_AREA = 1 } sttm_weight_mode;
/* Which of several overlapping nodes of frame t-1 above tau_t a node is linked to (Section 3.3):
 * the top-left one (the paper's choice), or the most similar one (the "optimal" destination of
 * the paper's ablation; equal similarities: the top-left of them). */
typedef enum { STTM_MATCH_TOPLEFT = 0, STTM_MATCH_BEST = 1 } sttm_match_mode;

typedef struct sttm_params {
    int B, T, H, W, D;            /* videos, frames, grid, channels                      */
    sttm_dtype in_dtype;          /* dtype of feats                                       */
    sttm_dtype out_dtype;         /* dtype of out_feats                                   */
    int lv1;                      /* coarsest map is at most lv1 x lv1 (paper: 4, or 2)   */
    float tau_s, tau_t;           /* thresholds, used when the per-video arrays are NULL  */
    const float* tau_s_per_video; /* host, [B] or NULL                                    */
    const float* tau_t_per_video; /* host, [B] or NULL                                    */
    sttm_pos_mode pos;
    sttm_weight_mode wt;
    long long out_capacity_rows;  /* rows available in out_feats / out_pos (all videos)   */
    sttm_match_mode match;        /* destination rule of the temporal link                */
} sttm_params;

/* The lowest-numbered condition whose (1 << status) bit is set in a device status word, STTM_OK
 * for 0.  Host only. */
sttm_status sttm_status_from_bits(int32_t bits);

/* Fills *p with defaults: B=1, bf16 in and out, lv1=4, survived ids, node weights,
 * top-left destination, capacity B*T*H*W.  Host only. */
void sttm_default_params(sttm_params* p, int T, int H, int W, int D, float tau_s, float tau_t);

/* Bytes of device workspace the calls below need for these params (0 on bad params). */
size_t sttm_workspace_bytes(const sttm_params* p);

/* Number of parent-child similarities per frame, stored level by level (level 0 first,
 * each level row-major); 0 when the grid has a single level. Host only. */
int sttm_sims_per_frame(int H, int W, int lv1);

/*
 * Spatial stage alone (Section 3.2).
 *   cover_level  [B, T, H, W] int8   out: quadtree level (0 = single cell) of the kept
 *                                    node covering each cell
 *   frame_counts [B, T] int32        out: kept nodes per frame
 *   spatial_sims [B, T, sttm_sims_per_frame] float32, out, may be NULL:
 *                                    cos(node, its parent) of every non-root node
 */
sttm_status sttm_spatial(const void* feats, const sttm_params* p, void* ws, size_t ws_bytes,
                         int8_t* cover_level, int32_t* frame_counts, float* spatial_sims,
                         void* stream);

/*
 * Spatial stage alone, for callers that cannot give the library any device memory beyond
 * inputs and outputs.  (The paper has no counterpart: this is a deployment convenience.)
 * Who that is: code running where device allocation is off the table - a serving process whose
 * whole HBM has already been handed to a tensor pool, a latency-critical loop in which a
 * cudaMalloc (which may synchronise the device) must not happen, a plug-in that receives raw
 * pointers and owns no allocator.  Same computation and same outputs as sttm_spatial; the one
 * scratch buffer the stage needs (a squared norm per quadtree node) sits in a fixed array of
 * STTM_STATIC_SCRATCH_BYTES inside the library image, which every GPU that loads the library
 * keeps until the process ends.
 *   - Problems that need more scratch (B*T*columns*nodes-per-column*4 bytes, e.g. 1024 frames
 *     of a 13x13 grid need 1.4 MB) are refused with STTM_ERR_WORKSPACE and nothing runs.
 *   - No allocation, no free, on any path.  The first call on a device asks the runtime for the
 *     array's device address (with that device current); make that first call outside any
 *     stream capture.
 *   - All calls on a device share the array and it keeps what the last call left there.  Nothing
 *     stale is read (the norms are rewritten, the counts are zeroed first), but two calls whose
 *     kernels overlap on the GPU - different streams, different threads - race on it: serialise
 *     them.  sttm_temporal needs the norms in a caller workspace, so it does not pair with this.
 */
#define STTM_STATIC_SCRATCH_BYTES (4u << 20)
sttm_status sttm_spatial_static(const void* feats, const sttm_params* p, int8_t* cover_level,
                                int32_t* frame_counts, float* spatial_sims, void* stream);

/*
 * Temporal stage alone (Section 3.3), given the spatial stage's cover map.
 *   link [B, T*H*W] int32  out, per cell: anchor id of the node (frame t-1) that the
 *                          cell's covering node is linked to, or -1
 *   root [B, T*H*W] int32  out, per cell: anchor id of the chain's root
 *   temporal_sims [B, T*H*W] float32, out, may be NULL: cosine of each compared pair,
 *                          stored at the anchor cell of the finer node of the pair
 *                          (frame t's index), NaN elsewhere
 * sttm_spatial must have run on the same ws before (it leaves the node norms there).
 */
sttm_status sttm_temporal(const void* feats, const sttm_params* p, void* ws, size_t ws_bytes,
                          const int8_t* cover_level, int32_t* link, int32_t* root,
                          float* temporal_sims, int32_t* device_status, void* stream);

/*
 * The whole path (Sections 3.2-3.4) for B videos.
 *   out_feats   [out_capacity_rows, D] out_dtype  packed rows, videos back to back
 *   out_pos     [out_capacity_rows] int32         position id per row (cell id inside
 *                                                 its video, or 0..count-1)
 *   merge_map   [B, T*H*W] int32, may be NULL     per cell: row (inside its video) it
 *                                                 was merged into
 *   out_count   [B] int32                         rows per video
 *   out_offsets [B+1] int64, may be NULL          first row of each video
 *   device_status int32, may be NULL              OR of (1 << sttm_status) bits; must be
 *                                                 zeroed by the caller
 * Rows beyond out_capacity_rows are not written; out_count stays exact.
 */
sttm_status sttm_merge_ex(const void* feats, const sttm_params* p, void* ws, size_t ws_bytes,
                          void* out_feats, int32_t* out_pos, int32_t* merge_map,
                          int32_t* out_count, int64_t* out_offsets, int32_t* device_status,
                          void* stream);

/*
 * One bf16 video with default params (lv1 = 4, survived ids, node weights, bf16 output,
 * capacity T*H*W rows).  Uses a workspace cached per device, grown with cudaMalloc when a
 * larger problem arrives (so the first call on a device synchronises and allocates).
 * Conditions found on the device go to a status word kept with that workspace; it is cleared
 * by every sttm_merge call and read back by sttm_merge_status.
 */
sttm_status sttm_merge(const void* feats, int T, int H, int W, int D, float tau_s, float tau_t,
                       void* out_feats, int32_t* out_pos, int32_t* out_count, void* stream);

/*
 * Waits for `stream` and returns what the last sttm_merge call on the current device left in its
 * status word: STTM_OK, or the lowest-numbered condition whose bit is set (the whole word goes to
 * *host_bits when that is not NULL).  Host pointer; synchronises.
 */
sttm_status sttm_merge_status(int32_t* host_bits, void* stream);

/*
 * One video cut into segments of consecutive frames, one segment per GPU (Section 3.3: a chain
 * of temporal links may cross a cut).  The paper has no counterpart: it merges a video on one
 * device.  Each segment is merged by sttm_merge_ex (fp32 rows, merge map, SURVIVED ids) with
 * the last frame of the segment before it, the halo, as its frame 0; the halo alone (T = 1)
 * is merged too, which gives its kept nodes u in order, their features F(u) and weights w_u.
 * The first n_h rows of the segment's result are rooted in the halo (row b at node b) and
 * belong to an earlier segment.  A row is held as (mean m, weight W); a contribution (S, V)
 * turns it into (W m + S) / (W + V).  Segments are finished from the last to the first:
 * sttm_segment_fold takes in what the next segment sent, sttm_segment_emit makes what goes to
 * the previous one, sttm_segment_finish writes the owned rows.  All pointers are device
 * pointers; nothing is allocated; every call is asynchronous on stream.
 *
 * sttm_row_weights: W of every row of a finished sttm_merge_ex call (same params, same ws,
 *   which still holds that call's cover map): one per member node or, for STTM_W_AREA, the
 *   node's cells.  weights float32 [min(cells, out_capacity_rows)].
 * sttm_segment_fold: n = min(*n_dev, n_max) contributions keyed by anchors[i], the cell
 *   (y*W + x) of a kept node of this segment's last frame; map_last int32 [HW] is the merge
 *   map of that frame (local rows).  Adds s[i, :] to extra[row, :] and v[i] to extra_w[row]
 *   with fp32 atomics (extra, extra_w: [capacity_rows, D] and [capacity_rows], zero before the
 *   first call).  Entries with v[i] == 0 are skipped; an anchor outside the frame sets
 *   (1 << STTM_ERR_ARG), a row outside capacity (1 << STTM_ERR_CAPACITY) in *device_status.
 * sttm_segment_emit: for b < min(*n_h_dev, n_max): v_out[b] = W_b + extra_w[b] - w_u and
 *   s_out[b, :] = W_b m_b + extra[b, :] - w_u F(u), the halo node itself left out because the
 *   owner's row has it already.  feats/weights/extra/extra_w are the local rows, halo_feats
 *   [n_h, D] and halo_w [n_h] the rows and weights of the halo's own merge.
 * sttm_segment_finish: owned row r = local row r + n_h (n_h_dev NULL: no halo) with its
 *   contributions, as out_dtype; out_pos[r] = local id + pos_shift for STTM_POS_SURVIVED (pass
 *   (first owned frame - frames in front of it in the local input) * H * W), r + pos_shift for
 *   STTM_POS_REASSIGNED (pass the rows owned by earlier segments); *owned_count = count - n_h.
 *   feats, extra and out_feats 16-byte aligned, D a multiple of 4.
 */
sttm_status sttm_row_weights(const sttm_params* p, const void* ws, const int32_t* merge_map,
                             const int64_t* out_offsets, float* weights, void* stream);
sttm_status sttm_segment_fold(const int32_t* map_last, const int32_t* anchors, const float* v, const float* s,
                              const int32_t* n_dev, int n_max, int HW, int D, float* extra, float* extra_w,
                              long long capacity_rows, int32_t* device_status, void* stream);
sttm_status sttm_segment_emit(const float* feats, const float* weights, const float* extra, const float* extra_w,
                              const float* halo_feats, const float* halo_w, const int32_t* n_h_dev, int n_max, int D,
                              float* v_out, float* s_out, void* stream);
sttm_status sttm_segment_finish(const float* feats, const int32_t* pos, const float* weights, const float* extra,
                                const float* extra_w, const int32_t* count_dev, const int32_t* n_h_dev, int D,
                                long long capacity_rows, long long pos_shift, sttm_pos_mode pos_mode,
                                sttm_dtype out_dtype, void* out_feats, int32_t* out_pos, int32_t* owned_count,
                                void* stream);

/*
 * Same computation with HOST buffers: copies feats to the device, runs sttm_merge_ex,
 * copies the used rows back and synchronises.  All pointers are host pointers (pinned
 * memory makes the copies asynchronous and faster).  h_merge_map and h_out_offsets may
 * be NULL.  Device buffers are cached per device and grown on demand.
 */
sttm_status sttm_merge_host(const void* h_feats, const sttm_params* p,
                            void* h_out_feats, int32_t* h_out_pos, int32_t* h_merge_map,
                            int32_t* h_out_count, int64_t* h_out_offsets, int32_t* h_device_status);

/*
 * Budget mode (the adaptive thresholds the paper leaves to future work in its limitations): tau_s
 * as given in *p, tau_t chosen per video on the device so that the video keeps at most
 * budget_rows[v] rows.  With the cover maps fixed, a kept node is merged into the frame before iff
 * the largest cosine to its candidates exceeds tau_t, so the row count is nodes - #{best cosine >
 * tau_t}; the threshold returned is the middle of the gap between the k-th and the (k+1)-th largest
 * best cosine, k = nodes - budget (2.0 when the spatial stage alone meets the budget; -2.0, and
 * more rows than asked for, when even linking every node that has a candidate does not).  Equal
 * best cosines at the cut leave the count off by their number.  The features are streamed once
 * for all similarities (whose sums are kept), the decisions are taken twice (once without links to
 * collect the best cosines, once with the chosen thresholds), then the averages are formed: about
 * 1.4 times the cost of a call with given thresholds.  Only for quadtrees of up to three levels,
 * bf16 input and D a multiple of 16 (STTM_ERR_UNSUPPORTED otherwise); tau_t / tau_t_per_video of
 * *p are ignored.
 *   budget_rows  host, [B]: rows allowed per video (>= 1)
 *   ws           at least sttm_budget_workspace_bytes(p) bytes, 256-byte aligned
 *   tau_t_out    [B] float32, may be NULL: the thresholds chosen
 * Other arguments as sttm_merge_ex.  Asynchronous on `stream`.
 */
size_t sttm_budget_workspace_bytes(const sttm_params* p);
sttm_status sttm_merge_budget(const void* feats, const sttm_params* p, const long long* budget_rows, void* ws,
                              size_t ws_bytes, void* out_feats, int32_t* out_pos, int32_t* merge_map,
                              int32_t* out_count, int64_t* out_offsets, float* tau_t_out, int32_t* device_status,
                              void* stream);

/*
 * "Merged" position strategy of Section 3.4 (the first of its three ways to give a merged token a
 * rotary position): the position of an output row is the average of the positions of the tokens
 * merged into it.  Reading taken here: the position of an input token is its index t*H*W + y*W + x
 * inside its video (the numbering of the survived ids), every cell of the video counts once, and the
 * average is returned as a number (a rotary embedding evaluated at it is left to the caller).
 *   merge_map     [B, N] int32, N = T*H*W: row (inside its video) of every cell, as written by
 *                 sttm_merge_ex
 *   out_offsets   [B + 1] int64: first row of every video in the packed output, as written by
 *                 sttm_merge_ex
 *   ws            at least sttm_merged_positions_workspace(capacity_rows) bytes, 256-byte aligned
 *   out_pos_mean  [capacity_rows] float32: sum of the member indices (exact, 64-bit) divided by their
 *                 number in double precision, rounded once to float; rows at or beyond capacity_rows
 *                 are dropped and (1 << STTM_ERR_CAPACITY) is OR-ed into *device_status (may be NULL)
 * Asynchronous on `stream`.
 */
size_t sttm_merged_positions_workspace(long long capacity_rows);
sttm_status sttm_merged_positions(const int32_t* merge_map, const int64_t* out_offsets, int B, long long N,
                                  void* ws, size_t ws_bytes, float* out_pos_mean, long long capacity_rows,
                                  int32_t* device_status, void* stream);

/* Frees the cached buffers of sttm_merge / sttm_merge_host on the current device. */
void sttm_release_cache(void);

/* Number of kernels the last sttm_merge_ex on this thread enqueued (for benchmarks). */
int sttm_last_launch_count(void);

/*
 * Per-stage timing of sttm_merge_ex for benchmarks.  The path runs as
 * sttm_stage_count() consecutive stages (their names depend on which kernels the last
 * call ran, see sttm_last_path).  After sttm_set_stage_events(events), with
 * `events` a host array of sttm_stage_count()+1 cudaEvent_t handles created by the
 * caller, every sttm_merge_ex on this thread records events[i] on its stream before
 * stage i and events[i+1] after it.  Pass NULL to switch recording off (the default).
 */
int sttm_stage_count(void);
const char* sttm_stage_name(int i);
void sttm_set_stage_events(void** events);

/*
 * Benchmark and test knobs; 0 leaves a choice to the library.
 *   path             0: the library's choice (the two-stream kernels from 0.2 GB of features on
 *                    and for the budget mode, else the single-pass kernel, else the three-pass
 *                    kernels), 1: always the three-pass kernels, 2: the single-pass kernel
 *                    wherever it applies (bf16 input, D a multiple of 16, at most 64 tiles of
 *                    4x4 cells per frame, D / cluster_size <= 1024), 3: the same without
 *                    packing the partial border tiles of a frame together, 5: the two-stream
 *                    kernels wherever they apply (bf16 input, D a multiple of 64), 6: the same
 *                    with the Gram stage on mma.sync instead of tcgen05
 *   cluster_size     single-pass kernel: CTAs that share one tile's channels (1, 2, 4 or 8)
 *   frames_per_item  frames of one tile that are processed in a row (two-stream kernels: at most 64)
 * Not thread safe; affects later calls of every entry point.
 */
void sttm_set_tuning(int path, int cluster_size, int frames_per_item);

/*
 * Second benchmark knob of the fused kernel.  By default a frame stays in the kernel's
 * shared-memory ring from its one read from HBM until its merge decisions exist and the chain
 * sums have used it.  With sum_slots > 0 the ring is split: the frame leaves the first ring
 * after the similarity products and is read a second time (an L2 hit) into a second ring of
 * sum_slots slots for the chain sums, which lets more frames be in flight.
 *   sum_slots    slots of the second ring (at least 2; the rest go to the first); 0: one ring
 *   lead_frames  the second copy of frame q starts once the similarity warp has finished frame
 *                q - lead_frames; 0: right after the frame's own decisions
 * Not thread safe; affects later calls of every entry point.
 */
void sttm_set_ring_split(int sum_slots, int lead_frames);

/* Which kernels the last sttm_merge_ex on this thread ran: 0 three-pass, 1 single-pass (fused),
 * 2 the general kernels for quadtrees of more than three levels, 3 two-stream. */
int sttm_last_path(void);
/* Which Gram stage the last sttm_merge_ex on this thread ran when it took the two-stream kernels:
 * 2 on tcgen05 with the sums in tensor memory, 1 on mma.sync; 0 when it took other kernels. */
int sttm_last_gram_stage(void);

/*
 * Launch shape the fused kernel would get for these params (host pointers; queries the
 * current device for the number of clusters that fit).  shape[12] = {cluster size, channels
 * per CTA, threads per CTA, slots of the first ring, dynamic shared memory bytes, frames per
 * item, items, clusters that can be resident, clusters launched, tensor-core (Gram) warps,
 * slots of the second ring, lead_frames}.  Returns 1, or 0
 * when the fused kernel does not apply to the params.
 */
int sttm_fused_launch_shape(const sttm_params* p, int* shape);

const char* sttm_status_string(sttm_status s);

#ifdef __cplusplus
}
#endif
#endif
