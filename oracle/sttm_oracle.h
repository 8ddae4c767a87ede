/*
 * CPU oracle for STTM token merging (spatial quadtree search, temporal directed merge,
 * reordering).  TEST INFRASTRUCTURE ONLY: a plain, slow, double-precision restatement
 * of the method, written from the paper's Section 3 (3.2 spatial, 3.3 temporal,
 * 3.4 reordering) so that a reader can check it against the text.  It shares no code
 * with the CUDA library and is never on the product path; only tests, the smoke check
 * and the CPU-baseline leg of the benchmark call it.
 *
 * Pins (see tests): brute-force enumeration on tiny grids, closed-form cosines of a
 * hand-worked 2x2 example, library average pooling, identity / run-length special
 * cases, the comparison counts of Eq. 1-2 and of Section 3.3, and invariants.
 * Choices the paper leaves open (averaging weights, candidate rule, scan order) are
 * switches here; for those the paper gives no value to compare against:
 * "parity unpinned" by the paper for weight_mode, match_mode and the row-major order.
 */
#ifndef STTM_ORACLE_H
#define STTM_ORACLE_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORACLE_BF16 = 0, ORACLE_F32 = 1, ORACLE_F64 = 2 };
enum { ORACLE_W_NODE = 0, ORACLE_W_AREA = 1 };
enum { ORACLE_POS_SURVIVED = 0, ORACLE_POS_REASSIGNED = 1 };
/* 0: top-left-most candidate among those above tau_t (Section 3.3);
 * 1: most similar candidate among those above tau_t (the "optimal" ablation);
 * 2: only the candidate covering the node's own top-left cell is examined. */
enum { ORACLE_MATCH_TOPLEFT = 0, ORACLE_MATCH_BEST = 1, ORACLE_MATCH_TOPLEFT_ONLY = 2 };

typedef struct {
    int T, H, W, D;
    int dtype;          /* ORACLE_BF16 (uint16 bit patterns), ORACLE_F32, ORACLE_F64 */
    int lv1;            /* coarsest map is at most lv1 x lv1 (2 or 4 in the paper)   */
    double tau_s, tau_t;
    int weight_mode, pos_mode, match_mode;
} oracle_cfg;

/* Number of quadtree levels and their sizes (level 0 = the token grid). Returns L. */
int oracle_levels(int H, int W, int lv1, int* Hl, int* Wl);

/* Parent-child similarities per frame are stored level by level:
 * level 0 (H0*W0 values, row-major), then level 1, ... level L-2. */
int oracle_sims_per_frame(int H, int W, int lv1);

/*
 * The whole path.  Every output pointer may be NULL.
 *   spatial_sims [T][oracle_sims_per_frame]   cos(node, its parent)
 *   cover_level  [T*H*W]   level of the kept node that covers each cell
 *   link         [T*H*W]   per cell: anchor id (t*H*W + y0*W + x0) of the node its
 *                          covering node is linked to in frame t-1, or -1
 *   root         [T*H*W]   per cell: anchor id of the root of its covering node
 *   merge_map    [T*H*W]   per cell: output row of that root
 *   out_feats    [out_capacity][D] doubles, row-major; rows beyond capacity are not
 *                          written (the count is still exact)
 *   out_pos      [out_capacity]
 *   out_members  [out_capacity] number of member nodes of each row
 *   tsim_v, tsim_u, tsim  [tsim_capacity]  every temporal candidate pair that was
 *                          evaluated: anchor ids of v (frame t) and u (frame t-1), cosine
 *   counters[0] = parent-child comparisons made by the top-down search,
 *   counters[1] = temporal comparisons, counters[2] = temporal pairs stored.
 * Returns the number of output rows, or a negative value on bad arguments.
 */
int64_t oracle_merge(const void* feats, const oracle_cfg* cfg,
                     double* spatial_sims, int8_t* cover_level,
                     int32_t* link, int32_t* root, int32_t* merge_map,
                     double* out_feats, int32_t* out_pos, int32_t* out_members,
                     int64_t out_capacity,
                     int32_t* tsim_v, int32_t* tsim_u, double* tsim, int64_t tsim_capacity,
                     int64_t* counters);

#ifdef __cplusplus
}
#endif
#endif
