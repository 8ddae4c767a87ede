/*
 * CPU oracle for STTM token merging.  TEST INFRASTRUCTURE ONLY (see sttm_oracle.h).
 *
 * Everything is double precision; inputs (bf16 / f32) are widened exactly and nothing
 * is rounded in between.  The code takes the method's steps in the paper's order:
 *   Section 3.2: leaves = the frame's tokens; 2x2 average pooling up to the coarsest
 *                map; cosine of every node with its parent; coarse-to-fine search that
 *                keeps a node when all of its children are above tau_S;
 *   Section 3.3: compare each kept node of frame t with the kept nodes of frame t-1
 *                that overlap its region, link it to one above tau_T (top-left first),
 *                follow links to the common root in the earliest frame, merge every
 *                node of a connected graph into that root;
 *   Section 3.4: order surviving tokens by frame, then by top-left coordinate, and
 *                give them position ids.
 * There is no blocking, fusion or reordering beyond that.
 */
#include "sttm_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

#define MAXL 24

typedef struct {
    double* F[MAXL];            /* F[l][(i*Wl+j)*D + d]: feature of node (l,i,j)            */
    double* sim[MAXL];          /* sim[l][i*Wl+j]: cos(node (l,i,j), its parent), l < L-1    */
    unsigned char* kept[MAXL];  /* kept[l][i*Wl+j]: node survives the search                 */
    int8_t* cover;              /* [H*W] level of the kept node covering each cell           */
    int32_t* root;              /* [H*W] per cell: anchor id of the root of its covering node */
    int64_t* row;               /* [H*W] per cell: output row of that root                    */
} frame_t;

static int imax(int a, int b) { return a > b ? a : b; }
static int imin(int a, int b) { return a < b ? a : b; }

/* Section 3.2, "recursively downsampling the feature map": level sizes.  The paper
 * writes H/2 x W/2; for odd sizes the halving rounds up, so that border parents have
 * two or one child (the paper's own 14x14 grid reaches its 4x4 and 2x2 coarsest maps
 * only this way: 14 -> 7 -> 4 -> 2). */
int oracle_levels(int H, int W, int lv1, int* Hl, int* Wl)
{
    int L = 1;
    Hl[0] = H; Wl[0] = W;
    while (imax(Hl[L - 1], Wl[L - 1]) > lv1 && L < MAXL) {
        Hl[L] = (Hl[L - 1] + 1) / 2;
        Wl[L] = (Wl[L - 1] + 1) / 2;
        L++;
    }
    return L;
}

int oracle_sims_per_frame(int H, int W, int lv1)
{
    int Hl[MAXL], Wl[MAXL], n = 0;
    int L = oracle_levels(H, W, lv1, Hl, Wl);
    for (int l = 0; l + 1 < L; l++) n += Hl[l] * Wl[l];
    return n;
}

static double widen(const void* feats, int dtype, int64_t idx)
{
    if (dtype == ORACLE_F64) return ((const double*)feats)[idx];
    if (dtype == ORACLE_F32) return (double)((const float*)feats)[idx];
    uint32_t bits = ((uint32_t)((const uint16_t*)feats)[idx]) << 16;   /* bf16 = top half of f32 */
    float f;
    memcpy(&f, &bits, 4);
    return (double)f;
}

/* Cosine similarity; 0 when either vector is all zero (the paper does not say). */
static double cosine(const double* a, const double* b, int D)
{
    double ab = 0.0, aa = 0.0, bb = 0.0;
    for (int d = 0; d < D; d++) { ab += a[d] * b[d]; aa += a[d] * a[d]; bb += b[d] * b[d]; }
    if (aa == 0.0 || bb == 0.0) return 0.0;
    return ab / (sqrt(aa) * sqrt(bb));
}

/* Section 3.2, second step: each parent is the average of its existing children
 * (four, or two / one on the border of an odd-sized map). */
static void build_pyramid(frame_t* fr, int L, const int* Hl, const int* Wl, int D)
{
    for (int l = 0; l + 1 < L; l++) {
        for (int i = 0; i < Hl[l + 1]; i++) for (int j = 0; j < Wl[l + 1]; j++) {
            double* p = fr->F[l + 1] + ((int64_t)i * Wl[l + 1] + j) * D;
            int n = 0;
            for (int d = 0; d < D; d++) p[d] = 0.0;
            for (int a = 0; a < 2; a++) for (int b = 0; b < 2; b++) {
                int ci = 2 * i + a, cj = 2 * j + b;
                if (ci >= Hl[l] || cj >= Wl[l]) continue;
                const double* c = fr->F[l] + ((int64_t)ci * Wl[l] + cj) * D;
                for (int d = 0; d < D; d++) p[d] += c[d];
                n++;
            }
            for (int d = 0; d < D; d++) p[d] /= (double)n;
        }
    }
}

/* Section 3.2: "cosine similarity between the current level's nodes and their child
 * nodes", stored at the child. */
static void parent_child_sims(frame_t* fr, int L, const int* Hl, const int* Wl, int D)
{
    for (int l = 0; l + 1 < L; l++)
        for (int i = 0; i < Hl[l]; i++) for (int j = 0; j < Wl[l]; j++) {
            const double* c = fr->F[l] + ((int64_t)i * Wl[l] + j) * D;
            const double* p = fr->F[l + 1] + ((int64_t)(i / 2) * Wl[l + 1] + (j / 2)) * D;
            fr->sim[l][i * Wl[l] + j] = cosine(c, p, D);
        }
}

/* Section 3.2 / Fig. 3, the granularity decision: start from every node of the
 * coarsest level; a node whose children are all above tau_S is kept and its subtree is
 * pruned, otherwise the node is pruned and its children are searched.  Nodes of the
 * finest level that are reached are kept.  Returns the number of comparisons made. */
static int64_t quadtree_search(frame_t* fr, int L, const int* Hl, const int* Wl, double tau_s)
{
    int64_t comparisons = 0;
    unsigned char* active[MAXL];
    for (int l = 0; l < L; l++) {
        active[l] = (unsigned char*)calloc((size_t)Hl[l] * Wl[l], 1);
        memset(fr->kept[l], 0, (size_t)Hl[l] * Wl[l]);
    }
    memset(active[L - 1], 1, (size_t)Hl[L - 1] * Wl[L - 1]);
    for (int l = L - 1; l >= 1; l--)
        for (int i = 0; i < Hl[l]; i++) for (int j = 0; j < Wl[l]; j++) {
            if (!active[l][i * Wl[l] + j]) continue;
            int all_pass = 1;
            for (int a = 0; a < 2; a++) for (int b = 0; b < 2; b++) {
                int ci = 2 * i + a, cj = 2 * j + b;
                if (ci >= Hl[l - 1] || cj >= Wl[l - 1]) continue;
                comparisons++;
                if (!(fr->sim[l - 1][ci * Wl[l - 1] + cj] > tau_s)) all_pass = 0;
            }
            if (all_pass) { fr->kept[l][i * Wl[l] + j] = 1; continue; }
            for (int a = 0; a < 2; a++) for (int b = 0; b < 2; b++) {
                int ci = 2 * i + a, cj = 2 * j + b;
                if (ci >= Hl[l - 1] || cj >= Wl[l - 1]) continue;
                active[l - 1][ci * Wl[l - 1] + cj] = 1;
            }
        }
    for (int k = 0; k < Hl[0] * Wl[0]; k++) if (active[0][k]) fr->kept[0][k] = 1;
    for (int l = 0; l < L; l++) free(active[l]);
    /* which kept node covers each cell */
    for (int y = 0; y < Hl[0]; y++) for (int x = 0; x < Wl[0]; x++) {
        int found = -1;
        for (int l = 0; l < L; l++) if (fr->kept[l][(y >> l) * Wl[l] + (x >> l)]) { found = l; break; }
        fr->cover[y * Wl[0] + x] = (int8_t)found;
    }
    return comparisons;
}

static void frame_alloc(frame_t* fr, int L, const int* Hl, const int* Wl, int D)
{
    for (int l = 0; l < L; l++) {
        size_t n = (size_t)Hl[l] * Wl[l];
        fr->F[l] = (double*)malloc(n * D * sizeof(double));
        fr->sim[l] = (double*)calloc(n, sizeof(double));
        fr->kept[l] = (unsigned char*)calloc(n, 1);
    }
    size_t hw = (size_t)Hl[0] * Wl[0];
    fr->cover = (int8_t*)malloc(hw);
    fr->root = (int32_t*)malloc(hw * sizeof(int32_t));
    fr->row = (int64_t*)malloc(hw * sizeof(int64_t));
}

static void frame_free(frame_t* fr, int L)
{
    for (int l = 0; l < L; l++) { free(fr->F[l]); free(fr->sim[l]); free(fr->kept[l]); }
    free(fr->cover); free(fr->root); free(fr->row);
}

int64_t oracle_merge(const void* feats, const oracle_cfg* cfg,
                     double* spatial_sims, int8_t* cover_level,
                     int32_t* link, int32_t* root, int32_t* merge_map,
                     double* out_feats, int32_t* out_pos, int32_t* out_members,
                     int64_t out_capacity,
                     int32_t* tsim_v, int32_t* tsim_u, double* tsim, int64_t tsim_capacity,
                     int64_t* counters)
{
    if (!feats || !cfg || cfg->T < 1 || cfg->H < 1 || cfg->W < 1 || cfg->D < 1 || cfg->lv1 < 1) return -1;
    const int T = cfg->T, H = cfg->H, W = cfg->W, D = cfg->D, HW = H * W;
    int Hl[MAXL], Wl[MAXL];
    const int L = oracle_levels(H, W, cfg->lv1, Hl, Wl);
    const int nsim = oracle_sims_per_frame(H, W, cfg->lv1);

    frame_t frames[2];
    frame_alloc(&frames[0], L, Hl, Wl, D);
    frame_alloc(&frames[1], L, Hl, Wl, D);
    double* wsum = out_feats ? (double*)calloc((size_t)(out_capacity > 0 ? out_capacity : 1), sizeof(double)) : NULL;
    int32_t* cand_level = (int32_t*)malloc((size_t)HW * sizeof(int32_t));
    int32_t* cand_index = (int32_t*)malloc((size_t)HW * sizeof(int32_t));

    int64_t n_rows = 0, cmp_spatial = 0, cmp_temporal = 0, n_pairs = 0;

    for (int t = 0; t < T; t++) {
        frame_t* cur = &frames[t & 1];
        frame_t* prev = &frames[(t & 1) ^ 1];

        /* leaves = the frame's token map (Section 3.2, first step) */
        for (int64_t k = 0; k < (int64_t)HW * D; k++)
            cur->F[0][k] = widen(feats, cfg->dtype, (int64_t)t * HW * D + k);
        build_pyramid(cur, L, Hl, Wl, D);
        parent_child_sims(cur, L, Hl, Wl, D);
        cmp_spatial += quadtree_search(cur, L, Hl, Wl, cfg->tau_s);

        if (spatial_sims) {
            double* dst = spatial_sims + (int64_t)t * nsim;
            for (int l = 0; l + 1 < L; l++) {
                memcpy(dst, cur->sim[l], (size_t)Hl[l] * Wl[l] * sizeof(double));
                dst += Hl[l] * Wl[l];
            }
        }
        if (cover_level) memcpy(cover_level + (int64_t)t * HW, cur->cover, (size_t)HW);

        /* kept nodes of this frame in order of their top-left (anchor) cell, row-major:
         * a node is met first at its anchor cell */
        for (int y0 = 0; y0 < H; y0++) for (int x0 = 0; x0 < W; x0++) {
            const int lv = cur->cover[y0 * W + x0];
            const int side = 1 << lv;
            if ((y0 & (side - 1)) || (x0 & (side - 1))) continue;      /* not an anchor */
            const int i = y0 >> lv, j = x0 >> lv;
            const double* Fv = cur->F[lv] + ((int64_t)i * Wl[lv] + j) * D;
            const int y1 = imin(y0 + side, H), x1 = imin(x0 + side, W);
            const int32_t v_id = t * HW + y0 * W + x0;

            /* Section 3.3: candidates = kept nodes of frame t-1 overlapping v's region */
            int32_t link_to = -1;
            if (t > 0) {
                int ncand = 0;
                if (cfg->match_mode == ORACLE_MATCH_TOPLEFT_ONLY) {
                    int lu = prev->cover[y0 * W + x0];
                    cand_level[0] = lu; cand_index[0] = (y0 >> lu) * Wl[lu] + (x0 >> lu); ncand = 1;
                } else {
                    for (int y = y0; y < y1; y++) for (int x = x0; x < x1; x++) {
                        int lu = prev->cover[y * W + x];
                        int idx = (y >> lu) * Wl[lu] + (x >> lu);
                        int seen = 0;
                        for (int c = 0; c < ncand; c++) if (cand_level[c] == lu && cand_index[c] == idx) seen = 1;
                        if (!seen) { cand_level[ncand] = lu; cand_index[ncand] = idx; ncand++; }
                    }
                }
                double best_sim = 0.0;
                for (int c = 0; c < ncand; c++) {
                    int lu = cand_level[c], iu = cand_index[c] / Wl[lu], ju = cand_index[c] % Wl[lu];
                    const double* Fu = prev->F[lu] + (int64_t)cand_index[c] * D;
                    int32_t u_id = (t - 1) * HW + (iu << lu) * W + (ju << lu);
                    double s = cosine(Fv, Fu, D);
                    cmp_temporal++;
                    if (n_pairs < tsim_capacity) {
                        if (tsim_v) tsim_v[n_pairs] = v_id;
                        if (tsim_u) tsim_u[n_pairs] = u_id;
                        if (tsim) tsim[n_pairs] = s;
                    }
                    n_pairs++;
                    if (!(s > cfg->tau_t)) continue;                 /* "similarity higher than tau_T" */
                    if (link_to < 0) { link_to = u_id; best_sim = s; }
                    else if (cfg->match_mode == ORACLE_MATCH_BEST) {
                        if (s > best_sim || (s == best_sim && u_id < link_to)) { link_to = u_id; best_sim = s; }
                    } else if (u_id < link_to) { link_to = u_id; best_sim = s; }   /* priority to the top-left */
                }
            }

            /* common root: the root of the node v is linked to, else v itself */
            int32_t root_id; int64_t row;
            if (link_to >= 0) {
                int cell = link_to - (t - 1) * HW;
                root_id = prev->root[cell];
                row = prev->row[cell];
            } else {
                root_id = v_id;
                row = n_rows++;                                       /* roots appear in (t, y0, x0) order */
                if (row < out_capacity) {
                    if (out_pos) out_pos[row] = cfg->pos_mode == ORACLE_POS_REASSIGNED ? (int32_t)row : v_id;
                    if (out_members) out_members[row] = 0;
                    if (out_feats) for (int d = 0; d < D; d++) out_feats[row * D + d] = 0.0;
                }
            }
            /* merge v into its root (weights: one per node, or the node's cell count) */
            if (row < out_capacity) {
                double w = cfg->weight_mode == ORACLE_W_AREA ? (double)((y1 - y0) * (x1 - x0)) : 1.0;
                if (out_feats) { for (int d = 0; d < D; d++) out_feats[row * D + d] += w * Fv[d]; wsum[row] += w; }
                if (out_members) out_members[row] += 1;
            }
            for (int y = y0; y < y1; y++) for (int x = x0; x < x1; x++) {
                cur->root[y * W + x] = root_id;
                cur->row[y * W + x] = row;
                if (link) link[(int64_t)t * HW + y * W + x] = link_to;
                if (root) root[(int64_t)t * HW + y * W + x] = root_id;
                if (merge_map) merge_map[(int64_t)t * HW + y * W + x] = (int32_t)row;
            }
        }
    }
    if (out_feats) {
        int64_t n = n_rows < out_capacity ? n_rows : out_capacity;
        for (int64_t r = 0; r < n; r++) for (int d = 0; d < D; d++) out_feats[r * D + d] /= wsum[r];
    }
    if (counters) { counters[0] = cmp_spatial; counters[1] = cmp_temporal; counters[2] = n_pairs; }
    free(wsum); free(cand_level); free(cand_index);
    frame_free(&frames[0], L); frame_free(&frames[1], L);
    return n_rows;
}
