// Host side of the STTM library: argument checks, workspace layout, kernel launches.
// Exports the C ABI declared in include/sttm.h.
#include "../../include/sttm.h"

#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <vector>

#include "sttm_kernels.cuh"
#include "sttm_fused.cuh"
#include "sttm_flow.cuh"
#include "sttm_generic.cuh"
#include "sttm_gram_tc.cuh"
#include "sttm_segments.cuh"

namespace {

using namespace sttm;

constexpr int kSmCount = 148;   // B200 (grid sizes of the older kernels; the streaming kernels ask the device)

// multiprocessors of the current device
int sm_count() {
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return kSmCount;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = kSmCount;
        cached[dev] = n;
    }
    return cached[dev];
}

thread_local int g_launches = 0;
// What the budget mode hands to its two passes of the ordinary path (nothing of it is global state).
struct Internal {
    float* tmax = nullptr;              // first pass: per kept node the largest cosine to its candidates goes here
    const float* tau_dev = nullptr;     // second pass: temporal thresholds in device memory
    bool second_pass = false;           // the Gram stage's numbers of the first pass are still in the workspace
    bool budget = false;                // plan as the budget mode does (two-stream kernels)
};
thread_local cudaEvent_t* g_stage_events = nullptr;   // when set: event i is recorded after stage i-1

constexpr int kStageCount = 5;
const char* const kStageNames[4][kStageCount] = {
    {"spatial", "temporal+roots", "ordering", "accumulate", "combine"},
    {"fused", "roots", "ordering", "gather", "-"},
    {"-", "-", "-", "-", "general"},
    {"gram", "decide+ordering+chain", "sum", "roots+pieces", "-"}};
thread_local int g_last_gram = 0;   // 0: no two-stream kernels, 1: their Gram stage on mma.sync, 2: on tcgen05
thread_local int g_last_path = 0;   // 0: three-pass kernels, 1: single-pass kernel, 2: general kernels, 3: two-stream kernels

// Stage boundary `boundary` (before stage `boundary`, after the one before it): an event for the
// benchmark when it asked for them, and an NVTX range named after the stage around the launches
// of the stage, so that a timeline shows the path's stages (costs nothing without a profiler).
thread_local bool g_range_open = false;
inline void close_stage_range() {
    if (g_range_open) { nvtxRangePop(); g_range_open = false; }
}
inline void mark_stage(int boundary, cudaStream_t st) {
    if (g_stage_events != nullptr) cudaEventRecord(g_stage_events[boundary], st);
    close_stage_range();
    if (boundary < kStageCount && kStageNames[g_last_path][boundary][0] != '-') {
        nvtxRangePushA(kStageNames[g_last_path][boundary]);
        g_range_open = true;
    }
}

inline size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

// index of the current device for the per-device tables below (function attributes and occupancy
// answers belong to a device); -1 when it cannot be had or is beyond the tables
constexpr int kMaxDevices = 64;
inline int device_slot() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}

// Launch shape of the fused kernel for one problem; ok == false: the three-pass kernels run.
struct FusedPlan {
    bool ok;
    int C, S, NM, NA, R, RB, lead, row_bytes, slot_bytes, F, nseg, nitems, ntiles, Wt;
    size_t smem;
    TileDesc tiles[kMaxTiles];      // most cells first
};

// Launch shape of the two-stream kernels; ok == false: the single-pass kernel (or the three-pass kernels) run.
struct FlowPlan {
    bool ok;
    int NS, NB, R, slot_bytes, F, nseg, nitems, ntiles;
    int NSg, NBg, NCg;              // Gram stage: slices, blocks per copy, copies per slice
    bool tc;                        // Gram stage on tcgen05 (else on mma.sync, with the sum stage's slices)
    size_t smem, smem_tc;
    TileDesc tiles[kMaxTiles];
    TileBox boxes[kMaxTiles];
};

struct Plan {
    Geo g;
    int Tc, nchunk, nslice;
    long long cells;          // B*N
    long long partial_slots;
    FusedPlan f;
    FlowPlan fl;
    bool generic;             // more than three quadtree levels: the plain kernels of sttm_generic.cuh
    Pyr py;
    size_t gen_pooled, gen_norms, gen_dots, gen_allpass, gen_cnt, gen_start, gen_list, gen_sorted;
    size_t norms_bytes;       // the spatial stage's only scratch: one squared norm per quadtree node
    // byte offsets into the workspace
    size_t norms, cover, link, root, row_at_root, cell_row, row_anchor, span_off, frame_roots,
        frame_base, vid_off, zero_begin, frame_counts, row_weight, row_last_t, span_total, status, queue,
        zero_end, partial, row_head, staging, pieces, piece_meta, piece_row, lead_n, lead_ids, lead_list, flow_progress, flow_partial,
        flow_hand, flow_recs, total;
};

// benchmark / test knobs (sttm_set_tuning): 0 = choose automatically
int g_tune_path = 0, g_tune_cluster = 0, g_tune_seg = 0, g_tune_pack = 0, g_tune_sum_slots = 0, g_tune_lead = 0;

constexpr size_t kMaxSmem = 232448;   // 227 KB per CTA on sm_100
constexpr double kFlowMinBytes = 200e6;                    // input size from which the two-stream kernels are the default
constexpr size_t kFlowSmemMax = (233472 - 2 * 1024) / 2;   // per CTA when two share an SM

// Cuts the grid into the kernel's tiles.  Full 4x4 tiles map one to one.  The partial tiles of
// the right and bottom border are packed several to a tile: a partial tile of r x c cells sits
// at an offset (oy, ox) of the 4x4 lane grid that keeps its own 2x2 blocks on lane pairs
// (ox even when c >= 2, ox = 0 when c > 2, the same for rows), and every lane records which
// neighbour lanes belong to its block and its coarsest node, so packed tiles never mix.
int fused_resident_clusters(const FusedPlan& f);

template <typename PlanT>
bool build_tiles(const Geo& g, PlanT* f) {
    struct Part { int y0, x0, r, c; };
    std::vector<Part> full, part;
    for (int y0 = 0; y0 < g.H; y0 += 4)
        for (int x0 = 0; x0 < g.W; x0 += 4) {
            Part pt{y0, x0, std::min(4, g.H - y0), std::min(4, g.W - x0)};
            (pt.r == 4 && pt.c == 4 ? full : part).push_back(pt);
        }
    std::vector<TileDesc> tiles;
    auto blank = [] { TileDesc t; std::memset(t.y, 255, 16); std::memset(t.x, 0, 16); std::memset(t.bits, 0, 16); return t; };
    auto place = [&](TileDesc& t, const Part& pt, int oy, int ox) {
        const int qb = (pt.c >= 2 ? 1 : 0) | (pt.r >= 2 ? 4 : 0);
        const int tb = qb | (pt.c > 2 ? 2 : 0) | (pt.r > 2 ? 8 : 0);
        for (int dy = 0; dy < pt.r; dy++)
            for (int dx = 0; dx < pt.c; dx++) {
                const int l = (oy + dy) * 4 + ox + dx;
                t.y[l] = (unsigned char)(pt.y0 + dy);
                t.x[l] = (unsigned char)(pt.x0 + dx);
                t.bits[l] = (unsigned char)(qb | (tb << 4));
            }
    };
    if (g.H > 254 || g.W > 254) return false;
    for (const Part& pt : full) { TileDesc t = blank(); place(t, pt, 0, 0); tiles.push_back(t); }
    std::vector<TileDesc> packed;
    std::stable_sort(part.begin(), part.end(), [](const Part& a, const Part& b) { return a.r * a.c > b.r * b.c; });
    for (const Part& pt : part) {
        bool done = false;
        for (size_t k = 0; k < packed.size() && !done; k++) {
            if (g_tune_pack == 1) break;
            for (int oy = 0; oy + pt.r <= 4 && !done; oy++) {
                if ((pt.r >= 2 && (oy & 1)) || (pt.r > 2 && oy != 0)) continue;
                for (int ox = 0; ox + pt.c <= 4 && !done; ox++) {
                    if ((pt.c >= 2 && (ox & 1)) || (pt.c > 2 && ox != 0)) continue;
                    bool free_ = true;
                    for (int dy = 0; dy < pt.r; dy++)
                        for (int dx = 0; dx < pt.c; dx++)
                            if (packed[k].y[(oy + dy) * 4 + ox + dx] != 255) free_ = false;
                    if (free_) { place(packed[k], pt, oy, ox); done = true; }
                }
            }
        }
        if (!done) { TileDesc t = blank(); place(t, pt, 0, 0); packed.push_back(t); }
    }
    for (const TileDesc& t : packed) tiles.push_back(t);
    if ((int)tiles.size() > kMaxTiles) return false;
    f->ntiles = (int)tiles.size();
    for (int t = 0; t < f->ntiles; t++) f->tiles[t] = tiles[t];
    return true;
}

// Tiles of the two-stream kernels: what one tensor copy brings in.  4x4 boxes over the part of the
// grid whose sides are multiples of four or end in a part of two or three cells (such a box reaches
// over the border and the copy fills the rows outside with zeros); a grid one cell wider than a
// multiple of four has its last column cut into runs of 16 cells instead, one cell higher its last
// row (so that 13x13 is 9 + 1 + 1 tiles).  A run of a column holds the column's share of up to four
// coarsest nodes, each on four consecutive lanes: lane pairs are 2x2 blocks (bit 1), lane quadruples
// coarsest nodes (bits 1 and 2).
bool build_flow_tiles(const Geo& g, FlowPlan* f) {
    if (g.H > 254 || g.W > 254) return false;
    const bool col_strip = g.W % 4 == 1, row_strip = g.H % 4 == 1;
    const int Wf = col_strip ? g.W - 1 : g.W, Hf = row_strip ? g.H - 1 : g.H;
    std::vector<TileDesc> tiles;
    std::vector<TileBox> boxes;
    auto blank = [] { TileDesc t; std::memset(t.y, 255, 16); std::memset(t.x, 0, 16); std::memset(t.bits, 0, 16); return t; };
    for (int y0 = 0; y0 < Hf; y0 += 4)
        for (int x0 = 0; x0 < Wf; x0 += 4) {
            const int r = std::min(4, g.H - y0), c = std::min(4, g.W - x0);
            const int qb = (c >= 2 ? 1 : 0) | (r >= 2 ? 4 : 0);
            const int tb = qb | (c > 2 ? 2 : 0) | (r > 2 ? 8 : 0);
            TileDesc t = blank();
            for (int dy = 0; dy < r; dy++)
                for (int dx = 0; dx < c; dx++) {
                    const int l = dy * 4 + dx;
                    t.y[l] = (unsigned char)(y0 + dy);
                    t.x[l] = (unsigned char)(x0 + dx);
                    t.bits[l] = (unsigned char)(qb | (tb << 4));
                }
            tiles.push_back(t);
            boxes.push_back(TileBox{0, x0, y0, 0});
        }
    // runs along the last column (kind 1) and the last row (kind 2); the corner cell goes with the column
    for (int kind = 1; kind <= 2; kind++) {
        if (kind == 1 ? !col_strip : !row_strip) continue;
        const int len = kind == 1 ? g.H : Wf;               // cells of the strip
        const int full = kind == 1 ? g.H : g.W;             // the grid's extent along the strip
        for (int a0 = 0; a0 < len; a0 += 16) {
            TileDesc t = blank();
            for (int l = 0; l < 16 && a0 + l < len; l++) {
                const int a = a0 + l;
                const int r = std::min(4, full - a / 4 * 4);    // cells of this coarsest node along the strip
                const int qb = r >= 2 ? 1 : 0, tb = qb | (r > 2 ? 2 : 0);
                t.y[l] = (unsigned char)(kind == 1 ? a : g.H - 1);
                t.x[l] = (unsigned char)(kind == 1 ? g.W - 1 : a);
                t.bits[l] = (unsigned char)(qb | (tb << 4));
            }
            tiles.push_back(t);
            boxes.push_back(kind == 1 ? TileBox{1, g.W - 1, a0, 0} : TileBox{2, a0, g.H - 1, 0});
        }
    }
    if (tiles.empty() || (int)tiles.size() > kMaxTiles) return false;
    f->ntiles = (int)tiles.size();
    for (int t = 0; t < f->ntiles; t++) { f->tiles[t] = tiles[t]; f->boxes[t] = boxes[t]; }
    return true;
}

// Two-stream kernels: bf16 input, channels a multiple of 64, slices of up to eight 64-channel blocks.
void plan_flow(const sttm_params* p, const Geo& g, FlowPlan* f, bool budget) {
    f->ok = false;
    // On request, for the budget mode (its second pass reuses the first pass's Gram stage), and for
    // large inputs: measured on B200, the two-stream kernels overtake the single-pass kernel between
    // 0.08 GB (llava: 0.094 against 0.077 ms) and 0.23 GB (qwen: 0.163 against 0.172 ms) of features.
    const bool large = (double)g.B * g.N * g.D * 2.0 >= kFlowMinBytes;
    if (!(g_tune_path == 5 || g_tune_path == 6 || (g_tune_path == 0 && (budget || large)))) return;
    if (p->in_dtype != STTM_BF16 || g.D % 64 != 0) return;
    if (!build_flow_tiles(g, f)) return;
    const int nblk = g.D / 64;
    // blocks per slice: the largest divisor of the block count up to 14, two to a sum warp (D = 3584:
    // four slices of 14 blocks, 896 channels; memory serves chunks of that size at nearly full speed,
    // chunks of half the size measurably slower)
    int NB = 0;
    for (int n = std::min(nblk, kFlowMaxNB); n >= 1 && NB == 0; n--)
        if (nblk % n == 0) NB = n;
    if (nblk / NB > 64) return;
    f->NB = NB;
    f->NS = nblk / NB;
    f->slot_bytes = NB * kBlkBytes;
    // two CTAs per SM: each gets half of the SM's shared memory (less the system's 1 KB per CTA)
    int R = 0;
    for (int r = kFlowMaxRing; r >= 2; r--)
        if ((size_t)r * f->slot_bytes + flow_fixed_smem(r) <= kFlowSmemMax) { R = r; break; }
    if (R == 0) return;
    f->R = R;
    f->smem = (size_t)f->R * f->slot_bytes + flow_fixed_smem(f->R);
    // Frames per item: the tasks (item x slice) are dealt round robin to two CTAs per SM, so the
    // stages take rounds x (frames of an item + the frame before it + what starting a task costs);
    // the shortest such product over the admissible item lengths (long items mean few pieces, short
    // items mean enough tasks for a short video to fill the GPU).
    if (g_tune_seg > 0) {
        f->F = std::min(g.T, std::min(g_tune_seg, kFlowMaxF));
    } else {
        const long long ctas = 2ll * sm_count();
        long long best_cost = -1;
        int best_F = std::min(g.T, 32);
        for (int F = std::min(g.T, kFlowMaxF); F >= std::min(g.T, 8); F--) {
            const long long nseg = (g.T + F - 1) / F;
            const long long tasks = (long long)g.B * f->ntiles * nseg * f->NS;
            // (two streams of that length, and the chain stage, one warp per run, a third of a frame's
            // streaming time per frame of the run)
            const long long cost = 20 * ((tasks + ctas - 1) / ctas) * (F + 1 + 3) + 6 * F;
            if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_F = F; }
        }
        f->F = best_F;
    }
    f->nseg = (g.T + f->F - 1) / f->F;
    f->nitems = g.B * f->ntiles * f->nseg;
    // Gram stage on tcgen05: slices of up to seven blocks (a ring slot holds five frames of a slice)
    f->tc = g_tune_path != 6;
    f->NBg = f->NB;
    f->NSg = f->NS;
    f->NCg = 1;
    f->smem_tc = 0;
    if (f->tc) {
        int nb = 0;
        for (int n = std::min(nblk, kTcMaxNB); n >= 1 && nb == 0; n--)
            if (nblk % n == 0) nb = n;
        // Slices: a slice's channels come in copies of nb blocks that are added in tensor memory, so the
        // number of slices is free among the divisors of the copy count.  Few slices: little to write, read
        // out and add up in the decision stage (about 1 % of the stage per slice, measured on `long`); many: even
        // task counts and short tasks (a CTA's last task ends about a fifth of a task after the average).
        const int ncopies = nblk / nb;
        int best_ns = 0;
        long long best_cost = 0;
        for (int ns = 1; ns <= std::min(ncopies, 64); ns++) {
            if (ncopies % ns != 0) continue;
            const long long tasks = (long long)f->nitems * ns;
            const long long rounds = (tasks + sm_count() - 1) / sm_count();
            const long long cost = (rounds * 1000 + 180) / ns + 11ll * ns * f->nitems / sm_count();
            if (best_ns == 0 || cost < best_cost) { best_ns = ns; best_cost = cost; }
        }
        if (best_ns == 0) {
            f->tc = false;
        } else {
            f->NBg = nb;
            f->NSg = best_ns;
            f->NCg = ncopies / best_ns;
            f->smem_tc = tc_smem_bytes(nb);
        }
    }
    f->ok = true;
}

void plan_fused(const sttm_params* p, const Geo& g, FusedPlan* f) {
    f->ok = false;
    if (g_tune_path == 1) return;
    if (p->in_dtype != STTM_BF16 || g.D % 16 != 0) return;
    f->Wt = (g.W + 3) / 4;
    if (!build_tiles(g, f)) return;
    int C = 0;
    for (int c = 1; c <= kMaxCluster; c *= 2) {
        if (g_tune_cluster && c != g_tune_cluster) continue;
        if (g.D % (16 * c) == 0 && g.D / c <= 128 * kMaxSumWarps) { C = c; break; }
    }
    if (C == 0) return;
    f->C = C;
    f->S = g.D / C;
    const int ksteps = f->S / 16;
    f->NM = ksteps >= 8 ? 4 : (ksteps >= 4 ? 2 : 1);
    f->NA = (f->S + 127) / 128;
    f->row_bytes = f->S * 2 + 16;          // +16: rows fall in different bank groups for ldmatrix
    f->slot_bytes = 16 * f->row_bytes;
    const size_t fixed = (size_t)f->NM * kGramVals * 4 + kGramVals * 4 + (size_t)kRecRing * C * kSumVals * 4 +
                         128 + kRecRing * kSumVals * 4 + kRecRing * 16 * 4 + sizeof(SlotTable) + kRecRing * sizeof(FrameRec) + 16 +
                         (4 * kMaxRing + 6 * kRecRing + 4) * 8;
    // the slots that fit: one ring in which a frame stays until the sum warps have used it, or,
    // on request, shared out between the Gram warps' ring (a frame stays for its own products and
    // the next frame's) and a ring of the sum warps (filled from L2 shortly before use)
    const int slots = std::min((int)((kMaxSmem - fixed) / f->slot_bytes), 2 * kMaxRing);
    if (slots < 5) return;
    int RB = 0;                                 // one ring for both unless asked otherwise
    if (g_tune_sum_slots > 0) RB = std::max(2, std::min(g_tune_sum_slots, std::min(slots - 3, kMaxRing)));
    f->RB = RB;
    f->R = std::min(slots - RB, kMaxRing);
    f->lead = std::max(0, g_tune_lead);
    f->smem = (size_t)(f->R + f->RB) * f->slot_bytes + fixed;
    // frames per item: about four items per resident cluster, with the number of items as close
    // below a multiple of the cluster count as the frame count allows (the items are dealt out
    // statically, and every item of a cluster costs about the same)
    if (g_tune_seg > 0) {
        f->F = std::min(g_tune_seg, g.T);
    } else {
        const int ncl = fused_resident_clusters(*f);
        const long long tiles_all = (long long)g.B * f->ntiles;
        const int lo = 1, hi = std::max(lo, std::min(g.T, std::max(1, g.T / 8)));
        double best_cost = 1e300;
        int best_nseg = lo;
        for (int nseg = lo; nseg <= hi; nseg++) {
            const int F = (g.T + nseg - 1) / nseg;
            if ((g.T + F - 1) / F != nseg) continue;
            const long long items = tiles_all * nseg;
            const long long rounds = (items + ncl - 1) / ncl;
            const double cost = (double)rounds * (F + 1 + 6);        // frames + the frame before + pipeline fill
            if (cost < best_cost - 1e-9) { best_cost = cost; best_nseg = nseg; }
        }
        f->F = (g.T + best_nseg - 1) / best_nseg;
    }
    f->nseg = (g.T + f->F - 1) / f->F;
    f->nitems = g.B * f->ntiles * f->nseg;
    f->ok = true;
}

int levels_of(int H, int W, int lv1, int* H1, int* W1, int* Hc, int* Wc) {
    int L = 1, h = H, w = W;
    *H1 = H; *W1 = W;
    while (std::max(h, w) > lv1) {
        h = (h + 1) / 2;
        w = (w + 1) / 2;
        if (L == 1) { *H1 = h; *W1 = w; }
        L++;
    }
    *Hc = h; *Wc = w;
    return L;
}

sttm_status make_plan(const sttm_params* p, Plan* pl, bool budget = false) {
    if (p == nullptr) return STTM_ERR_ARG;
    if (p->B < 1 || p->T < 1 || p->H < 1 || p->W < 1 || p->D < 1 || p->lv1 < 1) return STTM_ERR_ARG;
    if (p->D % 4 != 0) return STTM_ERR_ARG;
    if (p->in_dtype != STTM_BF16 && p->in_dtype != STTM_F32) return STTM_ERR_ARG;
    if (p->out_dtype != STTM_BF16 && p->out_dtype != STTM_F32) return STTM_ERR_ARG;
    if (p->match != STTM_MATCH_TOPLEFT && p->match != STTM_MATCH_BEST) return STTM_ERR_ARG;
    if (p->B > kMaxBatch) return STTM_ERR_UNSUPPORTED;
    if ((long long)p->B * p->T * p->H * p->W >= (1ll << 31)) return STTM_ERR_UNSUPPORTED;
    Geo& g = pl->g;
    g.B = p->B; g.T = p->T; g.H = p->H; g.W = p->W; g.D = p->D;
    g.L = levels_of(p->H, p->W, p->lv1, &g.H1, &g.W1, &g.Hc, &g.Wc);
    if (g.L > kMaxLevels) return STTM_ERR_UNSUPPORTED;
    pl->generic = g.L > 3;
    g.side = 1 << (g.L - 1);
    g.ncol = g.Hc * g.Wc;
    g.HW = p->H * p->W;
    g.N = p->T * g.HW;
    g.nsim = g.L == 1 ? 0 : (g.L == 2 ? g.HW : g.HW + g.H1 * g.W1);
    pl->cells = (long long)g.B * g.N;

    pl->nslice = (g.D + kSliceCh - 1) / kSliceCh;
    const long long per_chunk = (long long)g.B * g.ncol * pl->nslice;
    const long long target = 2ll * kSmCount * 16;       // (a fixed figure: the workspace layout must not depend on the device)
    long long nchunk = (target + per_chunk - 1) / per_chunk;
    nchunk = std::max(1ll, std::min<long long>(nchunk, std::max(1, g.T / 8)));
    pl->Tc = (int)((g.T + nchunk - 1) / nchunk);
    pl->nchunk = (g.T + pl->Tc - 1) / pl->Tc;
    const int NC = g.side * g.side;
    pl->partial_slots = pl->generic ? 0 : 2ll * NC * g.ncol * pl->nchunk * g.B;
    {
        Pyr& py = pl->py;
        py = Pyr{};
        py.L = g.L;
        int h = g.H, w = g.W, no = 0, uo = 0;
        for (int l = 0; l < g.L; l++) {
            py.H[l] = h; py.W[l] = w;
            py.noff[l] = no; no += h * w;
            py.uoff[l] = l == 0 ? 0 : uo;
            if (l >= 1) uo += h * w;
            h = (h + 1) / 2; w = (w + 1) / 2;
        }
        py.nodes = no; py.upper = uo;
    }

    const int NN = g.L == 3 ? 21 : (g.L == 2 ? 5 : 1);
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes); return at; };
    pl->norms_bytes = (size_t)g.B * g.T * g.ncol * NN * sizeof(float);
    pl->norms = take(pl->norms_bytes);
    pl->cover = take((size_t)pl->cells);
    pl->link = take((size_t)pl->cells * 4);
    pl->root = take((size_t)pl->cells * 4);
    pl->row_at_root = take((size_t)pl->cells * 4);
    pl->cell_row = take((size_t)pl->cells * 4);
    pl->row_anchor = take((size_t)pl->cells * 4);
    pl->span_off = take((size_t)pl->cells * 4);
    pl->frame_roots = take((size_t)g.B * g.T * 4);
    pl->frame_base = take((size_t)g.B * g.T * 4);
    pl->vid_off = take((size_t)(g.B + 1) * 8);
    pl->f.ok = false;
    pl->fl.ok = false;
    if (!pl->generic) {
        plan_flow(p, g, &pl->fl, budget);
        if (!pl->fl.ok) plan_fused(p, g, &pl->f);
    }
    const bool tiled = pl->fl.ok || pl->f.ok;
    // (one memset per call: everything that starts from zero lies together)
    pl->zero_begin = o;
    pl->frame_counts = take((size_t)g.B * g.T * 4);
    pl->row_weight = take((size_t)pl->cells * 4);
    pl->row_last_t = take((size_t)pl->cells * 4);
    pl->span_total = take(4);
    pl->status = take(4);
    pl->queue = take(4);
    pl->row_head = pl->flow_progress = o;
    if (tiled) pl->row_head = take((size_t)pl->cells * 4);
    if (pl->fl.ok) pl->flow_progress = take((size_t)pl->fl.nitems * 4);
    pl->zero_end = o;
    pl->partial = take(tiled ? 0 : (size_t)pl->partial_slots * g.D * sizeof(float));
    pl->gen_pooled = pl->gen_norms = pl->gen_dots = pl->gen_allpass = o;
    pl->gen_cnt = pl->gen_start = pl->gen_list = pl->gen_sorted = o;
    if (pl->generic) {
        const long long frames = (long long)g.B * g.T;
        pl->gen_pooled = take((size_t)frames * pl->py.upper * g.D * sizeof(float));
        pl->gen_norms = take((size_t)frames * pl->py.nodes * sizeof(float));
        pl->gen_dots = take((size_t)frames * pl->py.nodes * sizeof(float));
        pl->gen_allpass = take((size_t)frames * pl->py.nodes);
        pl->gen_cnt = take((size_t)pl->cells * 4);
        pl->gen_start = take(((size_t)pl->cells + 1) * 4);
        pl->gen_list = take((size_t)pl->cells * 4);
        pl->gen_sorted = take((size_t)pl->cells * 4);
    }
    pl->staging = pl->pieces = pl->piece_meta = o;
    pl->piece_row = pl->lead_n = pl->lead_ids = pl->lead_list = o;
    pl->flow_partial = pl->flow_hand = pl->flow_recs = o;
    if (pl->fl.ok) {
        const FlowPlan& f = pl->fl;
        pl->pieces = take((size_t)f.nitems * kPieceSlots * g.D * sizeof(float));
        pl->piece_meta = take((size_t)f.nitems * kPieceSlots * sizeof(int2));
        pl->piece_row = take((size_t)f.nitems * kPieceSlots * 4);
        pl->lead_n = take(((size_t)f.nitems * kPieceSlots + 1) * 4);
        pl->lead_list = take((size_t)f.nitems * kPieceSlots * 4);
        pl->lead_ids = take((size_t)f.nitems * kPieceSlots * kRowPieces * 4);
        pl->flow_partial = take((size_t)f.nitems * (f.F + 1) * f.NSg * kSumVals * sizeof(float));
        pl->flow_hand = take((size_t)f.nitems * (f.F + 1) * 16 * 4);
        pl->flow_recs = take((size_t)f.nitems * (f.F + 2) * sizeof(FrameRec));
    }
    if (pl->f.ok) {
        const size_t out_elt = p->out_dtype == STTM_BF16 ? 2 : 4;
        pl->staging = take((size_t)pl->cells * g.D * out_elt);
        pl->pieces = take((size_t)pl->f.nitems * kPieceSlots * g.D * sizeof(float));
        pl->piece_meta = take((size_t)pl->f.nitems * kPieceSlots * sizeof(int2));
        pl->piece_row = take((size_t)pl->f.nitems * kPieceSlots * 4);
        pl->lead_n = take(((size_t)pl->f.nitems * kPieceSlots + 1) * 4);
        pl->lead_list = take((size_t)pl->f.nitems * kPieceSlots * 4);
        pl->lead_ids = take((size_t)pl->f.nitems * kPieceSlots * kRowPieces * 4);
    }
    pl->total = o;
    return STTM_OK;
}

void fill_taus(const sttm_params* p, Taus* t) {
    for (int b = 0; b < p->B; b++) {
        t->s[b] = p->tau_s_per_video ? p->tau_s_per_video[b] : p->tau_s;
        t->t[b] = p->tau_t_per_video ? p->tau_t_per_video[b] : p->tau_t;
    }
}

template <typename F>
sttm_status by_levels_dtype(int L, sttm_dtype dt, F&& f) {
    if (dt == STTM_BF16) {
        if (L == 1) return f(std::integral_constant<int, 1>{}, (const __nv_bfloat16*)nullptr);
        if (L == 2) return f(std::integral_constant<int, 2>{}, (const __nv_bfloat16*)nullptr);
        return f(std::integral_constant<int, 3>{}, (const __nv_bfloat16*)nullptr);
    }
    if (L == 1) return f(std::integral_constant<int, 1>{}, (const float*)nullptr);
    if (L == 2) return f(std::integral_constant<int, 2>{}, (const float*)nullptr);
    return f(std::integral_constant<int, 3>{}, (const float*)nullptr);
}

#define STTM_CUDA_TRY(expr)                          \
    do {                                             \
        cudaError_t e_ = (expr);                     \
        if (e_ != cudaSuccess) return STTM_ERR_CUDA; \
    } while (0)

inline sttm_status launched() {
    g_launches++;
    return cudaPeekAtLastError() == cudaSuccess ? STTM_OK : STTM_ERR_CUDA;
}

// Launch with programmatic stream serialization: the kernel's blocks may be set up while the
// kernel before it in the stream drains; every kernel launched this way begins with
// wait_for_prior_kernel(), so it touches nothing before that kernel has completed.
template <typename... KArgs, typename... Args>
sttm_status launch_after(void (*kernel)(KArgs...), unsigned grid, unsigned block, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
    g_launches++;
    return e == cudaSuccess ? STTM_OK : STTM_ERR_CUDA;
}

inline unsigned blocks_for(long long items, int per_block) { return (unsigned)((items + per_block - 1) / per_block); }

sttm_status run_spatial(const void* feats, const sttm_params* p, const Plan& pl, float* norms, int8_t* cover,
                        int32_t* frame_counts, float* sims, cudaStream_t st) {
    Taus taus;
    fill_taus(p, &taus);
    const Geo g = pl.g;
    const long long warps = (long long)g.B * g.T * g.ncol;
    return by_levels_dtype(g.L, p->in_dtype, [&](auto lv, auto* tag) {
        using T = std::remove_const_t<std::remove_pointer_t<decltype(tag)>>;
        k_spatial<decltype(lv)::value, T><<<blocks_for(warps, kWarpsPerBlock), kWarpsPerBlock * 32, 0, st>>>(
            (const T*)feats, g, taus, cover, frame_counts, sims, norms);
        return launched();
    });
}

sttm_status run_temporal(const void* feats, const sttm_params* p, const Plan& pl, char* ws, const int8_t* cover,
                         int32_t* link, int32_t* root, float* tsim, int32_t* status, cudaStream_t st) {
    Taus taus;
    fill_taus(p, &taus);
    const Geo g = pl.g;
    const float* norms = (const float*)(ws + pl.norms);
    const long long warps = (long long)g.B * g.T * g.ncol;
    int max_rounds = 2;
    while ((1 << (max_rounds - 2)) < g.T) max_rounds++;
    return by_levels_dtype(g.L, p->in_dtype, [&](auto lv, auto* tag) {
        using T = std::remove_const_t<std::remove_pointer_t<decltype(tag)>>;
        constexpr int LV = decltype(lv)::value;
        k_temporal<LV, T><<<blocks_for(warps, kWarpsPerBlock), kWarpsPerBlock * 32, 0, st>>>(
            (const T*)feats, g, taus, cover, norms, link, tsim, p->match == STTM_MATCH_BEST ? 1 : 0);
        sttm_status s = launched();
        if (s != STTM_OK) return s;
        k_roots<LV><<<g.B * g.ncol, 256, 0, st>>>(g, cover, link, root, status, max_rounds);
        return launched();
    });
}

template <int LV, typename T, typename OutT>
sttm_status launch_accumulate(const void* feats, const Plan& pl, char* ws, void* out, long long capacity,
                              int weight_mode, cudaStream_t st) {
    const Geo g = pl.g;
    const size_t smem = (size_t)kAccWarps * Col<LV>::NC * kSliceCh * sizeof(float);
    static bool configured[kMaxDevices] = {};
    const int dev = device_slot();
    if (dev < 0) return STTM_ERR_UNSUPPORTED;
    if (!configured[dev]) {
        STTM_CUDA_TRY(cudaFuncSetAttribute(k_accumulate<LV, T, OutT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)smem));
        configured[dev] = true;
    }
    const long long warps = (long long)g.B * g.ncol * pl.nchunk * pl.nslice;
    k_accumulate<LV, T, OutT><<<blocks_for(warps, kAccWarps), kAccWarps * 32, smem, st>>>(
        (const T*)feats, g, pl.Tc, pl.nchunk, pl.nslice, (const int8_t*)(ws + pl.cover),
        (const int32_t*)(ws + pl.cell_row), (const int32_t*)(ws + pl.row_weight),
        (const int32_t*)(ws + pl.span_off), (const int32_t*)(ws + pl.row_anchor), (float*)(ws + pl.partial),
        (OutT*)out, capacity, weight_mode);
    sttm_status s = launched();
    if (s != STTM_OK) return s;
    mark_stage(4, st);
    k_combine<OutT><<<sm_count() * 2, 256, 0, st>>>(g, pl.Tc, (const long long*)(ws + pl.vid_off),
                                                 (const int32_t*)(ws + pl.span_off),
                                                 (const int32_t*)(ws + pl.row_anchor),
                                                 (const int32_t*)(ws + pl.row_last_t),
                                                 (const int32_t*)(ws + pl.row_weight),
                                                 (const float*)(ws + pl.partial), (OutT*)out, capacity);
    s = launched();
    mark_stage(5, st);
    return s;
}

// Resident clusters of the fused kernel for a launch shape (cached); falls back to SMs / C.
int fused_resident_clusters(const FusedPlan& f) {
    static int cached[kMaxDevices][kMaxCluster + 1][kFusedMaxThreads / 32 + 1];
    static size_t cached_smem[kMaxDevices][kMaxCluster + 1][kFusedMaxThreads / 32 + 1];
    const int warps = f.NM + kCombineWarps + f.NA + kTailWarps;
    const int dev = device_slot();
    if (dev < 0) return sm_count() / f.C;
    int& slot = cached[dev][f.C][warps];
    if (slot > 0 && cached_smem[dev][f.C][warps] == f.smem) return slot;
    int n = 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sm_count() / f.C * f.C);
    cfg.blockDim = dim3(warps * 32);
    cfg.dynamicSmemBytes = f.smem;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = f.C; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    cudaFuncSetAttribute(k_fused<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem);
    if (cudaOccupancyMaxActiveClusters(&n, k_fused<true, false>, &cfg) != cudaSuccess || n < 1) {
        cudaGetLastError();
        n = sm_count() / f.C;
    }
    slot = n;
    cached_smem[dev][f.C][warps] = f.smem;
    return n;
}

sttm_status run_fused(const void* feats, const sttm_params* p, const Plan& pl, char* ws, int32_t* device_status,
                      const Internal& in, cudaStream_t st) {
    const Geo g = pl.g;
    const FusedPlan& f = pl.f;
    static bool configured[kMaxDevices] = {};
    const int dev = device_slot();
    if (dev < 0) return STTM_ERR_UNSUPPORTED;
    if (!configured[dev]) {
        STTM_CUDA_TRY(cudaFuncSetAttribute(k_fused<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem));
        STTM_CUDA_TRY(cudaFuncSetAttribute(k_fused<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem));
        STTM_CUDA_TRY(cudaFuncSetAttribute(k_fused<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem));
        STTM_CUDA_TRY(cudaFuncSetAttribute(k_fused<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmem));
        configured[dev] = true;
    }
    FusedParams fp = {};
    fp.feats = (const __nv_bfloat16*)feats;
    fp.B = g.B; fp.T = g.T; fp.H = g.H; fp.W = g.W; fp.D = g.D; fp.L = g.L;
    fp.HW = g.HW; fp.N = g.N;
    fp.Wt = f.Wt; fp.ntiles = f.ntiles;
    fp.C = f.C; fp.S = f.S; fp.NM = f.NM; fp.NA = f.NA;
    fp.row_bytes = f.row_bytes; fp.slot_bytes = f.slot_bytes; fp.R = f.R; fp.RB = f.RB; fp.lead = f.lead;
    fp.F = f.F; fp.nseg = f.nseg; fp.nitems = f.nitems;
    fp.weight_mode = (int)p->wt;
    fp.match_best = p->match == STTM_MATCH_BEST ? 1 : 0;
    fp.out_f32 = p->out_dtype == STTM_F32;
    fp.cover = (int8_t*)(ws + pl.cover);
    fp.link = (int32_t*)(ws + pl.link);
    fp.tmax = in.tmax;
    fp.tau_t_dev = in.tau_dev;
    fp.frame_roots = (int32_t*)(ws + pl.frame_counts);   // inside the region that is cleared before every call
    fp.chain_key = (int32_t*)(ws + pl.cell_row);       // the three-pass kernels' cell_row array is free here
    fp.staging = ws + pl.staging;
    fp.pieces = (float*)(ws + pl.pieces);
    fp.piece_meta = (int2*)(ws + pl.piece_meta);
    fp.status = device_status;
    std::memcpy(fp.tiles, f.tiles, sizeof(fp.tiles));
    Taus taus;
    fill_taus(p, &taus);

    const int nclusters = std::min(f.nitems, fused_resident_clusters(f));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(nclusters * f.C);
    cfg.blockDim = dim3((f.NM + kCombineWarps + f.NA + kTailWarps) * 32);
    cfg.dynamicSmemBytes = f.smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = f.C; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    const bool lean = fp.tmax == nullptr && fp.tau_t_dev == nullptr && fp.RB == 0 && !fp.out_f32 && !fp.match_best;
    const bool flagship = fp.C == kFlagshipC && fp.S == kFlagshipS && fp.NM == kFlagshipNM && fp.NA == kFlagshipNA && fp.L == 3 &&
                          fp.D == kFlagshipC * kFlagshipS;
    if (flagship && lean) STTM_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_fused<true, true>, fp, taus));
    else if (flagship) STTM_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_fused<false, true>, fp, taus));
    else if (lean) STTM_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_fused<true, false>, fp, taus));
    else STTM_CUDA_TRY(cudaLaunchKernelEx(&cfg, k_fused<false, false>, fp, taus));
    g_launches++;
    return STTM_OK;
}

// launch with programmatic stream serialization and dynamic shared memory
template <typename... KArgs, typename... Args>
sttm_status launch_after_smem(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, bool after,
                              cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = after ? 1 : 0;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
    g_launches++;
    return e == cudaSuccess ? STTM_OK : STTM_ERR_CUDA;
}

// Ordering: rows of the surviving tokens from the per-frame counts.  Up to kRowsScanFrames frames every
// block of the row kernel adds up the counts before its own frame itself; beyond that the counts are
// scanned once by a kernel of their own.
constexpr long long kRowsScanFrames = 4096;
sttm_status launch_ordering(const Plan& pl, const sttm_params* p, char* ws, const int8_t* cover, const int32_t* link,
                            int32_t* out_pos, int32_t* out_count, int64_t* out_offsets, int32_t* device_status,
                            cudaStream_t st) {
    const Geo g = pl.g;
    const int32_t* frame_roots = (const int32_t*)(ws + pl.frame_counts);
    int32_t* frame_base = (int32_t*)(ws + pl.frame_base);
    long long* vid_off = (long long*)(ws + pl.vid_off);
    int32_t* row_at_root = (int32_t*)(ws + pl.row_at_root);
    int32_t* row_anchor = (int32_t*)(ws + pl.row_anchor);
    if ((long long)g.B * g.T <= kRowsScanFrames)
        return launch_after(k_rows_scan, (unsigned)(g.B * g.T), 256, st, g, cover, link, frame_roots, out_count, vid_off,
                            out_offsets, row_at_root, row_anchor, out_pos, (long long)p->out_capacity_rows, (int)p->pos,
                            device_status);
    sttm_status s = launch_after(k_scan_frames, 1u, 1024, st, g, frame_roots, frame_base, out_count, vid_off, out_offsets);
    if (s != STTM_OK) return s;
    return launch_after(k_rows, (unsigned)(g.B * g.T), 256, st, g, cover, link, (const int32_t*)frame_base,
                        (const long long*)vid_off, row_at_root, row_anchor, out_pos, (long long)p->out_capacity_rows,
                        (int)p->pos, device_status);
}

// Chains cut by item borders: rows, leaders and lists of the pieces, then the rows themselves.
template <typename OutT>
sttm_status launch_pieces(const Plan& pl, int npieces, char* ws, void* out, long long capacity, int32_t* status,
                          cudaStream_t st) {
    const Geo g = pl.g;
    sttm_status s = launch_after(k_piece_link, blocks_for(npieces, 256), 256, st, g, npieces,
                                 (pl.fl.ok ? pl.fl.nseg : pl.f.nseg) + 1,
                                 (const int2*)(ws + pl.piece_meta), (const int32_t*)(ws + pl.cell_row),
                                 (const int32_t*)(ws + pl.row_at_root), (const long long*)(ws + pl.vid_off),
                                 (int32_t*)(ws + pl.row_head), (int32_t*)(ws + pl.piece_row), (int32_t*)(ws + pl.lead_n),
                                 (int32_t*)(ws + pl.row_weight), status);
    if (s != STTM_OK) return s;
    s = launch_after(k_piece_group, blocks_for(npieces, 256), 256, st, npieces, (const int32_t*)(ws + pl.piece_row),
                     (const int32_t*)(ws + pl.row_head), (int32_t*)(ws + pl.lead_n), (int32_t*)(ws + pl.lead_ids),
                     (int32_t*)(ws + pl.lead_list));
    if (s != STTM_OK) return s;
    const unsigned blocks = std::min<unsigned>(blocks_for((long long)npieces * kPieceParts, 8), sm_count() * 3);
    return launch_after(k_gather_pieces<OutT>, blocks, 256, st, g, npieces, (const int32_t*)(ws + pl.piece_row),
                        (const int32_t*)(ws + pl.lead_n), (const int32_t*)(ws + pl.lead_ids),
                        (const int32_t*)(ws + pl.lead_list),
                        (const int32_t*)(ws + pl.row_weight), (const float*)(ws + pl.pieces), (OutT*)out, capacity);
}

// Tensor maps of the feature tensor for the three kinds of tile.  The tensor is described as
// [frame][64-channel block][y][x][64 channels] (a permutation of its dimensions in memory), so that
// a box of NB blocks x (4x4 | 16x1 | 1x16) cells lands in shared memory block by block, each block
// 16 rows of 128 bytes under the 128-byte swizzle.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// the driver's tensor-map encoder, through the runtime (no link against libcuda); null when it is not there
EncodeTiledFn tensor_map_encoder() {
    static EncodeTiledFn encode = nullptr;
    if (encode == nullptr) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            encode = (EncodeTiledFn)fn;
    }
    return encode;
}

sttm_status make_flow_maps(const void* feats, const Geo& g, int NB, FlowMaps* maps) {
    const EncodeTiledFn encode = tensor_map_encoder();
    if (encode == nullptr) return STTM_ERR_CUDA;
    const cuuint64_t dims[5] = {64, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)(g.D / 64), (cuuint64_t)g.B * g.T};
    const cuuint64_t strides[4] = {(cuuint64_t)g.D * 2, (cuuint64_t)g.W * g.D * 2, 128, (cuuint64_t)g.HW * g.D * 2};
    const cuuint32_t ones[5] = {1, 1, 1, 1, 1};
    const cuuint32_t boxes[3][5] = {{64, 4, 4, (cuuint32_t)NB, 1}, {64, 1, 16, (cuuint32_t)NB, 1}, {64, 16, 1, (cuuint32_t)NB, 1}};
    for (int k = 0; k < 3; k++) {
        const CUresult r = encode(&maps->m[k], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(feats), dims, strides,
                                  boxes[k], ones, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return STTM_ERR_CUDA;
    }
    return STTM_OK;
}

// The same tensor with the frame axis inside the block axis: a box of five frames and NB blocks lands as
// [block][frame][cell][64 channels], 80 rows of 128 bytes per block (the operand layout of k_flow_gram_tc).
sttm_status make_gram_tc_maps(const void* feats, const Geo& g, int NB, FlowMaps* maps) {
    const EncodeTiledFn encode = tensor_map_encoder();
    if (encode == nullptr) return STTM_ERR_CUDA;
    const cuuint64_t dims[5] = {64, (cuuint64_t)g.W, (cuuint64_t)g.H, (cuuint64_t)g.B * g.T, (cuuint64_t)(g.D / 64)};
    const cuuint64_t strides[4] = {(cuuint64_t)g.D * 2, (cuuint64_t)g.W * g.D * 2, (cuuint64_t)g.HW * g.D * 2, 128};
    const cuuint32_t ones[5] = {1, 1, 1, 1, 1};
    const cuuint32_t fr = kTcBoxFrames;
    const cuuint32_t boxes[3][5] = {{64, 4, 4, fr, (cuuint32_t)NB}, {64, 1, 16, fr, (cuuint32_t)NB}, {64, 16, 1, fr, (cuuint32_t)NB}};
    for (int k = 0; k < 3; k++) {
        const CUresult r = encode(&maps->m[k], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(feats), dims, strides,
                                  boxes[k], ones, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return STTM_ERR_CUDA;
    }
    return STTM_OK;
}

// The two-stream path: Gram stage, decisions, ordering, chain stage, sum stage, pieces.
sttm_status run_flow(const void* feats, const sttm_params* p, const Plan& pl, char* ws, void* out_feats,
                     int32_t* out_pos, int32_t* merge_map, int32_t* out_count, int64_t* out_offsets,
                     int32_t* device_status, const Internal& in, cudaStream_t st) {
    const Geo g = pl.g;
    const FlowPlan& f = pl.fl;
    static bool configured[kMaxDevices] = {};
    const int dev = device_slot();
    if (dev < 0) return STTM_ERR_UNSUPPORTED;
    if (!configured[dev]) {
        STTM_CUDA_TRY(cudaFuncSetAttribute(k_flow<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFlowSmemMax));
        STTM_CUDA_TRY(cudaFuncSetAttribute(k_flow<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFlowSmemMax));
        STTM_CUDA_TRY(cudaFuncSetAttribute(k_flow_gram_tc, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)tc_smem_bytes(kTcMaxNB)));
        configured[dev] = true;
    }
    FlowMaps maps;
    sttm_status s = make_flow_maps(feats, g, f.NB, &maps);
    if (s != STTM_OK) return s;
    FlowParams fp = {};
    fp.B = g.B; fp.T = g.T; fp.H = g.H; fp.W = g.W; fp.D = g.D; fp.L = g.L;
    fp.HW = g.HW; fp.N = g.N;
    fp.ntiles = f.ntiles;
    fp.NS = f.NS; fp.NB = f.NB;
    fp.NSg = f.NSg; fp.NBg = f.NBg; fp.NCg = f.NCg;
    fp.slot_bytes = f.slot_bytes; fp.R = f.R;
    fp.F = f.F; fp.nseg = f.nseg; fp.nitems = f.nitems;
    fp.weight_mode = (int)p->wt;
    fp.match_best = p->match == STTM_MATCH_BEST ? 1 : 0;
    fp.out_f32 = p->out_dtype == STTM_F32;
    fp.cover = (int8_t*)(ws + pl.cover);
    fp.link = (int32_t*)(ws + pl.link);
    fp.tmax = in.tmax;
    fp.tau_t_dev = in.tau_dev;
    fp.frame_roots = (int32_t*)(ws + pl.frame_counts);   // inside the region that is cleared before every call
    fp.chain_key = (int32_t*)(ws + pl.cell_row);
    fp.partial = (float*)(ws + pl.flow_partial);
    fp.hand = (int32_t*)(ws + pl.flow_hand);
    fp.recs = (FrameRec*)(ws + pl.flow_recs);
    fp.progress = (int32_t*)(ws + pl.flow_progress);
    fp.row_at_root = (const int32_t*)(ws + pl.row_at_root);
    fp.vid_off = (const long long*)(ws + pl.vid_off);
    fp.out = out_feats;
    fp.capacity = p->out_capacity_rows;
    fp.pieces = (float*)(ws + pl.pieces);
    fp.piece_meta = (int2*)(ws + pl.piece_meta);
    fp.status = device_status;
    std::memcpy(fp.tiles, f.tiles, sizeof(fp.tiles));
    std::memcpy(fp.boxes, f.boxes, sizeof(fp.boxes));
    Taus taus;
    fill_taus(p, &taus);

    const int ntasks = f.nitems * f.NS;
    const unsigned grid = (unsigned)std::min(ntasks, 2 * sm_count());
    mark_stage(0, st);
    if (!in.second_pass && f.tc) {
        FlowMaps gmaps;
        s = make_gram_tc_maps(feats, g, f.NBg, &gmaps);
        if (s != STTM_OK) return s;
        const unsigned ggrid = (unsigned)std::min(f.nitems * f.NSg, sm_count());
        s = launch_after_smem(k_flow_gram_tc, ggrid, kTcThreads, f.smem_tc, false, st, fp, gmaps);
        if (s != STTM_OK) return s;
    } else if (!in.second_pass) {
        s = launch_after_smem(k_flow<false>, grid, kFlowThreads, f.smem, false, st, fp, maps);
        if (s != STTM_OK) return s;
    }
    mark_stage(1, st);
    const int pairs = (f.F + 2) / 2;
    s = launch_after(k_flow_decide, blocks_for((long long)f.nitems * pairs, 8), 256, st, fp, taus);
    if (s != STTM_OK) return s;
    int32_t* row_at_root = (int32_t*)(ws + pl.row_at_root);
    int32_t* root = (int32_t*)(ws + pl.root);
    if (in.tmax != nullptr)                            // first pass of the budget mode: only the node counts are needed
        return launch_after(k_scan_frames, 1u, 1024, st, g, (const int32_t*)(ws + pl.frame_counts),
                            (int32_t*)(ws + pl.frame_base), out_count, (long long*)(ws + pl.vid_off), out_offsets);
    s = launch_ordering(pl, p, ws, (const int8_t*)fp.cover, (const int32_t*)fp.link, out_pos, out_count, out_offsets,
                        device_status, st);
    if (s != STTM_OK) return s;
    s = launch_after(k_flow_chain, blocks_for(f.nitems, kChainWarps), kChainWarps * 32, st, fp);
    if (s != STTM_OK) return s;
    mark_stage(2, st);
    s = launch_after_smem(k_flow<true>, grid, kFlowThreads, f.smem, true, st, fp, maps);
    if (s != STTM_OK) return s;
    mark_stage(3, st);
    if (merge_map != nullptr) {
        s = launch_after(k_resolve_roots, blocks_for(pl.cells, 256), 256, st, g, f.nseg + 1,
                         (const int32_t*)(ws + pl.cell_row), root, device_status);
        if (s != STTM_OK) return s;
        s = launch_after(k_merge_map, blocks_for(pl.cells, 256), 256, st, g, (const int32_t*)root,
                         (const int32_t*)row_at_root, merge_map);
        if (s != STTM_OK) return s;
    }
    const int npieces = f.nitems * kPieceSlots;
    s = p->out_dtype == STTM_BF16 ? launch_pieces<__nv_bfloat16>(pl, npieces, ws, out_feats, p->out_capacity_rows, device_status, st)
                                  : launch_pieces<float>(pl, npieces, ws, out_feats, p->out_capacity_rows, device_status, st);
    mark_stage(4, st);
    mark_stage(5, st);
    return s;
}

template <typename OutT>
sttm_status launch_gather(const Plan& pl, char* ws, void* out, long long capacity, int32_t* status, cudaStream_t st) {
    const Geo g = pl.g;
    // kGatherParts warps per row, striding; the row count is only known on the device, so the grid
    // covers the most rows there can be, up to a few waves of blocks (most tokens merge: few rows,
    // and blocks without a row would only cost their launch)
    const long long max_rows = std::min<long long>(pl.cells, std::max<long long>(capacity, 1));
    const unsigned blocks = std::min<unsigned>(blocks_for(max_rows * kGatherParts, 8), sm_count() * 16);
    // (first the rows made of pieces: the copy below leaves out the rows that have a leader piece)
    sttm_status s = launch_pieces<OutT>(pl, pl.f.nitems * kPieceSlots, ws, out, capacity, status, st);
    if (s != STTM_OK) return s;
    s = launch_after(k_gather_rows<OutT>, blocks, 256, st, g, (const long long*)(ws + pl.vid_off),
                                 (const int32_t*)(ws + pl.row_anchor), (const int32_t*)(ws + pl.row_head),
                                 (const OutT*)(ws + pl.staging), (OutT*)out, capacity);
    return s;
}

template <typename T, typename OutT>
sttm_status run_generic(const T* feats, const sttm_params* p, const Plan& pl, char* ws, OutT* out_feats,
                        int32_t* out_pos, int32_t* merge_map, int32_t* out_count, int64_t* out_offsets,
                        int32_t* device_status, cudaStream_t st) {
    const Geo g = pl.g;
    const Pyr py = pl.py;
    Taus taus;
    fill_taus(p, &taus);
    float* pooled = (float*)(ws + pl.gen_pooled);
    float* norms = (float*)(ws + pl.gen_norms);
    float* dots = (float*)(ws + pl.gen_dots);
    int8_t* allpass = (int8_t*)(ws + pl.gen_allpass);
    int32_t* cnt = (int32_t*)(ws + pl.gen_cnt);
    int32_t* start = (int32_t*)(ws + pl.gen_start);
    int32_t* list = (int32_t*)(ws + pl.gen_list);
    int32_t* sorted = (int32_t*)(ws + pl.gen_sorted);
    int8_t* cover = (int8_t*)(ws + pl.cover);
    int32_t* link = (int32_t*)(ws + pl.link);
    int32_t* root = (int32_t*)(ws + pl.root);
    const long long frames = (long long)g.B * g.T;
    const long long rows = std::min<long long>(pl.cells, std::max<long long>(p->out_capacity_rows, 1));
    sttm_status s;
    STTM_CUDA_TRY(cudaMemsetAsync(link, 0xff, (size_t)pl.cells * 4, st));
    STTM_CUDA_TRY(cudaMemsetAsync(cnt, 0, (size_t)pl.cells * 4, st));
    // (the general kernels serve quadtrees of four levels and more: levels 1 and 2 come from one pass)
    k_gen_pool2<T><<<blocks_for(frames * py.H[2] * py.W[2] * 32, 128), 128, 0, st>>>(feats, pooled, g, py, norms, dots);
    if ((s = launched()) != STTM_OK) return s;
    for (int l = 3; l < py.L; l++) {
        k_gen_pool<T><<<blocks_for(frames * py.H[l] * py.W[l] * 32, 256), 256, 0, st>>>(feats, pooled, g, py, l, norms,
                                                                                       dots);
        if ((s = launched()) != STTM_OK) return s;
    }
    k_gen_allpass<<<blocks_for(frames * py.nodes, 256), 256, 0, st>>>(g, py, taus, norms, dots, allpass);
    if ((s = launched()) != STTM_OK) return s;
    k_gen_cover<<<blocks_for(pl.cells, 256), 256, 0, st>>>(g, py, allpass, cover);
    if ((s = launched()) != STTM_OK) return s;
    k_gen_temporal<T><<<blocks_for(pl.cells * 32, 256), 256, 0, st>>>(feats, pooled, g, py, taus, cover, norms, link,
                                                                     p->match == STTM_MATCH_BEST ? 1 : 0);
    if ((s = launched()) != STTM_OK) return s;
    k_gen_root_init<<<blocks_for(pl.cells, 256), 256, 0, st>>>(g, cover, link, root);
    if ((s = launched()) != STTM_OK) return s;
    int rounds = 1;
    while ((1 << rounds) < g.T) rounds++;
    for (int r = 0; r <= rounds; r++) {
        k_gen_root_jump<<<blocks_for(pl.cells, 256), 256, 0, st>>>(g, root);
        if ((s = launched()) != STTM_OK) return s;
    }
    k_gen_root_fill<<<blocks_for(pl.cells, 256), 256, 0, st>>>(g, cover, root);
    if ((s = launched()) != STTM_OK) return s;

    int32_t* frame_roots = (int32_t*)(ws + pl.frame_roots);
    int32_t* frame_base = (int32_t*)(ws + pl.frame_base);
    long long* vid_off = (long long*)(ws + pl.vid_off);
    int32_t* row_at_root = (int32_t*)(ws + pl.row_at_root);
    int32_t* row_anchor = (int32_t*)(ws + pl.row_anchor);
    k_frame_roots<<<g.B * g.T, 256, 0, st>>>(g, cover, link, frame_roots);
    if ((s = launched()) != STTM_OK) return s;
    k_scan_frames<<<1, 1024, 0, st>>>(g, frame_roots, frame_base, out_count, vid_off, out_offsets);
    if ((s = launched()) != STTM_OK) return s;
    k_rows<<<g.B * g.T, 256, 0, st>>>(g, cover, link, frame_base, vid_off, row_at_root, row_anchor, out_pos,
                                      p->out_capacity_rows, (int)p->pos, device_status);
    if ((s = launched()) != STTM_OK) return s;
    k_members<<<blocks_for(pl.cells, 256), 256, 0, st>>>(g, cover, root, row_at_root, vid_off,
                                                        (int32_t*)(ws + pl.cell_row), merge_map,
                                                        (int32_t*)(ws + pl.row_weight),
                                                        (int32_t*)(ws + pl.row_last_t), (int)p->wt);
    if ((s = launched()) != STTM_OK) return s;
    const long long cap = p->out_capacity_rows;
    const int32_t* cell_row = (const int32_t*)(ws + pl.cell_row);
    k_gen_count<<<blocks_for(pl.cells, 256), 256, 0, st>>>(g, cover, cell_row, cnt, cap);
    if ((s = launched()) != STTM_OK) return s;
    k_gen_scan_rows<<<1, 1024, 0, st>>>(g, vid_off, cap, cnt, start);
    if ((s = launched()) != STTM_OK) return s;
    k_gen_fill<<<blocks_for(pl.cells, 256), 256, 0, st>>>(g, cover, cell_row, cnt, start, list, cap);
    if ((s = launched()) != STTM_OK) return s;
    k_gen_sort<<<blocks_for(rows * 32, 256), 256, 0, st>>>(g, vid_off, cap, start, list, sorted);
    if ((s = launched()) != STTM_OK) return s;
    k_gen_gather<T, OutT><<<blocks_for(rows * kGenParts * 32, 256), 256, 0, st>>>(
        feats, pooled, g, py, vid_off, cover, start, sorted, (const int32_t*)(ws + pl.row_weight), out_feats, cap,
        (int)p->wt);
    return launched();
}

bool misaligned(const void* p, size_t a) { return ((uintptr_t)p % a) != 0; }

// Scratch of sttm_spatial_static: lives in the library image, so every GPU that loads the
// library holds these bytes until the process exits.  In host code the name below is only a
// handle for the runtime, never an address a kernel may use; the device address comes from
// cudaGetSymbolAddress, asked once per device while that device is current.
constexpr size_t kStaticScratchBytes = STTM_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
void* g_static_scratch_addr[kMaxDevices] = {};

sttm_status static_scratch_address(void** out) {
    int dev = 0;
    STTM_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return STTM_ERR_UNSUPPORTED;
    if (g_static_scratch_addr[dev] == nullptr) {
        void* ptr = nullptr;
        STTM_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
        if (ptr == nullptr) return STTM_ERR_CUDA;
        g_static_scratch_addr[dev] = ptr;
    }
    *out = g_static_scratch_addr[dev];
    return STTM_OK;
}

// cached buffers for sttm_merge / sttm_merge_host, one set per device
struct Cache {
    void* ws = nullptr; size_t ws_bytes = 0;
    void* feats = nullptr; size_t feats_bytes = 0;
    void* out = nullptr; size_t out_bytes = 0;
    void* ints = nullptr; size_t ints_bytes = 0;   // pos, map, count, offsets, status
    int32_t* merge_status = nullptr;               // status word of sttm_merge
};
Cache g_cache[kMaxDevices];

sttm_status grow(void** ptr, size_t* have, size_t need) {
    if (*have >= need) return STTM_OK;
    if (*ptr) { STTM_CUDA_TRY(cudaFree(*ptr)); *ptr = nullptr; *have = 0; }
    STTM_CUDA_TRY(cudaMalloc(ptr, need));
    *have = need;
    return STTM_OK;
}

sttm_status merge_impl(const void* feats, const sttm_params* p, void* ws_, size_t ws_bytes, void* out_feats,
                       int32_t* out_pos, int32_t* merge_map, int32_t* out_count, int64_t* out_offsets,
                       int32_t* device_status, const Internal& in, void* stream);

}  // namespace

extern "C" {

const char* sttm_status_string(sttm_status s) {
    switch (s) {
        case STTM_OK: return "ok";
        case STTM_ERR_ARG: return "bad argument";
        case STTM_ERR_UNSUPPORTED: return "unsupported shape";
        case STTM_ERR_WORKSPACE: return "workspace too small";
        case STTM_ERR_CAPACITY: return "output capacity exceeded";
        case STTM_ERR_NOT_CONVERGED: return "root search did not converge";
        case STTM_ERR_CUDA: return "CUDA error";
        case STTM_ERR_TIMEOUT: return "a wait inside a kernel ran out";
    }
    return "unknown";
}

sttm_status sttm_status_from_bits(int32_t bits) {
    for (int code = STTM_ERR_ARG; code <= STTM_ERR_TIMEOUT; code++)
        if (bits & (1 << code)) return (sttm_status)code;
    return STTM_OK;
}

void sttm_default_params(sttm_params* p, int T, int H, int W, int D, float tau_s, float tau_t) {
    if (!p) return;
    std::memset(p, 0, sizeof(*p));
    p->B = 1; p->T = T; p->H = H; p->W = W; p->D = D;
    p->in_dtype = STTM_BF16; p->out_dtype = STTM_BF16;
    p->lv1 = 4;
    p->tau_s = tau_s; p->tau_t = tau_t;
    p->pos = STTM_POS_SURVIVED; p->wt = STTM_W_NODE; p->match = STTM_MATCH_TOPLEFT;
    p->out_capacity_rows = (long long)T * H * W;
}

size_t sttm_workspace_bytes(const sttm_params* p) {
    Plan pl;
    if (make_plan(p, &pl) != STTM_OK) return 0;
    return pl.total;
}

int sttm_sims_per_frame(int H, int W, int lv1) {
    if (H < 1 || W < 1 || lv1 < 1) return 0;
    int n = 0, h = H, w = W;
    while (std::max(h, w) > lv1) { n += h * w; h = (h + 1) / 2; w = (w + 1) / 2; }
    return n;
}

int sttm_last_launch_count(void) { return g_launches; }

int sttm_stage_count(void) { return kStageCount; }

const char* sttm_stage_name(int i) { return i >= 0 && i < kStageCount ? kStageNames[g_last_path][i] : ""; }

int sttm_last_path(void) { return g_last_path; }

int sttm_last_gram_stage(void) { return g_last_gram; }

int sttm_fused_launch_shape(const sttm_params* p, int* shape) {
    Plan pl;
    if (shape == nullptr || make_plan(p, &pl) != STTM_OK || !pl.f.ok) return 0;
    const FusedPlan& f = pl.f;
    const int resident = fused_resident_clusters(f);
    const int v[12] = {f.C, f.S, (f.NM + kCombineWarps + f.NA + kTailWarps) * 32, f.R, (int)f.smem, f.F, f.nitems, resident,
                       std::min(f.nitems, resident), f.NM, f.RB, f.lead};
    std::memcpy(shape, v, sizeof(v));
    return 1;
}

void sttm_set_stage_events(void** events) { g_stage_events = (cudaEvent_t*)events; }

void sttm_set_tuning(int path, int cluster_size, int frames_per_item) {
    g_tune_path = path == 3 ? 2 : path;
    g_tune_pack = path == 3 ? 1 : 0;
    g_tune_cluster = cluster_size;
    g_tune_seg = frames_per_item;
}

void sttm_set_ring_split(int sum_slots, int lead_frames) {
    g_tune_sum_slots = sum_slots;
    g_tune_lead = lead_frames;
}

sttm_status sttm_spatial(const void* feats, const sttm_params* p, void* ws, size_t ws_bytes,
                         int8_t* cover_level, int32_t* frame_counts, float* spatial_sims, void* stream) {
    Plan pl;
    sttm_status s = make_plan(p, &pl);
    if (s != STTM_OK) return s;
    if (pl.generic) return STTM_ERR_UNSUPPORTED;      // the stage calls cover up to three quadtree levels
    if (!feats || !ws || !cover_level || !frame_counts) return STTM_ERR_ARG;
    if (misaligned(feats, 16) || misaligned(ws, 256)) return STTM_ERR_ARG;
    if (ws_bytes < pl.total) return STTM_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    g_launches = 0;
    STTM_CUDA_TRY(cudaMemsetAsync(frame_counts, 0, (size_t)pl.g.B * pl.g.T * 4, st));
    return run_spatial(feats, p, pl, (float*)((char*)ws + pl.norms), cover_level, frame_counts, spatial_sims, st);
}

sttm_status sttm_spatial_static(const void* feats, const sttm_params* p, int8_t* cover_level, int32_t* frame_counts,
                                float* spatial_sims, void* stream) {
    Plan pl;
    sttm_status s = make_plan(p, &pl);
    if (s != STTM_OK) return s;
    if (pl.generic) return STTM_ERR_UNSUPPORTED;      // the stage calls cover up to three quadtree levels
    if (!feats || !cover_level || !frame_counts) return STTM_ERR_ARG;
    if (misaligned(feats, 16)) return STTM_ERR_ARG;
    // the only scratch of the spatial stage: one squared norm per quadtree node
    if (pl.norms_bytes > kStaticScratchBytes) return STTM_ERR_WORKSPACE;
    void* scratch = nullptr;
    if ((s = static_scratch_address(&scratch)) != STTM_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    g_launches = 0;
    // the counts are added to, so they start at zero; the norms are overwritten, nothing of an
    // earlier call is read
    STTM_CUDA_TRY(cudaMemsetAsync(frame_counts, 0, (size_t)pl.g.B * pl.g.T * 4, st));
    return run_spatial(feats, p, pl, (float*)scratch, cover_level, frame_counts, spatial_sims, st);
}

sttm_status sttm_temporal(const void* feats, const sttm_params* p, void* ws, size_t ws_bytes,
                          const int8_t* cover_level, int32_t* link, int32_t* root, float* temporal_sims,
                          int32_t* device_status, void* stream) {
    Plan pl;
    sttm_status s = make_plan(p, &pl);
    if (s != STTM_OK) return s;
    if (pl.generic) return STTM_ERR_UNSUPPORTED;      // the stage calls cover up to three quadtree levels
    if (!feats || !ws || !cover_level || !link || !root) return STTM_ERR_ARG;
    if (misaligned(feats, 16) || misaligned(ws, 256)) return STTM_ERR_ARG;
    if (ws_bytes < pl.total) return STTM_ERR_WORKSPACE;
    g_launches = 0;
    return run_temporal(feats, p, pl, (char*)ws, cover_level, link, root, temporal_sims, device_status,
                        (cudaStream_t)stream);
}

sttm_status sttm_merge_ex(const void* feats, const sttm_params* p, void* ws_, size_t ws_bytes, void* out_feats,
                          int32_t* out_pos, int32_t* merge_map, int32_t* out_count, int64_t* out_offsets,
                          int32_t* device_status, void* stream) {
    const sttm_status s = merge_impl(feats, p, ws_, ws_bytes, out_feats, out_pos, merge_map, out_count, out_offsets,
                                     device_status, Internal(), stream);
    close_stage_range();
    return s;
}

}  // extern "C"

namespace {

// The whole path; `in` carries what the budget mode adds to its two passes.
sttm_status merge_impl(const void* feats, const sttm_params* p, void* ws_, size_t ws_bytes, void* out_feats,
                       int32_t* out_pos, int32_t* merge_map, int32_t* out_count, int64_t* out_offsets,
                       int32_t* device_status, const Internal& in, void* stream) {
    Plan pl;
    sttm_status s = make_plan(p, &pl, in.budget);
    if (s != STTM_OK) return s;
    if (!feats || !ws_ || !out_feats || !out_pos || !out_count) return STTM_ERR_ARG;
    if (p->out_capacity_rows < 0) return STTM_ERR_ARG;
    if (misaligned(feats, 16) || misaligned(ws_, 256) || misaligned(out_feats, 16)) return STTM_ERR_ARG;
    if (ws_bytes < pl.total) return STTM_ERR_WORKSPACE;
    char* ws = (char*)ws_;
    cudaStream_t st = (cudaStream_t)stream;
    const Geo g = pl.g;
    g_launches = 0;

    STTM_CUDA_TRY(cudaMemsetAsync(ws + pl.zero_begin, 0, pl.zero_end - pl.zero_begin, st));
    int8_t* cover = (int8_t*)(ws + pl.cover);
    int32_t* link = (int32_t*)(ws + pl.link);
    int32_t* root = (int32_t*)(ws + pl.root);
    g_last_path = pl.generic ? 2 : (pl.fl.ok ? 3 : (pl.f.ok ? 1 : 0));
    g_last_gram = !pl.generic && pl.fl.ok ? (pl.fl.tc ? 2 : 1) : 0;
    if (pl.generic) {
        // more than three quadtree levels: the plain kernels, no stage breakdown
        for (int i = 0; i <= 4; i++) mark_stage(i, st);
        if (p->in_dtype == STTM_BF16)
            s = p->out_dtype == STTM_BF16
                    ? run_generic((const __nv_bfloat16*)feats, p, pl, ws, (__nv_bfloat16*)out_feats, out_pos, merge_map,
                                  out_count, out_offsets, device_status, st)
                    : run_generic((const __nv_bfloat16*)feats, p, pl, ws, (float*)out_feats, out_pos, merge_map,
                                  out_count, out_offsets, device_status, st);
        else
            s = p->out_dtype == STTM_BF16
                    ? run_generic((const float*)feats, p, pl, ws, (__nv_bfloat16*)out_feats, out_pos, merge_map,
                                  out_count, out_offsets, device_status, st)
                    : run_generic((const float*)feats, p, pl, ws, (float*)out_feats, out_pos, merge_map, out_count,
                                  out_offsets, device_status, st);
        mark_stage(5, st);
        return s;
    }
    if (pl.fl.ok) {
        return run_flow(feats, p, pl, ws, out_feats, out_pos, merge_map, out_count, out_offsets, device_status, in, st);
    }
    if (pl.f.ok) {
        // single-read path: fused kernel, roots, ordering, gather
        mark_stage(0, st);
        s = run_fused(feats, p, pl, ws, device_status, in, st);
        if (s != STTM_OK) return s;
        mark_stage(1, st);
        if (in.tmax != nullptr) {
            // first pass of the budget mode: only the node counts per video are needed
            return launch_after(k_scan_frames, 1u, 1024, st, g, (const int32_t*)(ws + pl.frame_counts),
                                (int32_t*)(ws + pl.frame_base), out_count, (long long*)(ws + pl.vid_off), out_offsets);
        }
        mark_stage(2, st);
        s = launch_ordering(pl, p, ws, (const int8_t*)cover, (const int32_t*)link, out_pos, out_count, out_offsets,
                            device_status, st);
        if (s != STTM_OK) return s;
        if (merge_map != nullptr) {
            s = launch_after(k_resolve_roots, blocks_for(pl.cells, 256), 256, st, g, pl.f.nseg + 1,
                             (const int32_t*)(ws + pl.cell_row), root, device_status);
            if (s != STTM_OK) return s;
            s = launch_after(k_merge_map, blocks_for(pl.cells, 256), 256, st, g, (const int32_t*)root,
                             (const int32_t*)(ws + pl.row_at_root), merge_map);
            if (s != STTM_OK) return s;
        }
        mark_stage(3, st);
        s = p->out_dtype == STTM_BF16 ? launch_gather<__nv_bfloat16>(pl, ws, out_feats, p->out_capacity_rows, device_status, st)
                                      : launch_gather<float>(pl, ws, out_feats, p->out_capacity_rows, device_status, st);
        mark_stage(4, st);
        mark_stage(5, st);
        return s;
    }
    mark_stage(0, st);
    s = run_spatial(feats, p, pl, (float*)(ws + pl.norms), cover, (int32_t*)(ws + pl.frame_counts), nullptr, st);
    if (s != STTM_OK) return s;
    mark_stage(1, st);
    s = run_temporal(feats, p, pl, ws, cover, link, root, nullptr, device_status, st);
    if (s != STTM_OK) return s;
    mark_stage(2, st);

    int32_t* frame_roots = (int32_t*)(ws + pl.frame_roots);
    int32_t* frame_base = (int32_t*)(ws + pl.frame_base);
    long long* vid_off = (long long*)(ws + pl.vid_off);
    int32_t* row_at_root = (int32_t*)(ws + pl.row_at_root);
    int32_t* row_anchor = (int32_t*)(ws + pl.row_anchor);
    k_frame_roots<<<g.B * g.T, 256, 0, st>>>(g, cover, link, frame_roots);
    if ((s = launched()) != STTM_OK) return s;
    k_scan_frames<<<1, 1024, 0, st>>>(g, frame_roots, frame_base, out_count, vid_off, out_offsets);
    if ((s = launched()) != STTM_OK) return s;
    k_rows<<<g.B * g.T, 256, 0, st>>>(g, cover, link, frame_base, vid_off, row_at_root, row_anchor, out_pos,
                                      p->out_capacity_rows, (int)p->pos, device_status);
    if ((s = launched()) != STTM_OK) return s;
    k_members<<<blocks_for(pl.cells, 256), 256, 0, st>>>(g, cover, root, row_at_root, vid_off,
                                                        (int32_t*)(ws + pl.cell_row), merge_map,
                                                        (int32_t*)(ws + pl.row_weight),
                                                        (int32_t*)(ws + pl.row_last_t), (int)p->wt);
    if ((s = launched()) != STTM_OK) return s;
    k_span<<<blocks_for(pl.cells, 256), 256, 0, st>>>(g, pl.Tc, vid_off, row_anchor,
                                                     (const int32_t*)(ws + pl.row_last_t),
                                                     (int32_t*)(ws + pl.span_off), (int32_t*)(ws + pl.span_total));
    if ((s = launched()) != STTM_OK) return s;
    mark_stage(3, st);

    return by_levels_dtype(g.L, p->in_dtype, [&](auto lv, auto* tag) {
        using T = std::remove_const_t<std::remove_pointer_t<decltype(tag)>>;
        constexpr int LV = decltype(lv)::value;
        if (p->out_dtype == STTM_BF16)
            return launch_accumulate<LV, T, __nv_bfloat16>(feats, pl, ws, out_feats, p->out_capacity_rows,
                                                           (int)p->wt, st);
        return launch_accumulate<LV, T, float>(feats, pl, ws, out_feats, p->out_capacity_rows, (int)p->wt, st);
    });
}

}  // namespace

extern "C" {

sttm_status sttm_merge(const void* feats, int T, int H, int W, int D, float tau_s, float tau_t, void* out_feats,
                       int32_t* out_pos, int32_t* out_count, void* stream) {
    sttm_params p;
    sttm_default_params(&p, T, H, W, D, tau_s, tau_t);
    const size_t need = sttm_workspace_bytes(&p);
    if (need == 0) {
        Plan pl;
        return make_plan(&p, &pl);
    }
    const int dev = device_slot();
    if (dev < 0) return STTM_ERR_UNSUPPORTED;
    Cache& c = g_cache[dev];
    if (c.ws_bytes < need || c.merge_status == nullptr) {
        STTM_CUDA_TRY(cudaDeviceSynchronize());
        sttm_status s = grow(&c.ws, &c.ws_bytes, need);
        if (s != STTM_OK) return s;
        if (c.merge_status == nullptr) STTM_CUDA_TRY(cudaMalloc((void**)&c.merge_status, 256));
    }
    STTM_CUDA_TRY(cudaMemsetAsync(c.merge_status, 0, 4, (cudaStream_t)stream));
    return sttm_merge_ex(feats, &p, c.ws, c.ws_bytes, out_feats, out_pos, nullptr, out_count, nullptr, c.merge_status,
                         stream);
}

sttm_status sttm_merge_status(int32_t* host_bits, void* stream) {
    const int dev = device_slot();
    if (dev < 0) return STTM_ERR_UNSUPPORTED;
    Cache& c = g_cache[dev];
    int32_t bits = 0;
    if (c.merge_status != nullptr) {
        STTM_CUDA_TRY(cudaMemcpyAsync(&bits, c.merge_status, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
        STTM_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    }
    if (host_bits != nullptr) *host_bits = bits;
    return sttm_status_from_bits(bits);
}

size_t sttm_budget_workspace_bytes(const sttm_params* p) {
    Plan pl;
    if (make_plan(p, &pl, true) != STTM_OK || !(pl.f.ok || pl.fl.ok)) return 0;
    return (pl.total + 255) / 256 * 256 + ((size_t)pl.cells * 4 + 255) / 256 * 256 + 256;
}

sttm_status sttm_merge_budget(const void* feats, const sttm_params* p, const long long* budget_rows, void* ws,
                              size_t ws_bytes, void* out_feats, int32_t* out_pos, int32_t* merge_map,
                              int32_t* out_count, int64_t* out_offsets, float* tau_t_out, int32_t* device_status,
                              void* stream) {
    Plan pl;
    sttm_status s = make_plan(p, &pl, true);
    if (s != STTM_OK) return s;
    if (!(pl.f.ok || pl.fl.ok)) return STTM_ERR_UNSUPPORTED;
    if (!budget_rows || !ws || !out_count) return STTM_ERR_ARG;
    for (int b = 0; b < p->B; b++)
        if (budget_rows[b] < 1) return STTM_ERR_ARG;
    if (ws_bytes < sttm_budget_workspace_bytes(p)) return STTM_ERR_WORKSPACE;
    char* base = (char*)ws;
    const size_t main_bytes = (pl.total + 255) / 256 * 256;
    float* tmax = (float*)(base + main_bytes);
    float* tau_dev = (float*)(base + main_bytes + ((size_t)pl.cells * 4 + 255) / 256 * 256);
    cudaStream_t st = (cudaStream_t)stream;
    // first pass: no temporal merging (tau_t = 2), every kept node reports its best candidate
    sttm_params q = *p;
    q.tau_t = 2.f;
    q.tau_t_per_video = nullptr;
    Internal first;
    first.budget = true;
    first.tmax = tmax;
    s = merge_impl(feats, &q, ws, main_bytes, out_feats, out_pos, nullptr, out_count, out_offsets, device_status, first,
                   stream);
    close_stage_range();
    if (s != STTM_OK) return s;
    Budgets bd = {};
    for (int b = 0; b < p->B; b++) bd.rows[b] = budget_rows[b];
    s = launch_after(k_budget_tau, (unsigned)p->B, 1024, st, (long long)pl.g.N, (const float*)tmax,
                     (const int32_t*)out_count, bd, tau_dev);
    if (s != STTM_OK) return s;
    // second pass: the whole path with the thresholds read from device memory
    Internal second;
    second.budget = true;
    second.tau_dev = tau_dev;
    second.second_pass = pl.fl.ok;      // the two-stream kernels keep the first pass's Gram stage
    s = merge_impl(feats, p, ws, main_bytes, out_feats, out_pos, merge_map, out_count, out_offsets, device_status, second,
                   stream);
    close_stage_range();
    if (s != STTM_OK) return s;
    if (tau_t_out != nullptr)
        STTM_CUDA_TRY(cudaMemcpyAsync(tau_t_out, tau_dev, sizeof(float) * p->B, cudaMemcpyDeviceToDevice, st));
    return STTM_OK;
}

size_t sttm_merged_positions_workspace(long long capacity_rows) {
    if (capacity_rows <= 0) return 0;
    return ((size_t)capacity_rows * 8 + 255) / 256 * 256 + (size_t)capacity_rows * 4;
}

sttm_status sttm_merged_positions(const int32_t* merge_map, const int64_t* out_offsets, int B, long long N, void* ws,
                                  size_t ws_bytes, float* out_pos_mean, long long capacity_rows,
                                  int32_t* device_status, void* stream) {
    if (!merge_map || !out_offsets || !ws || !out_pos_mean) return STTM_ERR_ARG;
    if (B < 1 || N < 1 || capacity_rows < 1 || misaligned(ws, 256)) return STTM_ERR_ARG;
    if (B > kMaxBatch || (long long)B * N >= (1ll << 31)) return STTM_ERR_UNSUPPORTED;
    const size_t need = sttm_merged_positions_workspace(capacity_rows);
    if (ws_bytes < need) return STTM_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned long long* sum = (unsigned long long*)ws;
    unsigned int* cnt = (unsigned int*)((char*)ws + ((size_t)capacity_rows * 8 + 255) / 256 * 256);
    STTM_CUDA_TRY(cudaMemsetAsync(ws, 0, need, st));
    k_pos_accumulate<<<blocks_for((long long)B * N, 256), 256, 0, st>>>(B, N, merge_map, out_offsets, sum, cnt,
                                                                       capacity_rows, device_status);
    sttm_status s = launched();
    if (s != STTM_OK) return s;
    const long long rows_max = std::min<long long>(capacity_rows, (long long)B * N);
    k_pos_finish<<<blocks_for(rows_max, 256), 256, 0, st>>>(rows_max, out_offsets, B, sum, cnt, out_pos_mean);
    return launched();
}

sttm_status sttm_row_weights(const sttm_params* p, const void* ws, const int32_t* merge_map,
                             const int64_t* out_offsets, float* weights, void* stream) {
    Plan pl;
    sttm_status s = make_plan(p, &pl);
    if (s != STTM_OK) return s;
    if (!ws || !merge_map || !out_offsets || !weights || misaligned(ws, 256)) return STTM_ERR_ARG;
    if (p->out_capacity_rows < 1) return STTM_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const long long rows = std::min<long long>(pl.cells, p->out_capacity_rows);
    STTM_CUDA_TRY(cudaMemsetAsync(weights, 0, (size_t)rows * sizeof(float), st));
    k_row_weights<<<blocks_for(pl.cells, 256), 256, 0, st>>>(pl.g, (const int8_t*)((const char*)ws + pl.cover),
                                                            merge_map, out_offsets, weights, rows,
                                                            (int)p->wt);
    return launched();
}

sttm_status sttm_segment_fold(const int32_t* map_last, const int32_t* anchors, const float* v, const float* s,
                              const int32_t* n_dev, int n_max, int HW, int D, float* extra, float* extra_w,
                              long long capacity_rows, int32_t* device_status, void* stream) {
    if (!map_last || !anchors || !v || !s || !n_dev || !extra || !extra_w) return STTM_ERR_ARG;
    if (n_max < 1 || HW < 1 || D < 1 || capacity_rows < 1) return STTM_ERR_ARG;
    k_segment_fold<<<blocks_for((long long)n_max * 32, 256), 256, 0, (cudaStream_t)stream>>>(
        map_last, anchors, v, s, n_dev, n_max, HW, D, extra, extra_w, capacity_rows, device_status);
    return launched();
}

sttm_status sttm_segment_emit(const float* feats, const float* weights, const float* extra, const float* extra_w,
                              const float* halo_feats, const float* halo_w, const int32_t* n_h_dev, int n_max, int D,
                              float* v_out, float* s_out, void* stream) {
    if (!feats || !weights || !extra || !extra_w || !halo_feats || !halo_w || !n_h_dev || !v_out || !s_out)
        return STTM_ERR_ARG;
    if (n_max < 1 || D < 1) return STTM_ERR_ARG;
    k_segment_emit<<<blocks_for((long long)n_max * 32, 256), 256, 0, (cudaStream_t)stream>>>(
        feats, weights, extra, extra_w, halo_feats, halo_w, n_h_dev, n_max, D, v_out, s_out);
    return launched();
}

sttm_status sttm_segment_finish(const float* feats, const int32_t* pos, const float* weights, const float* extra,
                                const float* extra_w, const int32_t* count_dev, const int32_t* n_h_dev, int D,
                                long long capacity_rows, long long pos_shift, sttm_pos_mode pos_mode,
                                sttm_dtype out_dtype, void* out_feats, int32_t* out_pos, int32_t* owned_count,
                                void* stream) {
    if (!feats || !pos || !weights || !extra || !extra_w || !count_dev || !out_feats || !out_pos || !owned_count)
        return STTM_ERR_ARG;
    if (D < 1 || D % 4 != 0 || capacity_rows < 1) return STTM_ERR_ARG;
    if (misaligned(feats, 16) || misaligned(extra, 16) || misaligned(out_feats, 16)) return STTM_ERR_ARG;
    if (out_dtype != STTM_BF16 && out_dtype != STTM_F32) return STTM_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const unsigned blocks = blocks_for(capacity_rows * (D / VEC), 256);
    const int re = pos_mode == STTM_POS_REASSIGNED ? 1 : 0;
    if (out_dtype == STTM_BF16)
        k_segment_finish<__nv_bfloat16><<<blocks, 256, 0, st>>>(feats, pos, weights, extra, extra_w, count_dev,
                                                                n_h_dev, D, capacity_rows, pos_shift, re,
                                                                (__nv_bfloat16*)out_feats, out_pos, owned_count);
    else
        k_segment_finish<float><<<blocks, 256, 0, st>>>(feats, pos, weights, extra, extra_w, count_dev, n_h_dev, D,
                                                        capacity_rows, pos_shift, re, (float*)out_feats, out_pos,
                                                        owned_count);
    return launched();
}

sttm_status sttm_merge_host(const void* h_feats, const sttm_params* p, void* h_out_feats, int32_t* h_out_pos,
                            int32_t* h_merge_map, int32_t* h_out_count, int64_t* h_out_offsets,
                            int32_t* h_device_status) {
    Plan pl;
    sttm_status s = make_plan(p, &pl);
    if (s != STTM_OK) return s;
    if (!h_feats || !h_out_feats || !h_out_pos || !h_out_count) return STTM_ERR_ARG;
    if (p->out_capacity_rows < 0) return STTM_ERR_ARG;
    int dev = 0;
    STTM_CUDA_TRY(cudaGetDevice(&dev));
    Cache& c = g_cache[dev % 64];
    const Geo g = pl.g;
    const size_t in_elt = p->in_dtype == STTM_BF16 ? 2 : 4, out_elt = p->out_dtype == STTM_BF16 ? 2 : 4;
    const size_t feats_bytes = (size_t)pl.cells * g.D * in_elt;
    const size_t out_bytes = (size_t)p->out_capacity_rows * g.D * out_elt;
    // ints: out_pos [cap] | merge_map [cells] | out_count [B] | status [1] | offsets [B+1] (int64)
    const size_t o_pos = 0, o_map = align_up((size_t)p->out_capacity_rows * 4),
                 o_cnt = o_map + align_up((size_t)pl.cells * 4), o_status = o_cnt + align_up((size_t)g.B * 4),
                 o_off = o_status + 256, ints_bytes = o_off + align_up((size_t)(g.B + 1) * 8);
    if (c.ws_bytes < pl.total || c.feats_bytes < feats_bytes || c.out_bytes < out_bytes ||
        c.ints_bytes < ints_bytes) {
        STTM_CUDA_TRY(cudaDeviceSynchronize());
        if ((s = grow(&c.ws, &c.ws_bytes, pl.total)) != STTM_OK) return s;
        if ((s = grow(&c.feats, &c.feats_bytes, feats_bytes)) != STTM_OK) return s;
        if ((s = grow(&c.out, &c.out_bytes, std::max<size_t>(out_bytes, 256))) != STTM_OK) return s;
        if ((s = grow(&c.ints, &c.ints_bytes, ints_bytes)) != STTM_OK) return s;
    }
    char* ints = (char*)c.ints;
    cudaStream_t st = 0;
    STTM_CUDA_TRY(cudaMemcpyAsync(c.feats, h_feats, feats_bytes, cudaMemcpyHostToDevice, st));
    STTM_CUDA_TRY(cudaMemsetAsync(ints + o_status, 0, 4, st));
    s = sttm_merge_ex(c.feats, p, c.ws, c.ws_bytes, c.out, (int32_t*)(ints + o_pos),
                      h_merge_map ? (int32_t*)(ints + o_map) : nullptr, (int32_t*)(ints + o_cnt),
                      (int64_t*)(ints + o_off), (int32_t*)(ints + o_status), st);
    if (s != STTM_OK) return s;
    long long offsets[kMaxBatch + 1];
    STTM_CUDA_TRY(cudaMemcpyAsync(offsets, ints + o_off, (size_t)(g.B + 1) * 8, cudaMemcpyDeviceToHost, st));
    STTM_CUDA_TRY(cudaMemcpyAsync(h_out_count, ints + o_cnt, (size_t)g.B * 4, cudaMemcpyDeviceToHost, st));
    int32_t status = 0;
    STTM_CUDA_TRY(cudaMemcpyAsync(&status, ints + o_status, 4, cudaMemcpyDeviceToHost, st));
    STTM_CUDA_TRY(cudaStreamSynchronize(st));
    const long long rows = std::min<long long>(offsets[g.B], p->out_capacity_rows);
    STTM_CUDA_TRY(cudaMemcpyAsync(h_out_feats, c.out, (size_t)rows * g.D * out_elt, cudaMemcpyDeviceToHost, st));
    STTM_CUDA_TRY(cudaMemcpyAsync(h_out_pos, ints + o_pos, (size_t)rows * 4, cudaMemcpyDeviceToHost, st));
    if (h_merge_map)
        STTM_CUDA_TRY(cudaMemcpyAsync(h_merge_map, ints + o_map, (size_t)pl.cells * 4, cudaMemcpyDeviceToHost, st));
    STTM_CUDA_TRY(cudaStreamSynchronize(st));
    if (h_out_offsets) std::memcpy(h_out_offsets, offsets, (size_t)(g.B + 1) * 8);
    if (h_device_status) *h_device_status = status;
    return STTM_OK;
}

void sttm_release_cache(void) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return;
    Cache& c = g_cache[dev % 64];
    cudaDeviceSynchronize();
    if (c.ws) cudaFree(c.ws);
    if (c.feats) cudaFree(c.feats);
    if (c.merge_status) cudaFree(c.merge_status);
    if (c.out) cudaFree(c.out);
    if (c.ints) cudaFree(c.ints);
    c = Cache();
}

}  // extern "C"
