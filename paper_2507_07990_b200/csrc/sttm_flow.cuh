// Two-stream STTM kernels (sm_100a): every similarity first, then every average.
//
// The decisions of Sections 3.2 and 3.3 (cover map, links) are pure functions of the input:
// they depend on dot products of a frame's cells with each other and with the cells of the
// frame before it, never on what was merged earlier.  So the work splits into stages that
// have no serial dependence through time:
//   Gram stage    streams the features once and leaves, per (tile, frame, channel slice), the
//                 128 numbers the decisions need (8 per cell: linear combinations of the tile's
//                 Gram matrix X_t X_t^T and cross matrix X_t X_{t-1}^T, see combine_sums()).
//                 Every (tile, run of frames, channel slice) is an independent task.
//   decision stage adds the slices in a fixed order and takes the decisions, one half warp per
//                 (tile, frame): cover level and link of every cell.
//   ordering      row numbers of the surviving tokens (Section 3.4): integer scans.
//   chain stage   one warp per (tile, run of frames) follows the chains through the run and
//                 leaves one command record per frame: a 16 x 16 matrix W (chain slot x cell)
//                 and the list of chains that ended, each with its final output row.
//   sum stage     streams the features a second time and forms the chain averages of Section 3.3
//                 as running sums
//                 sums[16 chain slots x channels] += W X on the tensor cores.  A chain that ends
//                 is divided by its weight and written straight to its output row.  Chains that
//                 cross the border between two runs of frames leave fp32 pieces that a small
//                 kernel adds up.
// A tile is 16 cells: a 4x4 block of the grid (clipped at the border), or, when the grid is one
// cell wider (higher) than a multiple of four, 16 cells of its last column (row).  One tensor
// copy (cp.async.bulk.tensor, 128-byte swizzle) brings a tile's frame and channel slice into a
// shared-memory ring as [64-channel block][cell][64 channels]; rows outside the grid arrive as zeros.
#pragma once

#include <cuda.h>

#include "sttm_fused.cuh"

namespace sttm {

constexpr int kFlowWorkers = 7;                      // Gram warps / sum warps (with the producer: 256 threads,
                                                     // so that two CTAs on an SM leave 128 registers a thread)
constexpr int kFlowWarps = kFlowWorkers + 1;         // + producer warp
constexpr int kFlowThreads = kFlowWarps * 32;
constexpr int kFlowMaxRing = 16;
constexpr int kFlowMaxNB = 14;                       // 64-channel blocks per slice: two per sum warp
constexpr int kFlowMaxKs = 8;                        // 16-channel steps per Gram warp
constexpr int kBlkBytes = 2048;                      // 16 cells x 128 bytes
constexpr int kFlowMaxF = 64;                        // frames per item, the frame before it not counted
constexpr int kRecBytes = (int)sizeof(FrameRec);

struct TileBox { int kind, x0, y0, pad; };           // 0: 4x4 box at (x0, y0); 1: 16 cells down column x0; 2: 16 cells along row y0

struct FlowParams {
    int B, T, H, W, D, L;
    int HW, N;
    int ntiles;
    int NS, NB;              // channel slices, 64-channel blocks per slice (sum stage)
    int NSg, NBg, NCg;       // Gram stage: slices (`partial` holds NSg per frame), blocks per copy, copies per slice
    int slot_bytes, R;
    int F, nseg, nitems;     // frames per item, items per (video, tile), items
    int weight_mode, out_f32, match_best;
    int8_t* cover;
    int32_t* link;
    int32_t* chain_key;      // [B*N] per cell: root cell id of its chain as far as the item knows it
    int32_t* frame_roots;    // [B*T] chains that start in a frame (= its output rows), zero on entry
    float* tmax;             // budget mode, may be null (see FusedParams::tmax)
    const float* tau_t_dev;  // budget mode, may be null: [B] temporal thresholds in device memory
    float* partial;          // [nitems][F+1][NSg][128]: the Gram stage's numbers, [cell][number]
    int32_t* hand;           // [nitems][F+1][16]: cover level | (link lane + 1) << 8 of every tile row
    FrameRec* recs;          // [nitems][F+2]: the chain stage's records, one per frame and a closing one
    int32_t* progress;       // [nitems]: number of records the chain stage has published (zero before the call)
    const int32_t* row_at_root;   // [B*N] row (inside its video) of every surviving token
    const long long* vid_off;     // [B+1] first row of every video
    void* out;               // [rows][D] output rows
    long long capacity;
    float* pieces;           // [nitems][kPieceSlots][D]
    int2* piece_meta;        // [nitems][kPieceSlots] {key cell id or -1, weight}
    int* status;
    TileDesc tiles[kMaxTiles];
    TileBox boxes[kMaxTiles];
};

struct FlowMaps { CUtensorMap m[3]; };               // one per kind of TileBox

struct FlowItem {
    int item, b, tile, tstart, n, halo, last_seg;
};

// item = (video, run of frames, tile), tiles fastest: items of one run of frames are neighbours
__device__ __forceinline__ FlowItem flow_item(const FlowParams& p, int item) {
    FlowItem it;
    it.item = item;
    it.tile = item % p.ntiles;
    const int bs = item / p.ntiles;
    const int seg = bs % p.nseg;
    it.b = bs / p.nseg;
    const int t0 = seg * p.F, t1 = min(p.T, t0 + p.F);
    it.halo = t0 > 0;
    it.tstart = t0 - it.halo;
    it.n = t1 - it.tstart;
    it.last_seg = t1 == p.T;
    return it;
}

// Where the Gram stage's numbers of frame j of an item are: [slice][cell][number].  The frame before a
// run is the last frame of the run before it, and its numbers are taken from there.
__device__ __forceinline__ const float* flow_numbers(const FlowParams& p, const FlowItem& it, int j) {
    if (it.halo && j == 0) {
        const int seg = (it.item / p.ntiles) % p.nseg;
        const int prev_n = p.F + (seg > 1 ? 1 : 0);         // frames of the run before, its own frame-before included
        return p.partial + ((long long)(it.item - p.ntiles) * (p.F + 1) + prev_n - 1) * p.NSg * kSumVals;
    }
    return p.partial + ((long long)it.item * (p.F + 1) + j) * p.NSg * kSumVals;
}

// has the phase with this parity completed?  Suspends the thread for a while (the hardware's own
// limit) instead of returning at once: a waiting warp of these kernels must not take issue slots
// from the warps that have work.
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded wait (see mbar_wait) on the suspending form
__device__ __forceinline__ bool mbar_wait_sleep(uint32_t bar, int use, bool& timed_out) {
    if (timed_out) return false;
    const uint32_t parity = (uint32_t)(use & 1);
    if (mbar_try(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    while (!mbar_try(bar, parity)) {
        if (global_timer_ns() - t0 > kWaitLimitNs) {
            timed_out = true;
            return false;
        }
    }
    return true;
}
// The k-th task a kernel takes up.  The Gram stage goes through the video forwards, the sum stage
// backwards: what the Gram stage read last is what L2 still holds when the sum stage begins.
__device__ __forceinline__ int flow_task(bool sum_stage, int k, int ntasks) { return sum_stage ? ntasks - 1 - k : k; }

// bounded wait whose outcome is the same in every lane of the warp
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, int use, bool& timed_out) {
    const bool ok = mbar_wait_sleep(bar, use, timed_out);
    const bool all = __all_sync(0xffffffffu, ok);
    if (!all) timed_out = true;
    return all;
}

// one tile of one frame, NB 64-channel blocks from block `blk0` on: global -> shared memory,
// completion counted in bytes on an mbarrier
__device__ __forceinline__ void tma_load_tile(uint32_t dst, const CUtensorMap* map, int x, int y, int blk0, int frame,
                                              uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(x), "r"(y), "r"(blk0), "r"(frame), "r"(bar)
        : "memory");
}

// Section 3.2 for one frame, 16 lanes per frame (both halves of the warp at once, each on its own
// frame): the cover level of the lane's cell and the squared norm of the node that covers it.
// n0 = |x_c|^2, d0 = x_c . parent(c), rr = x_c . top.
__device__ __forceinline__ int spatial_level(float n0, float d0, float rr, const LaneGeo& lg, int L, float tau_s,
                                             int half, float& nk) {
    const unsigned full = 0xffffffffu;
    const float n1 = lg.w1 * quad_sum(d0, lg.qbits);     // |parent|^2
    const float d1 = lg.w1 * quad_sum(rr, lg.qbits);     // parent . top
    const float n2 = top_sum(lg.w2 * rr, lg.tbits);      // |top|^2
    int lv = 0;
    if (L >= 2) {
        const bool p0 = !lg.valid || cos_above(d0, n0, n1, tau_s);
        const uint32_t pm0 = (__ballot_sync(full, p0) >> (16 * half)) & 0xffffu;
        const bool quad_pass = (pm0 & lg.qmask) == lg.qmask;
        if (L == 3) {
            const bool p1 = !lg.valid || cos_above(d1, n1, n2, tau_s);
            const uint32_t pm1 = (__ballot_sync(full, p1) >> (16 * half)) & 0xffffu;
            lv = (pm1 & lg.tmask) == lg.tmask ? 2 : (quad_pass ? 1 : 0);
        } else {
            lv = quad_pass ? 1 : 0;
        }
    }
    nk = lv == 0 ? n0 : (lv == 1 ? n1 : n2);
    return lv;
}

// ---------------------------------------------------------------------------------
// Decision stage.  One warp per (item, pair of frames); lanes 0..15 take the even frame, lanes
// 16..31 the odd one; lane c and lane c + 16 are cell c of the tile.
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
k_flow_decide(const __grid_constant__ FlowParams p, const __grid_constant__ Taus taus) {
    wait_for_prior_kernel();
    const unsigned full = 0xffffffffu;
    const int lane = threadIdx.x & 31, c = lane & 15, half = lane >> 4;
    const int pairs = (p.F + 2) / 2;                    // pairs of frames per item, the frame before it included
    const long long w = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (w >= (long long)p.nitems * pairs) return;
    const FlowItem it = flow_item(p, (int)(w / pairs));
    const int j = (int)(w % pairs) * 2 + half;
    const bool mine = j < it.n;
    const LaneGeo lg = lane_geo(p.tiles[it.tile], c, p.L, p.W);
    const bool valid = lg.valid;
    const float tau_s = taus.s[it.b], tau_t = p.tau_t_dev != nullptr ? p.tau_t_dev[it.b] : taus.t[it.b];

    // the slices' shares, in slice order; the frame before (numbers 0..2 only) for its cover level
    float v[8], u[3];
#pragma unroll
    for (int k = 0; k < 8; k++) v[k] = 0.f;
    u[0] = u[1] = u[2] = 0.f;
    const bool has_prev = mine && j > 0;
    if (mine && valid) {
        const float4* src = reinterpret_cast<const float4*>(flow_numbers(p, it, j) + c * 8);
        for (int s = 0; s < p.NSg; s++) {
            const float4 a = __ldcg(src + s * (kSumVals / 4)), b = __ldcg(src + s * (kSumVals / 4) + 1);
            v[0] += a.x; v[1] += a.y; v[2] += a.z; v[3] += a.w;
            v[4] += b.x; v[5] += b.y; v[6] += b.z; v[7] += b.w;
        }
        if (has_prev) {
            const float4* sp = reinterpret_cast<const float4*>(flow_numbers(p, it, j - 1) + c * 8);
            for (int s = 0; s < p.NSg; s++) {
                const float4 a = __ldcg(sp + s * (kSumVals / 4));
                u[0] += a.x; u[1] += a.y; u[2] += a.z;
            }
        }
    }
    float nk, pnk;
    const int lv = spatial_level(v[0], v[1], v[2], lg, p.L, tau_s, half, nk);
    const int lu = spatial_level(u[0], u[1], u[2], lg, p.L, tau_s, half, pnk);

    // Section 3.3: the node covering the cell against the overlapping kept node of the frame
    // before; a pair is evaluated at the top-left cell of its finer node
    int link_local = -1;
    {
        const float w1 = lg.w1, w2 = lg.w2;
        const float t11 = w1 * quad_sum(v[4], lg.qbits), t12 = w1 * quad_sum(v[5], lg.qbits);
        const float t21 = w1 * quad_sum(v[7], lg.qbits), t22 = top_sum(w2 * v[5], lg.tbits);
        float dot;
        if (lv == 0) dot = lu == 0 ? v[3] : (lu == 1 ? v[4] : v[5]);
        else if (lv == 1) dot = lu == 0 ? v[6] : (lu == 1 ? t11 : t12);
        else dot = lu == 0 ? v[7] : (lu == 1 ? t21 : t22);
        const bool rep = valid && has_prev && lane_anchor(lg, c, min(lv, lu)) == c;
        const bool pass = rep && cos_above(dot, nk, pnk, tau_t);
        const uint32_t passm = (__ballot_sync(full, pass) >> (16 * half)) & 0xffffu;
        const uint32_t cand = passm & lane_region(lg, c, lv);
        int cstar = cand ? __ffs(cand) - 1 : 0;             // first in row-major order: the top-left one
        if (p.match_best) {
            // the most similar of them instead (equal ones: the first)
            const float cosv = pass ? dot / (sqrtf(nk) * sqrtf(pnk)) : -2.f;
            float best = -2.f;
#pragma unroll
            for (int i = 0; i < 16; i++) {
                const float si = __shfl_sync(full, cosv, 16 * half + i);
                if (((cand >> i) & 1u) && si > best) { best = si; cstar = i; }
            }
        }
        if (p.tmax != nullptr) {
            // budget mode: per kept node the largest cosine to its candidates
            const float cosv = rep ? ((nk == 0.f || pnk == 0.f) ? 0.f : dot / (sqrtf(nk) * sqrtf(pnk))) : -2.f;
            const uint32_t candm = ((__ballot_sync(full, rep) >> (16 * half)) & 0xffffu) & lane_region(lg, c, lv);
            float most = -2.f;
#pragma unroll
            for (int i = 0; i < 16; i++) {
                const float si = __shfl_sync(full, cosv, 16 * half + i);
                if (((candm >> i) & 1u) && si > most) most = si;
            }
            if (mine && valid && !(it.halo && j == 0))
                p.tmax[(long long)it.b * p.N + (long long)(it.tstart + j) * p.HW + lg.cell] =
                    lane_anchor(lg, c, lv) == c ? most : -2.f;
        }
        const int lu_star = __shfl_sync(full, lu, 16 * half + cstar);
        link_local = cand ? lane_anchor(lg, cstar, lu_star) : -1;
    }
    const int lcell = __shfl_sync(full, lg.cell, 16 * half + (link_local < 0 ? 0 : link_local));
    if (mine) p.hand[((long long)it.item * (p.F + 1) + j) * 16 + c] = lv | ((link_local + 1) << 8);
    const bool owned = mine && !(it.halo && j == 0);        // the frame before the item belongs to the item before
    const int tt = it.tstart + j;
    if (owned && valid) {
        const long long gcc = (long long)it.b * p.N + (long long)tt * p.HW + lg.cell;
        p.cover[gcc] = (int8_t)lv;
        p.link[gcc] = link_local < 0 ? -1 : (tt - 1) * p.HW + lcell;
    }
    // every chain that starts here is an output row of this frame
    const bool fresh = owned && valid && lane_anchor(lg, c, lv) == c && link_local < 0;
    const uint32_t freshm = (__ballot_sync(full, fresh) >> (16 * half)) & 0xffffu;
    if (c == 0 && freshm != 0 && owned) atomicAdd(p.frame_roots + it.b * p.T + tt, __popc(freshm));
}

// ---------------------------------------------------------------------------------
// Chain stage.  One warp per item follows the tile's chains through the item's frames: which
// running sum (chain slot) every kept node joins, which chains ended and where they go.  Leaves
// one record per frame and a closing record that writes out what still runs at the item's end.
// ---------------------------------------------------------------------------------
constexpr int kChainWarps = 4;

__global__ void __launch_bounds__(kChainWarps * 32)
k_flow_chain(const __grid_constant__ FlowParams p) {
    wait_for_prior_kernel();
    // The sum stage may become resident now: it takes a frame's record only after this kernel has
    // published it (`progress`), so its stream of features starts while the records are still written.
    let_next_kernel_start();
    __shared__ __align__(16) FrameRec s_rec[kChainWarps];
    __shared__ SlotTable s_tab[kChainWarps];
    const unsigned full = 0xffffffffu;
    const int wib = threadIdx.x >> 5, lane = threadIdx.x & 31, c = lane & 15;
    const bool low = lane < 16;
    const int item = blockIdx.x * kChainWarps + wib;
    if (item >= p.nitems) return;
    const FlowItem it = flow_item(p, item);
    FrameRec* rec = &s_rec[wib];
    SlotTable* tab = &s_tab[wib];
    const LaneGeo lg = lane_geo(p.tiles[it.tile], c, p.L, p.W);
    const bool valid = lg.valid;
    const float w1 = lg.w1, w2 = lg.w2;
    const long long vrow0 = p.vid_off[it.b];
    p.piece_meta[(long long)it.item * kPieceSlots + lane] = make_int2(-1, 0);
    FrameRec* dst = p.recs + (long long)it.item * (p.F + 2);
    const int32_t* hand = p.hand + (long long)it.item * (p.F + 1) * 16;
    int prev_slot = 0;
    uint32_t active_slots = 0;
    // The run's decisions and row numbers, fetched at once: the frames are worked on one after the other,
    // and a load per frame would put the memory's latency (long while the sum stage streams) into every step.
    __shared__ int32_t s_hand[kChainWarps][(kFlowMaxF + 1) * 16], s_rows[kChainWarps][(kFlowMaxF + 1) * 16];
    for (int i = lane; i < it.n * 16; i += 32) {
        s_hand[wib][i] = hand[i];
        s_rows[wib][i] = valid ? p.row_at_root[(long long)it.b * p.N + (long long)(it.tstart + (i >> 4)) * p.HW + lg.cell] : -1;
    }
    __syncwarp();
    for (int j = 0; j <= it.n; j++) {
        const int packed = j < it.n ? s_hand[wib][j * 16 + c] : 0, my_row = j < it.n ? s_rows[wib][j * 16 + c] : -1;
        if (j == it.n) {
            // Closing record: everything still running is written out.  A chain goes on into the next
            // item iff a node of that item's first frame is linked to its node of this frame; the
            // others end here like any chain that ends inside the item.
            uint32_t goes_on = 0;
            if (!it.last_seg) {
                const int nxt = p.hand[((long long)(it.item + p.ntiles) * (p.F + 1) + 1) * 16 + c];
                const int nlv = nxt & 3, nlink = (nxt >> 8) - 1;
                const bool nlinked = valid && lane_anchor(lg, c, nlv) == c && nlink >= 0;
                const int tslot = __shfl_sync(full, prev_slot, nlink < 0 ? 0 : nlink);
                goes_on = __reduce_or_sync(full, nlinked ? 1u << tslot : 0u);
            }
            uint32_t empty = 0;
            if (low && ((active_slots >> lane) & 1u)) {
                const bool on = (goes_on >> lane) & 1u;
                if (!tab->virt[lane] && !on) {
                    const long long grow = vrow0 + tab->row[lane];
                    rec->flush[lane] = FlushCmd{lane, 0, grow < p.capacity ? (int)grow : -1, (float)tab->weight[lane]};
                } else if (tab->virt[lane] && tab->weight[lane] == 0 && !on) {
                    empty = 1u << lane;             // came in from the frame before the item and got no member here
                } else {
                    const int pc = it.item * kPieceSlots + 16 + lane;
                    rec->flush[lane] = FlushCmd{lane, 1, pc, 0.f};
                    p.piece_meta[pc] = make_int2(tab->key[lane], tab->weight[lane]);
                }
            }
            empty = __reduce_or_sync(full, empty);
            if (lane == 0) rec->flush_mask = active_slots & ~empty;
        } else {
            const int lv = packed & 3, link_local = (packed >> 8) - 1;
            const int t = it.tstart + j;
            const bool is_halo = it.halo && j == 0;
            // nodes with a link join the chain of their target; chains without a member in this
            // frame have ended; the remaining nodes start new chains in free slots
            const bool anchor = valid && lane_anchor(lg, c, lv) == c;
            const bool linked = anchor && link_local >= 0;
            const bool fresh = anchor && link_local < 0;
            const int slot_linked = __shfl_sync(full, prev_slot, link_local < 0 ? 0 : link_local);
            const uint32_t memb = __reduce_or_sync(full, linked ? 1u << slot_linked : 0u);
            const uint32_t dead = active_slots & ~memb;
            const uint32_t freem = ~memb & 0xffffu;
            const uint32_t freshm = __ballot_sync(full, fresh && low);
            const int slot_fresh = kth_set_bit16(freem, __popc(freshm & ((1u << c) - 1)));
            const int node_slot = linked ? slot_linked : slot_fresh;
            const int cur_slot = __shfl_sync(full, node_slot, (lane & 16) + lane_anchor(lg, c, lv));
            const uint32_t cells = lane_region(lg, c, lv);
            const int wint = p.weight_mode ? __popc(cells) : 1;
            const long long gc = (long long)it.b * p.N + (long long)t * p.HW + lg.cell;
            // chains that ended: lane s looks at slot s (before the slot is given away again)
            uint32_t empty = 0;
            if (low && ((dead >> lane) & 1u)) {
                if (tab->virt[lane] && tab->weight[lane] == 0) {
                    empty = 1u << lane;             // a node of the frame before the item that nothing was linked to: no piece
                } else if (tab->virt[lane]) {
                    const int pc = it.item * kPieceSlots + tab->cell[lane];
                    rec->flush[lane] = FlushCmd{lane, 1, pc, 0.f};
                    p.piece_meta[pc] = make_int2(tab->key[lane], tab->weight[lane]);
                } else {
                    const long long grow = vrow0 + tab->row[lane];
                    rec->flush[lane] = FlushCmd{lane, 0, grow < p.capacity ? (int)grow : -1, (float)tab->weight[lane]};
                }
            }
            __syncwarp();
            if (low && fresh) {
                tab->key[slot_fresh] = (int)gc;
                tab->weight[slot_fresh] = is_halo ? 0 : wint;
                tab->virt[slot_fresh] = is_halo ? 1 : 0;
                tab->cell[slot_fresh] = c;
                tab->row[slot_fresh] = my_row;
            }
            __syncwarp();
            if (low && linked) atomicAdd(&tab->weight[slot_linked], wint);
            // the frame's weight matrix: row = chain slot, column = cell
            reinterpret_cast<uint4*>(rec->wmat)[lane] = make_uint4(0u, 0u, 0u, 0u);
            const int wnode = __shfl_sync(full, wint, (lane & 16) + lane_anchor(lg, c, lv));
            __syncwarp();
            if (low && valid && !is_halo) {
                const float wc = (lv == 0 ? 1.f : (lv == 1 ? w1 : w2)) * (float)wnode;
                rec->wmat[cur_slot * 16 + c] = __bfloat16_as_ushort(__float2bfloat16_rn(wc));
            }
            empty = __reduce_or_sync(full, empty);
            if (lane == 0) rec->flush_mask = dead & ~empty;
            if (!is_halo && low && valid) p.chain_key[gc] = tab->key[cur_slot] - it.b * p.N;
            active_slots = memb | __reduce_or_sync(full, fresh ? 1u << slot_fresh : 0u);
            prev_slot = cur_slot;
        }
        __syncwarp();
        {
            const uint4* src = reinterpret_cast<const uint4*>(rec);
            uint4* d4 = reinterpret_cast<uint4*>(dst + j);
            for (int i = lane; i < kRecBytes / 16; i += 32) d4[i] = src[i];
        }
        __syncwarp();
        // (published every eighth record and at the end: the release costs about as much as a record)
        if (lane == 0 && ((j & 7) == 7 || j == it.n)) store_release(p.progress + it.item, j + 1);
    }
}

// ---------------------------------------------------------------------------------
// The streaming kernel.  kSum == false: Gram stage; kSum == true: sum stage.  A task is (item,
// channel slice); tasks are dealt to the CTAs round robin.  Warps: [0, 7) workers, 7 producer.
// Two CTAs share an SM: each runs its frames through its phases in step, and the two fill each
// other's gaps.
//   Gram stage: the seven workers share the slice's 16-channel steps and keep a frame's fragments
//   in registers for the next frame's cross products (a ring slot is free again as soon as it has
//   been read); their parts of G and C meet in shared memory between two named barriers, are added
//   in warp order and contracted to the 128 numbers.
//   Sum stage: warp a owns the slice's 64-channel blocks 2a and 2a + 1.
// Shared memory: ring of R slots (1024-byte aligned), R records, the Gram warps' parts, barriers.
// ---------------------------------------------------------------------------------
__host__ __device__ inline size_t flow_fixed_smem(int R) {
    return (size_t)R * kRecBytes + (size_t)kFlowWorkers * kGramVals * 4 + kGramVals * 4 + 128 + 2 * kFlowMaxRing * 8 + 1024;
}

template <bool kSum>
__global__ void __launch_bounds__(kFlowThreads, 2)
k_flow(const __grid_constant__ FlowParams p, const __grid_constant__ FlowMaps maps) {
    extern __shared__ unsigned char smem_raw[];
    // the swizzle pattern of the tensor copies is a function of the shared-memory address
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* ring = smem;
    size_t off = (size_t)p.R * p.slot_bytes;
    unsigned char* recs = smem + off;                              off += (size_t)p.R * kRecBytes;
    float* red = reinterpret_cast<float*>(smem + off);             off += (size_t)kFlowWorkers * kGramVals * 4;
    float* redsum = reinterpret_cast<float*>(smem + off);          off += kGramVals * 4;
    float* wtab = reinterpret_cast<float*>(smem + off);            off += 128;
    const uint32_t bar0 = smem_u32(smem + off);
    const uint32_t full_bar = bar0, empty_bar = bar0 + 8 * kFlowMaxRing;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t ring_base = smem_u32(ring), recs_base = smem_u32(recs);
    const int ntasks = p.nitems * p.NS;
    const int nsum = (p.NB + 1) / 2;                    // sum warps at work

    if (tid == 0) {
        for (int s = 0; s < p.R; s++) {
            mbar_init(full_bar + 8 * s, 1);
            mbar_init(empty_bar + 8 * s, kSum ? nsum : kFlowWorkers);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // (the sum stage does not wait for the chain stage as a whole: its producer waits per record)

    bool timed_out = false;
    int q = 0;                      // slots used so far by this CTA's tasks: slot q % R, filled q / R times before

    if (warp < kFlowWorkers && !kSum) {
        // ------------------------------------ Gram warps ------------------------------------
        const uint32_t lrow = (lane & 7) + ((lane >> 3) & 1) * 8;
        const int ksteps = p.NB * 4;
        const int k0 = ksteps * warp / kFlowWorkers, nk = ksteps * (warp + 1) / kFlowWorkers - k0;
        uint32_t koff[kFlowMaxKs];          // where this lane's rows of the warp's 16-channel steps sit in a slot
#pragma unroll
        for (int i = 0; i < kFlowMaxKs; i++) {
            const uint32_t kk = (uint32_t)(k0 + i);
            koff[i] = (kk >> 2) * kBlkBytes + lrow * 128 + ((((kk & 3) * 2 + (lane >> 4)) ^ (lrow & 7)) << 4);
        }
        const int nthr = kFlowWorkers * 32;
        const uint32_t redsum_a = smem_u32(redsum), W2s = smem_u32(wtab);
        for (int task = blockIdx.x; task < ntasks && !timed_out; task += gridDim.x) {
            const int tk = flow_task(kSum, task, ntasks);
            const FlowItem it = flow_item(p, tk / p.NS);
            const int slice = tk % p.NS;
            const LaneGeo lg = lane_geo(p.tiles[it.tile], tid & 15, p.L, p.W);
            named_sync(1, nthr);                       // the previous task's weights are not read any more
            if (tid < 16) wtab[tid] = lg.w2;
            float* dst = p.partial + ((long long)it.item * (p.F + 1) * p.NS + slice) * kSumVals;
            uint32_t prv[kFlowMaxKs][4];
#pragma unroll
            for (int i = 0; i < kFlowMaxKs; i++) prv[i][0] = prv[i][1] = prv[i][2] = prv[i][3] = 0u;
            for (int j = 0; j < it.n; j++, q++) {
                const int s = q % p.R;
                mbar_wait_warp(full_bar + 8 * s, q / p.R, timed_out);
                uint32_t cur[kFlowMaxKs][4];
                const uint32_t base = ring_base + s * p.slot_bytes;
#pragma unroll
                for (int i = 0; i < kFlowMaxKs; i++) {
                    if (i < nk) ldmatrix_x4(base + koff[i], cur[i]);
                    else cur[i][0] = cur[i][1] = cur[i][2] = cur[i][3] = 0u;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_bar + 8 * s);
                float g0[4] = {0.f, 0.f, 0.f, 0.f}, g1[4] = {0.f, 0.f, 0.f, 0.f};
                float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int i = 0; i < kFlowMaxKs; i++) {
                    if (i < nk) {
                        mma_bf16(g0, cur[i], cur[i][0], cur[i][2]);
                        mma_bf16(g1, cur[i], cur[i][1], cur[i][3]);
                        mma_bf16(c0, cur[i], prv[i][0], prv[i][2]);
                        mma_bf16(c1, cur[i], prv[i][1], prv[i][3]);
                    }
                }
                {
                    float* r = red + warp * kGramVals;
                    const int gr = lane >> 2, gc = (lane & 3) * 2;
                    *reinterpret_cast<float2*>(r + gr * 16 + gc) = make_float2(g0[0], g0[1]);
                    *reinterpret_cast<float2*>(r + (gr + 8) * 16 + gc) = make_float2(g0[2], g0[3]);
                    *reinterpret_cast<float2*>(r + gr * 16 + 8 + gc) = make_float2(g1[0], g1[1]);
                    *reinterpret_cast<float2*>(r + (gr + 8) * 16 + 8 + gc) = make_float2(g1[2], g1[3]);
                    *reinterpret_cast<float2*>(r + 256 + gr * 16 + gc) = make_float2(c0[0], c0[1]);
                    *reinterpret_cast<float2*>(r + 256 + (gr + 8) * 16 + gc) = make_float2(c0[2], c0[3]);
                    *reinterpret_cast<float2*>(r + 256 + gr * 16 + 8 + gc) = make_float2(c1[0], c1[1]);
                    *reinterpret_cast<float2*>(r + 256 + (gr + 8) * 16 + 8 + gc) = make_float2(c1[2], c1[3]);
                }
                // (the barrier also spreads a wait that ran out: every worker leaves together)
                if (named_sync_or(2, nthr, timed_out)) { timed_out = true; break; }
                for (int e = tid * 2; e < kGramVals; e += nthr * 2) {
                    // add the warps' parts in warp order, two entries at a time
                    float2 sum = *reinterpret_cast<const float2*>(red + e);
#pragma unroll
                    for (int w = 1; w < kFlowWorkers; w++) {
                        const float2 x = *reinterpret_cast<const float2*>(red + w * kGramVals + e);
                        sum.x += x.x; sum.y += x.y;
                    }
                    *reinterpret_cast<float2*>(redsum + e) = sum;
                }
                named_sync(1, nthr);
                // contract to 8 numbers per cell: thread = (number, cell), stored [cell][number]
                if (tid < kSumVals)
                    dst[(long long)j * p.NS * kSumVals + (tid & 15) * 8 + (tid >> 4)] = combine_sums(redsum_a, tid & 15, tid >> 4, lg, W2s);
#pragma unroll
                for (int i = 0; i < kFlowMaxKs; i++) {
                    prv[i][0] = cur[i][0]; prv[i][1] = cur[i][1]; prv[i][2] = cur[i][2]; prv[i][3] = cur[i][3];
                }
            }
        }
    } else if (warp < kFlowWorkers && kSum) {
        // ------------------------------------ sum warps ------------------------------------
        // Warp a owns the slice's 64-channel blocks 2a and 2a + 1: 16 tiles of 8 channels.  sums[nt][0..3]
        // is the accumulator fragment of tile nt: chain slots g and g + 8 (g = lane / 4), channels 2 t
        // and 2 t + 1 of the tile (t = lane % 4).
        if (warp < nsum) {
            float sums[16][4];
#pragma unroll
            for (int nt = 0; nt < 16; nt++)
#pragma unroll
                for (int k = 0; k < 4; k++) sums[nt][k] = 0.f;
            const int g = lane >> 2, t4 = lane & 3;
            const uint32_t lrow = (lane & 7) + ((lane >> 3) & 1) * 8;
            uint32_t xoff[4];
#pragma unroll
            for (int pr = 0; pr < 4; pr++)
                xoff[pr] = 2 * warp * kBlkBytes + lrow * 128 + ((((uint32_t)pr * 2 + (lane >> 4)) ^ (lrow & 7)) << 4);
            const uint32_t woff = 16 + 256 + lrow * 32 + (lane >> 4) * 16;
            const int ntmax = 2 * warp + 1 < p.NB ? 16 : 8;     // an odd block count leaves the last warp one block
            for (int task = blockIdx.x; task < ntasks && !timed_out; task += gridDim.x) {
                const int tk = flow_task(kSum, task, ntasks);
                const FlowItem it = flow_item(p, tk / p.NS);
                const int slice = tk % p.NS;
                const long long chan0 = ((long long)slice * p.NB + 2 * warp) * 64;
                // one record per frame, and a closing one that writes out what the item leaves
                for (int j = 0; j <= it.n; j++, q++) {
                    // (the frame before a run only opens the chains that come in from it: its features are not
                    // added here, so they are not loaded either)
                    const bool frame = j < it.n && !(it.halo && j == 0);
                    const int s = q % p.R;
                    if (!mbar_wait_warp(full_bar + 8 * s, q / p.R, timed_out)) break;
                    const uint32_t rec = recs_base + s * kRecBytes;
                    const uint32_t flush_mask = lds_u32x4(rec).x;
#pragma unroll 1
                    for (int hi = 0; hi < 2; hi++) {
                        const uint32_t m8 = (flush_mask >> (8 * hi)) & 0xffu;
                        if (m8 == 0) continue;
                        // chains that ended: slot g + 8 hi is held by the four lanes of group g, which
                        // scale its 128 channels and write them to the chain's row (or piece)
                        const bool mine = (m8 >> g) & 1u;
                        const uint4 fc = lds_u32x4(rec + 16 + (g + 8 * hi) * 16);       // slot, kind, dst, weight
                        const float inv = mine && fc.y == 0 ? 1.f / __uint_as_float(fc.w) : 1.f;
                        const long long row = (long long)(int)fc.z * p.D + chan0 + 2 * t4;
                        const bool skip = (int)fc.z < 0;                                // a row beyond the capacity
                        // bf16 rows leave in 16-byte stores: the four lanes of a group first exchange their
                        // words so that each holds whole 8-channel tiles (the lanes that take part)
                        const unsigned quads = __ballot_sync(0xffffffffu, mine && fc.y == 0 && !p.out_f32);
#define STTM_FLOW_FLUSH(I0, I1)                                                                               \
    if (fc.y != 0 || p.out_f32) {                                                                             \
        float* dst = (fc.y != 0 ? p.pieces : reinterpret_cast<float*>(p.out)) + row;                          \
        _Pragma("unroll") for (int nt = 0; nt < 16; nt++) {                                                   \
            const float x = sums[nt][I0] * inv, y = sums[nt][I1] * inv;                                       \
            sums[nt][I0] = 0.f;                                                                               \
            sums[nt][I1] = 0.f;                                                                               \
            if (nt < ntmax && !skip) *reinterpret_cast<float2*>(dst + nt * 8) = make_float2(x, y);            \
        }                                                                                                     \
    } else {                                                                                                  \
        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.out) + (row - 2 * t4);                        \
        uint32_t w[16];                                                                                       \
        _Pragma("unroll") for (int nt = 0; nt < 16; nt++) {                                                   \
            w[nt] = pack_bf16x2(sums[nt][I0] * inv, sums[nt][I1] * inv);                                      \
            sums[nt][I0] = 0.f;                                                                               \
            sums[nt][I1] = 0.f;                                                                               \
        }                                                                                                     \
        _Pragma("unroll") for (int m = 0; m < 4; m++) {                                                       \
            uint32_t a0 = w[4 * m], a1 = w[4 * m + 1], a2 = w[4 * m + 2], a3 = w[4 * m + 3], r;               \
            r = __shfl_xor_sync(quads, (t4 & 1) ? a0 : a1, 1); if (t4 & 1) a0 = r; else a1 = r;               \
            r = __shfl_xor_sync(quads, (t4 & 1) ? a2 : a3, 1); if (t4 & 1) a2 = r; else a3 = r;               \
            r = __shfl_xor_sync(quads, (t4 & 2) ? a0 : a2, 2); if (t4 & 2) a0 = r; else a2 = r;               \
            r = __shfl_xor_sync(quads, (t4 & 2) ? a1 : a3, 2); if (t4 & 2) a1 = r; else a3 = r;               \
            const int nt = 4 * m + t4;                      /* lane t4 now holds tile 4 m + t4 whole */      \
            if (nt < ntmax && !skip) *reinterpret_cast<uint4*>(dst + nt * 8) = make_uint4(a0, a1, a2, a3);    \
        }                                                                                                     \
    }
                        if (mine) {
                            if (hi) { STTM_FLOW_FLUSH(2, 3) } else { STTM_FLOW_FLUSH(0, 1) }
                        }
#undef STTM_FLOW_FLUSH
                    }
                    __syncwarp();
                    if (frame) {
                        uint32_t wa[4];
                        ldmatrix_x4(rec + woff, wa);
                        const uint32_t xb = ring_base + s * p.slot_bytes;
#pragma unroll
                        for (int pr = 0; pr < 8; pr++) {
                            if (pr * 2 < ntmax) {
                                uint32_t xb4[4];
                                ldmatrix_x4_trans(xb + xoff[pr & 3] + (pr >> 2) * kBlkBytes, xb4);
                                mma_bf16(sums[2 * pr], wa, xb4[0], xb4[1]);
                                mma_bf16(sums[2 * pr + 1], wa, xb4[2], xb4[3]);
                            }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty_bar + 8 * s);
                }
            }
        }
    } else if (warp == kFlowWorkers) {
        // ------------------------------------- producer -------------------------------------
        // One tensor copy per frame (and, in the sum stage, one plain bulk copy of the frame's
        // record), all on the slot's barrier.
        for (int task = blockIdx.x; task < ntasks && !timed_out; task += gridDim.x) {
            const int tk = flow_task(kSum, task, ntasks);
            const FlowItem it = flow_item(p, tk / p.NS);
            const int slice = tk % p.NS;
            const TileBox bx = p.boxes[it.tile];
            const int nslots = it.n + (kSum ? 1 : 0);
            int seen = 0;                               // records of this run known to exist
            for (int j = 0; j < nslots; j++, q++) {
                const int s = q % p.R;
                const uint32_t bar = full_bar + 8 * s;
                if (q >= p.R && !mbar_wait_warp(empty_bar + 8 * s, q / p.R - 1, timed_out)) break;
                if (kSum && seen <= j) {
                    // the record of this frame exists?  (bounded like every wait; the chain stage's blocks
                    // are all resident before this kernel's first block is)
                    bool late = false;
                    if (lane == 0) {
                        const unsigned long long t0 = global_timer_ns();
                        while ((seen = load_acquire(p.progress + it.item)) <= j) {
                            __nanosleep(100);
                            if (global_timer_ns() - t0 > kWaitLimitNs) { late = true; break; }
                        }
                        asm volatile("fence.proxy.async.global;" ::: "memory");
                    }
                    seen = __shfl_sync(0xffffffffu, seen, 0);
                    if (__any_sync(0xffffffffu, late)) { timed_out = true; break; }
                }
                if (lane == 0) {
                    const bool frame = j < it.n && !(kSum && it.halo && j == 0);
                    mbar_expect_tx(bar, (uint32_t)((frame ? p.slot_bytes : 0) + (kSum ? kRecBytes : 0)));
                    if (frame)
                        tma_load_tile(ring_base + s * p.slot_bytes, &maps.m[bx.kind], bx.x0, bx.y0, slice * p.NB,
                                      it.b * p.T + it.tstart + j, bar);
                    if (kSum)
                        bulk_g2s(recs_base + s * kRecBytes, p.recs + (long long)it.item * (p.F + 2) + j, kRecBytes, bar);
                }
                __syncwarp();
            }
        }
        // the CTA must not end with copies in flight: the last R slots issued have landed?
        for (int qq = max(0, q - p.R); qq < q; qq++) {
            bool late = false;
            mbar_wait_sleep(full_bar + 8 * (qq % p.R), qq / p.R, late);
            timed_out |= late;
        }
    }
    __syncthreads();
    if (timed_out && p.status != nullptr) atomicOr(p.status, kStatusWaitTimeout);
}

}  // namespace sttm
