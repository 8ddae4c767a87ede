// STTM kernels, first generation: one warp per (frame, column), no shared-memory
// staging; three passes over the features (spatial, temporal, averaging).
#pragma once

#include "sttm_device.cuh"

namespace sttm {

constexpr int kWarpsPerBlock = 4;

enum : int { kStatusCapacity = 1 << 4, kStatusNotConverged = 1 << 5 };

// ---------------------------------------------------------------------------------
// Spatial stage (Section 3.2): pyramid, parent-child cosines, coarse-to-fine search.
// One warp reads a column of one frame once (lanes stride over channels), keeps the
// pooled parents in registers and reduces 2 numbers per node with warp shuffles.
// ---------------------------------------------------------------------------------
template <int LEVELS, typename T>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
k_spatial(const T* __restrict__ feats, Geo g, Taus taus, int8_t* __restrict__ cover,
          int32_t* __restrict__ frame_counts, float* __restrict__ sims, float* __restrict__ norms) {
    using C = Col<LEVELS>;
    const int lane = threadIdx.x & 31;
    const long long w = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (w >= (long long)g.B * g.T * g.ncol) return;
    const int col = (int)(w % g.ncol);
    const long long bt = w / g.ncol;
    const int b = (int)(bt / g.T);
    const int y0 = (col / g.Wc) * C::SIDE, x0 = (col % g.Wc) * C::SIDE;
    ColShape<LEVELS> sh;
    sh.init(min(C::SIDE, g.H - y0), min(C::SIDE, g.W - x0));
    const T* base = feats + ((bt * g.H + y0) * g.W + x0) * (long long)g.D;

    float n0[C::NC], d0[C::NC], n1[4], d1[4], n2 = 0.f;
#pragma unroll
    for (int c = 0; c < C::NC; c++) n0[c] = d0[c] = 0.f;
#pragma unroll
    for (int q = 0; q < 4; q++) n1[q] = d1[q] = 0.f;

    for (int d = lane * VEC; d < g.D; d += kSliceCh) {
        float x[C::NC][VEC], p1[4][VEC], p2[VEC];
#pragma unroll
        for (int c = 0; c < C::NC; c++) {
            if (sh.cell(c)) load4(base + ((long long)C::dy(c) * g.W + C::dx(c)) * g.D + d, x[c]);
            else {
#pragma unroll
                for (int v = 0; v < VEC; v++) x[c][v] = 0.f;
            }
        }
        pool_column<LEVELS>(x, sh, p1, p2);
#pragma unroll
        for (int c = 0; c < C::NC; c++)
#pragma unroll
            for (int v = 0; v < VEC; v++) {
                n0[c] = fmaf(x[c][v], x[c][v], n0[c]);
                if constexpr (LEVELS == 3) d0[c] = fmaf(x[c][v], p1[C::quad(c)][v], d0[c]);
                if constexpr (LEVELS == 2) d0[c] = fmaf(x[c][v], p2[v], d0[c]);
            }
        if constexpr (LEVELS == 3) {
#pragma unroll
            for (int q = 0; q < 4; q++)
#pragma unroll
                for (int v = 0; v < VEC; v++) {
                    n1[q] = fmaf(p1[q][v], p1[q][v], n1[q]);
                    d1[q] = fmaf(p1[q][v], p2[v], d1[q]);
                }
        }
        if constexpr (LEVELS >= 2) {
#pragma unroll
            for (int v = 0; v < VEC; v++) n2 = fmaf(p2[v], p2[v], n2);
        }
    }
#pragma unroll
    for (int c = 0; c < C::NC; c++) {
        n0[c] = warp_sum(n0[c]);
        if constexpr (LEVELS >= 2) d0[c] = warp_sum(d0[c]);
    }
    if constexpr (LEVELS == 3) {
#pragma unroll
        for (int q = 0; q < 4; q++) { n1[q] = warp_sum(n1[q]); d1[q] = warp_sum(d1[q]); }
    }
    if constexpr (LEVELS >= 2) n2 = warp_sum(n2);

    // similarities and the coarse-to-fine decision (every lane holds all totals)
    const float tau = taus.s[b];
    float s0[C::NC], s1[4];
    int level_of_quad[4] = {0, 0, 0, 0};
    int top_pass = 0, kept = 0;
    if constexpr (LEVELS == 3) {
        top_pass = 1;
#pragma unroll
        for (int q = 0; q < 4; q++) {
            s1[q] = cos_from(d1[q], n1[q], n2);
            if (sh.quad(q) && !(s1[q] > tau)) top_pass = 0;
            int pass = 1, cells = 0;
#pragma unroll
            for (int k = 0; k < 4; k++) {
                const int c = C::quad_cell(q, k);
                s0[c] = cos_from(d0[c], n0[c], n1[q]);
                if (sh.cell(c)) { cells++; if (!(s0[c] > tau)) pass = 0; }
            }
            level_of_quad[q] = pass;
            if (sh.quad(q)) kept += pass ? 1 : cells;
        }
        if (top_pass) kept = 1;
    } else if constexpr (LEVELS == 2) {
        top_pass = 1;
#pragma unroll
        for (int c = 0; c < C::NC; c++) {
            s0[c] = cos_from(d0[c], n0[c], n2);
            if (sh.cell(c) && !(s0[c] > tau)) top_pass = 0;
        }
        kept = top_pass ? 1 : __popc(sh.valid);
    } else {
        kept = 1;
    }

    // outputs: lane c writes cell c, lanes NC.. write the inner nodes
    const long long frame_cell0 = bt * g.HW;
#pragma unroll
    for (int c = 0; c < C::NC; c++) {
        if (lane == c && sh.cell(c)) {
            int lv = 0;
            if constexpr (LEVELS == 3) lv = top_pass ? 2 : level_of_quad[C::quad(c)];
            if constexpr (LEVELS == 2) lv = top_pass ? 1 : 0;
            const int cell = (y0 + C::dy(c)) * g.W + x0 + C::dx(c);
            cover[frame_cell0 + cell] = (int8_t)lv;
            if (sims != nullptr && LEVELS >= 2) sims[bt * g.nsim + cell] = s0[c];
        }
    }
    float* nrm = norms + (bt * g.ncol + col) * C::NN;
#pragma unroll
    for (int c = 0; c < C::NC; c++) if (lane == c) nrm[c] = n0[c];
    if constexpr (LEVELS == 3) {
#pragma unroll
        for (int q = 0; q < 4; q++) {
            if (lane == C::NC + q) {
                nrm[C::NC + q] = n1[q];
                if (sims != nullptr && sh.quad(q)) {
                    const int i1 = (y0 >> 1) + (q >> 1), j1 = (x0 >> 1) + (q & 1);
                    sims[bt * g.nsim + g.HW + i1 * g.W1 + j1] = s1[q];
                }
            }
        }
    }
    if constexpr (LEVELS >= 2) if (lane == C::NN - 1) nrm[C::NN - 1] = n2;
    if (lane == 0 && frame_counts != nullptr) atomicAdd(frame_counts + bt, kept);
}

// ---------------------------------------------------------------------------------
// Temporal stage (Section 3.3), similarities and link choice.  One warp handles a
// column of frames t-1 and t.  Two kept nodes overlap exactly when one contains the
// other, so every compared pair is named by the anchor cell of its finer node; the
// warp accumulates one dot product per such cell.
// ---------------------------------------------------------------------------------
template <int LEVELS, typename T>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
k_temporal(const T* __restrict__ feats, Geo g, Taus taus, const int8_t* __restrict__ cover,
           const float* __restrict__ norms, int32_t* __restrict__ link, float* __restrict__ tsim,
           int match_best) {
    using C = Col<LEVELS>;
    const int lane = threadIdx.x & 31;
    const long long w = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    if (w >= (long long)g.B * g.T * g.ncol) return;
    const int col = (int)(w % g.ncol);
    const long long bt = w / g.ncol;
    const int b = (int)(bt / g.T), t = (int)(bt % g.T);
    const int y0 = (col / g.Wc) * C::SIDE, x0 = (col % g.Wc) * C::SIDE;
    ColShape<LEVELS> sh;
    sh.init(min(C::SIDE, g.H - y0), min(C::SIDE, g.W - x0));

    const bool mine = lane < C::NC && sh.cell(lane);
    const int my_cell = mine ? (y0 + C::dy(lane)) * g.W + x0 + C::dx(lane) : 0;
    const long long my_idx = (long long)b * g.N + (long long)t * g.HW + my_cell;
    if (t == 0) {
        if (mine) {
            link[my_idx] = -1;
            if (tsim != nullptr) tsim[my_idx] = __int_as_float(0x7fc00000);
        }
        return;
    }
    const int lc_mine = mine ? cover[bt * g.HW + my_cell] : 0;
    const int lp_mine = mine ? cover[(bt - 1) * g.HW + my_cell] : 0;
    const uint32_t lcm = __reduce_or_sync(0xffffffffu, mine ? (uint32_t)lc_mine << (2 * lane) : 0u);
    const uint32_t lpm = __reduce_or_sync(0xffffffffu, mine ? (uint32_t)lp_mine << (2 * lane) : 0u);

    // rep bit c: cell c is the anchor of the finer node of the pair (v(c), u(c))
    uint32_t rep = 0;
#pragma unroll
    for (int c = 0; c < C::NC; c++) {
        const int lv = (lcm >> (2 * c)) & 3, lu = (lpm >> (2 * c)) & 3;
        if (sh.cell(c) && is_anchor<LEVELS>(c, min(lv, lu))) rep |= 1u << c;
    }

    const T* cur = feats + ((bt * g.H + y0) * g.W + x0) * (long long)g.D;
    const T* prv = cur - (long long)g.HW * g.D;
    float acc[C::NC];
#pragma unroll
    for (int c = 0; c < C::NC; c++) acc[c] = 0.f;

    for (int d = lane * VEC; d < g.D; d += kSliceCh) {
        float xc[C::NC][VEC], xp[C::NC][VEC], p1c[4][VEC], p2c[VEC], p1p[4][VEC], p2p[VEC];
#pragma unroll
        for (int c = 0; c < C::NC; c++) {
            if (sh.cell(c)) {
                const long long off = ((long long)C::dy(c) * g.W + C::dx(c)) * g.D + d;
                load4(cur + off, xc[c]);
                load4(prv + off, xp[c]);
            } else {
#pragma unroll
                for (int v = 0; v < VEC; v++) xc[c][v] = xp[c][v] = 0.f;
            }
        }
        pool_column<LEVELS>(xc, sh, p1c, p2c);
        pool_column<LEVELS>(xp, sh, p1p, p2p);
#pragma unroll
        for (int c = 0; c < C::NC; c++) {
            if ((rep >> c) & 1u) {
                const int lv = (lcm >> (2 * c)) & 3, lu = (lpm >> (2 * c)) & 3;
#pragma unroll
                for (int v = 0; v < VEC; v++)
                    acc[c] = fmaf(node_feat<LEVELS>(lv, c, v, xc, p1c, p2c),
                                  node_feat<LEVELS>(lu, c, v, xp, p1p, p2p), acc[c]);
            }
        }
    }

    const float* nc = norms + (bt * g.ncol + col) * C::NN;
    const float* np = nc - (long long)g.ncol * C::NN;
    const float tau = taus.t[b];
    // lane a keeps the link of the node of frame t anchored at cell a; pairs are visited
    // in row-major order of their finer node, so the first passing one is the top-left (and
    // with match_best a later one only replaces it when it is strictly more similar)
    int my_link = -1;
    float my_best = 0.f;
    float my_sim = __int_as_float(0x7fc00000);
#pragma unroll
    for (int c = 0; c < C::NC; c++) {
        if ((rep >> c) & 1u) {
            const int lv = (lcm >> (2 * c)) & 3, lu = (lpm >> (2 * c)) & 3;
            const float dot = warp_sum(acc[c]);
            const float s = cos_from(dot, nc[C::node_of(c, lv)], np[C::node_of(c, lu)]);
            if (lane == c) my_sim = s;
            const int mv = ~((1 << lv) - 1), mu = ~((1 << lu) - 1);
            const int anchor_v = (C::dy(c) & mv) * C::SIDE + (C::dx(c) & mv);
            const int anchor_u = (t - 1) * g.HW + (y0 + (C::dy(c) & mu)) * g.W + x0 + (C::dx(c) & mu);
            if (lane == anchor_v && s > tau && (my_link < 0 || (match_best && s > my_best))) {
                my_link = anchor_u;
                my_best = s;
            }
        }
    }
    const int mvm = ~((1 << lc_mine) - 1);
    const int src = mine ? (C::dy(lane) & mvm) * C::SIDE + (C::dx(lane) & mvm) : 0;
    const int node_link = __shfl_sync(0xffffffffu, my_link, src);
    if (mine) {
        link[my_idx] = node_link;
        if (tsim != nullptr) tsim[my_idx] = my_sim;
    }
}

// ---------------------------------------------------------------------------------
// Roots (Section 3.3, "common root node"): pointer jumping inside one column.
// root[] starts as "the node I am linked to, else my own anchor" and is squared until
// nothing changes; a chain moves one frame per link, so ceil(log2 T) rounds suffice.
// ---------------------------------------------------------------------------------
template <int LEVELS>
__global__ void __launch_bounds__(256)
k_roots(Geo g, const int8_t* __restrict__ cover, const int32_t* __restrict__ link, int32_t* root,
        int32_t* status, int max_rounds) {
    using C = Col<LEVELS>;
    const int col = blockIdx.x % g.ncol, b = blockIdx.x / g.ncol;
    const int y0 = (col / g.Wc) * C::SIDE, x0 = (col % g.Wc) * C::SIDE;
    const int rows = min(C::SIDE, g.H - y0), cols = min(C::SIDE, g.W - x0);
    const int entries = g.T * C::NC;
    const long long vb = (long long)b * g.N;
    for (int e = threadIdx.x; e < entries; e += blockDim.x) {
        const int t = e / C::NC, c = e % C::NC;
        if (C::dy(c) >= rows || C::dx(c) >= cols) continue;
        const int cell = t * g.HW + (y0 + C::dy(c)) * g.W + x0 + C::dx(c);
        const int lv = cover[vb + cell];
        const int m = ~((1 << lv) - 1);
        const int anchor = t * g.HW + (y0 + (C::dy(c) & m)) * g.W + x0 + (C::dx(c) & m);
        const int lk = link[vb + cell];
        root[vb + cell] = lk >= 0 ? lk : anchor;
    }
    __syncthreads();
    int round = 0;
    while (true) {
        int changed = 0;
        for (int e = threadIdx.x; e < entries; e += blockDim.x) {
            const int t = e / C::NC, c = e % C::NC;
            if (C::dy(c) >= rows || C::dx(c) >= cols) continue;
            const int cell = t * g.HW + (y0 + C::dy(c)) * g.W + x0 + C::dx(c);
            const int r = __ldcg(root + vb + cell);
            const int rr = __ldcg(root + vb + r);
            if (rr != r) { __stcg(root + vb + cell, rr); changed = 1; }
        }
        if (!__syncthreads_or(changed)) break;
        if (++round > max_rounds) {
            if (threadIdx.x == 0 && status != nullptr) atomicOr(status, kStatusNotConverged);
            break;
        }
    }
}

// ---------------------------------------------------------------------------------
// Ordering (Section 3.4): a cell is a surviving token iff it is the anchor of a kept
// node that has no link.  Rows are numbered in (video, frame, y, x) order.
// ---------------------------------------------------------------------------------
__device__ __forceinline__ bool is_root_anchor(const Geo& g, int cell_in_frame, int lv, int lk) {
    const int y = cell_in_frame / g.W, x = cell_in_frame % g.W;
    const int m = (1 << lv) - 1;
    return lk < 0 && ((y & m) | (x & m)) == 0;
}

// block-wide exclusive scan of one int per thread (blockDim.x <= 1024); returns the
// exclusive prefix and the block total
__device__ __forceinline__ int block_exclusive_scan(int v, int& total, int* smem33) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    __syncthreads();
    if (lane == 31) smem33[wid] = inc;
    __syncthreads();
    if (wid == 0) {
        int s = lane < (int)((blockDim.x + 31) >> 5) ? smem33[lane] : 0;
        int si = s;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int n = __shfl_up_sync(0xffffffffu, si, o);
            if (lane >= o) si += n;
        }
        smem33[lane] = si - s;
        if (lane == 31) smem33[32] = si;
    }
    __syncthreads();
    total = smem33[32];
    return inc - v + smem33[wid];
}

// one block per frame: number of surviving tokens in the frame
__global__ void __launch_bounds__(256)
k_frame_roots(Geo g, const int8_t* __restrict__ cover, const int32_t* __restrict__ link,
              int32_t* __restrict__ frame_roots) {
    wait_for_prior_kernel();
    const long long bt = blockIdx.x;
    int n = 0;
    for (int cell = threadIdx.x; cell < g.HW; cell += blockDim.x)
        n += is_root_anchor(g, cell, cover[bt * g.HW + cell], link[bt * g.HW + cell]) ? 1 : 0;
    __shared__ int sm[33];
    int total;
    block_exclusive_scan(n, total, sm);
    if (threadIdx.x == 0) frame_roots[bt] = total;
}

// one block: per video, exclusive scan of the frame counts; video offsets
__global__ void __launch_bounds__(1024)
k_scan_frames(Geo g, const int32_t* __restrict__ frame_roots, int32_t* __restrict__ frame_base,
              int32_t* __restrict__ out_count, long long* __restrict__ vid_off, int64_t* out_offsets) {
    wait_for_prior_kernel();
    __shared__ int sm[33];
    __shared__ long long running_rows;
    if (threadIdx.x == 0) running_rows = 0;
    __syncthreads();
    for (int b = 0; b < g.B; b++) {
        int carry = 0;
        for (int t0 = 0; t0 < g.T; t0 += blockDim.x) {
            const int t = t0 + threadIdx.x;
            const int v = t < g.T ? frame_roots[(long long)b * g.T + t] : 0;
            int total;
            const int ex = block_exclusive_scan(v, total, sm);
            if (t < g.T) frame_base[(long long)b * g.T + t] = carry + ex;
            carry += total;
            __syncthreads();
        }
        if (threadIdx.x == 0) {
            out_count[b] = carry;
            vid_off[b] = running_rows;
            if (out_offsets != nullptr) out_offsets[b] = running_rows;
            running_rows += carry;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        vid_off[g.B] = running_rows;
        if (out_offsets != nullptr) out_offsets[g.B] = running_rows;
    }
}

// one block per frame: row of every surviving token, position ids
__global__ void __launch_bounds__(256)
k_rows(Geo g, const int8_t* __restrict__ cover, const int32_t* __restrict__ link,
       const int32_t* __restrict__ frame_base, const long long* __restrict__ vid_off,
       int32_t* __restrict__ row_at_root, int32_t* __restrict__ row_anchor, int32_t* __restrict__ out_pos,
       long long capacity, int pos_mode, int32_t* status) {
    wait_for_prior_kernel();
    __shared__ int sm[33];
    const long long bt = blockIdx.x;
    const int b = (int)(bt / g.T), t = (int)(bt % g.T);
    int carry = frame_base[bt];
    const long long off = vid_off[b];
    for (int c0 = 0; c0 < g.HW; c0 += blockDim.x) {
        const int cell = c0 + threadIdx.x;
        const int flag = cell < g.HW && is_root_anchor(g, cell, cover[bt * g.HW + cell], link[bt * g.HW + cell]);
        int total;
        const int ex = block_exclusive_scan(flag, total, sm);
        if (flag) {
            const int row = carry + ex;
            const long long grow = off + row;
            row_at_root[bt * g.HW + cell] = row;
            row_anchor[grow] = t * g.HW + cell;
            if (grow < capacity) out_pos[grow] = pos_mode ? row : t * g.HW + cell;
            else if (status != nullptr) atomicOr(status, kStatusCapacity);
        }
        carry += total;
        __syncthreads();
    }
}

// The same with the scan folded in (one launch less): every block adds up the root counts of the
// frames before its own (all frames of the earlier videos, the earlier frames of its video); the
// first block of a video also writes the video's count and offset.
__global__ void __launch_bounds__(256)
k_rows_scan(Geo g, const int8_t* __restrict__ cover, const int32_t* __restrict__ link,
            const int32_t* __restrict__ frame_roots, int32_t* __restrict__ out_count, long long* __restrict__ vid_off,
            int64_t* out_offsets, int32_t* __restrict__ row_at_root, int32_t* __restrict__ row_anchor,
            int32_t* __restrict__ out_pos, long long capacity, int pos_mode, int32_t* status) {
    wait_for_prior_kernel();
    __shared__ int sm[33];
    const long long bt = blockIdx.x;
    const int b = (int)(bt / g.T), t = (int)(bt % g.T);
    int before_videos = 0, before_frames = 0, after_frames = 0;
    for (int i = threadIdx.x; i < b * g.T; i += blockDim.x) before_videos += frame_roots[i];
    for (int i = threadIdx.x; i < g.T; i += blockDim.x) {
        const int v = frame_roots[(long long)b * g.T + i];
        if (i < t) before_frames += v; else after_frames += v;
    }
    // the three totals in one pass: warp sums, then one thread per total adds the warps' sums
    __shared__ int tot3[3][8];
    {
        int v0 = before_videos, v1 = before_frames, v2 = after_frames;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            v0 += __shfl_xor_sync(0xffffffffu, v0, o);
            v1 += __shfl_xor_sync(0xffffffffu, v1, o);
            v2 += __shfl_xor_sync(0xffffffffu, v2, o);
        }
        if ((threadIdx.x & 31) == 0) {
            tot3[0][threadIdx.x >> 5] = v0;
            tot3[1][threadIdx.x >> 5] = v1;
            tot3[2][threadIdx.x >> 5] = v2;
        }
    }
    __syncthreads();
    int off_i = 0, carry = 0, rest = 0;
#pragma unroll
    for (int w = 0; w < 8; w++) { off_i += tot3[0][w]; carry += tot3[1][w]; rest += tot3[2][w]; }
    const long long off = off_i;
    if (t == 0 && threadIdx.x == 0) {
        out_count[b] = carry + rest;
        vid_off[b] = off;
        if (out_offsets != nullptr) out_offsets[b] = off;
        if (b == g.B - 1) {
            vid_off[g.B] = off + carry + rest;
            if (out_offsets != nullptr) out_offsets[g.B] = off + carry + rest;
        }
    }
    for (int c0 = 0; c0 < g.HW; c0 += blockDim.x) {
        const int cell = c0 + threadIdx.x;
        const int flag = cell < g.HW && is_root_anchor(g, cell, cover[bt * g.HW + cell], link[bt * g.HW + cell]);
        int total;
        const int ex = block_exclusive_scan(flag, total, sm);
        if (flag) {
            const int row = carry + ex;
            const long long grow = off + row;
            row_at_root[bt * g.HW + cell] = row;
            row_anchor[grow] = t * g.HW + cell;
            if (grow < capacity) out_pos[grow] = pos_mode ? row : t * g.HW + cell;
            else if (status != nullptr) atomicOr(status, kStatusCapacity);
        }
        carry += total;
        __syncthreads();
    }
}

// one thread per cell: row of the cell's root; per row: total weight and last frame
__global__ void __launch_bounds__(256)
k_members(Geo g, const int8_t* __restrict__ cover, const int32_t* __restrict__ root,
          const int32_t* __restrict__ row_at_root, const long long* __restrict__ vid_off,
          int32_t* __restrict__ cell_row, int32_t* merge_map, int32_t* __restrict__ row_weight,
          int32_t* __restrict__ row_last_t, int weight_mode) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)g.B * g.N) return;
    const int b = (int)(i / g.N), c = (int)(i % g.N);
    const int t = c / g.HW, cell = c % g.HW;
    const int y = cell / g.W, x = cell % g.W;
    const int r = root[i];
    const int row = row_at_root[(long long)b * g.N + r];
    const long long grow = vid_off[b] + row;
    cell_row[i] = (int32_t)grow;
    if (merge_map != nullptr) merge_map[i] = row;
    const int lv = cover[i], m = (1 << lv) - 1;
    if (((y & m) | (x & m)) == 0) {
        const int side = 1 << lv;
        const int wgt = weight_mode ? min(side, g.H - y) * min(side, g.W - x) : 1;
        atomicAdd(row_weight + grow, wgt);
        atomicMax(row_last_t + grow, t);
    }
}

// one thread per row: rows whose members span several time chunks get a run of slots in
// the partial-sum buffer (one per chunk)
__global__ void __launch_bounds__(256)
k_span(Geo g, int Tc, const long long* __restrict__ vid_off, const int32_t* __restrict__ row_anchor,
       const int32_t* __restrict__ row_last_t, int32_t* __restrict__ span_off, int32_t* span_total) {
    const long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= vid_off[g.B]) return;
    const int k0 = (row_anchor[r] / g.HW) / Tc, k1 = row_last_t[r] / Tc;
    span_off[r] = k1 > k0 ? atomicAdd(span_total, k1 - k0 + 1) : -1;
}

// ---------------------------------------------------------------------------------
// Averaging into roots (Section 3.3, "merged into a single token").  One warp owns
// (video, column, time chunk, 128-channel slice) and walks its frames in order.  The
// sums of the chains that are alive in the column (at most one per cell) sit in shared
// memory; a chain that gets no member in a frame is finished and is written out.
// Rows whose members lie in more than one chunk go to an fp32 partial buffer and are
// combined, in chunk order, by k_combine.
// ---------------------------------------------------------------------------------
constexpr int kAccWarps = 8;

template <int LEVELS, typename T, typename OutT>
__global__ void __launch_bounds__(kAccWarps * 32)
k_accumulate(const T* __restrict__ feats, Geo g, int Tc, int nchunk, int nslice,
             const int8_t* __restrict__ cover, const int32_t* __restrict__ cell_row,
             const int32_t* __restrict__ row_weight, const int32_t* __restrict__ span_off,
             const int32_t* __restrict__ row_anchor, float* __restrict__ partial,
             OutT* __restrict__ out, long long capacity, int weight_mode) {
    using C = Col<LEVELS>;
    extern __shared__ float acc_smem[];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    float* acc = acc_smem + (size_t)wib * C::NC * kSliceCh + lane * VEC;
    long long w = (long long)blockIdx.x * kAccWarps + wib;
    if (w >= (long long)g.B * g.ncol * nchunk * nslice) return;
    const int s = (int)(w % nslice); w /= nslice;
    const int col = (int)(w % g.ncol); w /= g.ncol;
    const int k = (int)(w % nchunk);
    const int b = (int)(w / nchunk);
    const int y0 = (col / g.Wc) * C::SIDE, x0 = (col % g.Wc) * C::SIDE;
    ColShape<LEVELS> sh;
    sh.init(min(C::SIDE, g.H - y0), min(C::SIDE, g.W - x0));
    const int d = s * kSliceCh + lane * VEC;
    const bool active = d < g.D;
    const bool mine = lane < C::NC && sh.cell(lane);
    const int my_cell = mine ? (y0 + C::dy(lane)) * g.W + x0 + C::dx(lane) : 0;
    const int t_begin = k * Tc, t_end = min(g.T, t_begin + Tc);

    int slot_row = -1;    // lane s < NC: global row held by slot s, -1 = free

    auto flush = [&](int sl, int r) {
        if (!active || r >= capacity) return;
        float v[VEC];
#pragma unroll
        for (int i = 0; i < VEC; i++) v[i] = acc[sl * kSliceCh + i];
        const int so = span_off[r];
        if (so < 0) {
            const float wsum = (float)row_weight[r];
#pragma unroll
            for (int i = 0; i < VEC; i++) v[i] = v[i] / wsum;
            store4(out + (long long)r * g.D + d, v);
        } else {
            const int k0 = (row_anchor[r] / g.HW) / Tc;
            store4(partial + (long long)(so + k - k0) * g.D + d, v);
        }
    };

    for (int t = t_begin; t < t_end; t++) {
        const long long fc = ((long long)b * g.T + t) * g.HW;
        const int lv_mine = mine ? cover[fc + my_cell] : 0;
        const int row_mine = mine ? cell_row[fc + my_cell] : -1;
        const uint32_t lcm = __reduce_or_sync(0xffffffffu, mine ? (uint32_t)lv_mine << (2 * lane) : 0u);

        // chains without a member in this frame are finished
        bool present = false;
#pragma unroll
        for (int c = 0; c < C::NC; c++) {
            const int r = __shfl_sync(0xffffffffu, row_mine, c);
            present |= (r == slot_row);
        }
        uint32_t dead = __ballot_sync(0xffffffffu, lane < C::NC && slot_row >= 0 && !present);
        while (dead) {
            const int sl = __ffs(dead) - 1;
            dead &= dead - 1;
            flush(sl, __shfl_sync(0xffffffffu, slot_row, sl));
            if (lane == sl) slot_row = -1;
        }

        float x[C::NC][VEC], p1[4][VEC], p2[VEC];
        const T* base = feats + (((long long)b * g.T + t) * g.HW + y0 * g.W + x0) * (long long)g.D + d;
#pragma unroll
        for (int c = 0; c < C::NC; c++) {
            if (active && sh.cell(c)) load4(base + ((long long)C::dy(c) * g.W + C::dx(c)) * g.D, x[c]);
            else {
#pragma unroll
                for (int v = 0; v < VEC; v++) x[c][v] = 0.f;
            }
        }
        pool_column<LEVELS>(x, sh, p1, p2);
#pragma unroll
        for (int c = 0; c < C::NC; c++) {
            const int lv = (lcm >> (2 * c)) & 3;
            if (sh.cell(c) && is_anchor<LEVELS>(c, lv)) {
                const int r = __shfl_sync(0xffffffffu, row_mine, c);
                uint32_t m = __ballot_sync(0xffffffffu, lane < C::NC && slot_row == r);
                bool fresh = false;
                if (m == 0) {
                    m = __ballot_sync(0xffffffffu, lane < C::NC && slot_row < 0);
                    fresh = true;
                }
                const int sl = __ffs(m) - 1;
                if (fresh && lane == sl) slot_row = r;
                float wgt = 1.f;
                if (weight_mode) {
                    const int side = 1 << lv;
                    wgt = (float)(min(side, g.H - y0 - C::dy(c)) * min(side, g.W - x0 - C::dx(c)));
                }
#pragma unroll
                for (int v = 0; v < VEC; v++) {
                    const float f = wgt * node_feat<LEVELS>(lv, c, v, x, p1, p2);
                    acc[sl * kSliceCh + v] = fresh ? f : acc[sl * kSliceCh + v] + f;
                }
            }
        }
    }
    uint32_t live = __ballot_sync(0xffffffffu, lane < C::NC && slot_row >= 0);
    while (live) {
        const int sl = __ffs(live) - 1;
        live &= live - 1;
        flush(sl, __shfl_sync(0xffffffffu, slot_row, sl));
    }
}

// rows that span several chunks: add their partial sums in chunk order and divide
template <typename OutT>
__global__ void __launch_bounds__(256)
k_combine(Geo g, int Tc, const long long* __restrict__ vid_off, const int32_t* __restrict__ span_off,
          const int32_t* __restrict__ row_anchor, const int32_t* __restrict__ row_last_t,
          const int32_t* __restrict__ row_weight, const float* __restrict__ partial,
          OutT* __restrict__ out, long long capacity) {
    const int lane = threadIdx.x & 31;
    const long long nrows = min(vid_off[g.B], capacity);
    const long long nwarps = (long long)gridDim.x * (blockDim.x >> 5);
    for (long long r = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); r < nrows; r += nwarps) {
        const int so = span_off[r];
        if (so < 0) continue;
        const int n = row_last_t[r] / Tc - (row_anchor[r] / g.HW) / Tc + 1;
        const float wsum = (float)row_weight[r];
        for (int d = lane * VEC; d < g.D; d += kSliceCh) {
            float sum[VEC] = {0.f, 0.f, 0.f, 0.f};
            for (int j = 0; j < n; j++) {
                const float4 p = *reinterpret_cast<const float4*>(partial + (long long)(so + j) * g.D + d);
                sum[0] += p.x; sum[1] += p.y; sum[2] += p.z; sum[3] += p.w;
            }
#pragma unroll
            for (int v = 0; v < VEC; v++) sum[v] = sum[v] / wsum;
            store4(out + r * g.D + d, sum);
        }
    }
}

// ---------------------------------------------------------------------------------
// "Merged" positions (Section 3.4): per output row the mean of its member cells' indices.
// Integer sums (exact), one division per row.
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
k_pos_accumulate(int B, long long N, const int32_t* __restrict__ merge_map, const int64_t* __restrict__ out_offsets,
                 unsigned long long* __restrict__ sum, unsigned int* __restrict__ cnt, long long capacity,
                 int32_t* status) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)B * N) return;
    const int b = (int)(i / N);
    const long long row = out_offsets[b] + merge_map[i];
    if (row >= capacity) {
        if (status != nullptr) atomicOr(status, kStatusCapacity);
        return;
    }
    atomicAdd(sum + row, (unsigned long long)(i - (long long)b * N));
    atomicAdd(cnt + row, 1u);
}

__global__ void __launch_bounds__(256)
k_pos_finish(long long rows_max, const int64_t* __restrict__ out_offsets, int B,
             const unsigned long long* __restrict__ sum, const unsigned int* __restrict__ cnt,
             float* __restrict__ out_pos_mean) {
    const long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= rows_max || r >= out_offsets[B]) return;
    out_pos_mean[r] = cnt[r] ? (float)((double)sum[r] / (double)cnt[r]) : 0.f;
}

}  // namespace sttm
