// General path for quadtrees of more than three levels (grids of more than 16 cells a side
// with a 4x4 coarsest map, or the 2x2 coarsest map of the paper's ablation on a 13x13 / 14x14 /
// 16x16 grid).  Plain kernels, one step of Section 3 each, pooled features kept in fp32 in the
// workspace; nothing here is tuned for speed: the fused kernel covers the shapes that matter there.
#pragma once

#include "sttm_device.cuh"
#include "sttm_kernels.cuh"

namespace sttm {

constexpr int kMaxLevels = 8;

// sizes of the pyramid's maps and where a level starts in the per-frame node lists
struct Pyr {
    int L;
    int H[kMaxLevels], W[kMaxLevels];
    int noff[kMaxLevels];       // all levels, level 0 first
    int uoff[kMaxLevels];       // pooled levels only (level 1 first); uoff[0] unused
    int nodes, upper;           // nodes per frame: all levels / pooled levels
};

// four channels of a node's feature: level 0 from the input, higher levels from the pooled maps
template <typename T>
__device__ __forceinline__ void node4(const T* __restrict__ feats, const float* __restrict__ pooled, const Geo& g,
                                      const Pyr& py, long long bt, int l, int idx, int d, float (&x)[VEC]) {
    if (l == 0) load4(feats + ((bt * g.HW + idx) * (long long)g.D + d), x);
    else load4(pooled + ((bt * py.upper + py.uoff[l] + idx) * (long long)g.D + d), x);
}

// Section 3.2: level l = 2x2 average pooling of level l - 1 (border parents average the children
// that exist).  One warp per node of level l; with the children in registers it also takes what the
// search needs: the node's squared norm, every child's dot product with it and, at level 1, the
// children's (the cells') squared norms.
template <typename T>
__global__ void __launch_bounds__(256)
k_gen_pool(const T* __restrict__ feats, float* __restrict__ pooled, Geo g, Pyr py, int l,
           float* __restrict__ norms, float* __restrict__ dots) {
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const int per = py.H[l] * py.W[l];
    if (warp >= (long long)g.B * g.T * per) return;
    const long long bt = warp / per;
    const int idx = (int)(warp % per), i = idx / py.W[l], j = idx % py.W[l];
    int child[4], n = 0;
    for (int a = 0; a < 2; a++)
        for (int b = 0; b < 2; b++)
            if (2 * i + a < py.H[l - 1] && 2 * j + b < py.W[l - 1]) child[n++] = (2 * i + a) * py.W[l - 1] + 2 * j + b;
    const float inv = 1.f / (float)n;
    float* dst = pooled + (bt * py.upper + py.uoff[l] + idx) * (long long)g.D;
    float nn = 0.f, dp[4] = {0.f, 0.f, 0.f, 0.f}, cn[4] = {0.f, 0.f, 0.f, 0.f};
    for (int d = lane * VEC; d < g.D; d += 32 * VEC) {
        float s[VEC] = {0.f, 0.f, 0.f, 0.f};
        float x[4][VEC];
#pragma unroll
        for (int c = 0; c < 4; c++) {
            if (c < n) {
                node4(feats, pooled, g, py, bt, l - 1, child[c], d, x[c]);
#pragma unroll
                for (int v = 0; v < VEC; v++) s[v] += x[c][v];
            }
        }
#pragma unroll
        for (int v = 0; v < VEC; v++) s[v] *= inv;
        store4(dst + d, s);
#pragma unroll
        for (int v = 0; v < VEC; v++) nn = fmaf(s[v], s[v], nn);
#pragma unroll
        for (int c = 0; c < 4; c++) {
            if (c < n) {
#pragma unroll
                for (int v = 0; v < VEC; v++) {
                    dp[c] = fmaf(x[c][v], s[v], dp[c]);
                    cn[c] = fmaf(x[c][v], x[c][v], cn[c]);
                }
            }
        }
    }
    nn = warp_sum(nn);
#pragma unroll
    for (int c = 0; c < 4; c++) { dp[c] = warp_sum(dp[c]); cn[c] = warp_sum(cn[c]); }
    if (lane == 0) {
        const long long at = bt * py.nodes;
        norms[at + py.noff[l] + idx] = nn;
        if (l + 1 == py.L) dots[at + py.noff[l] + idx] = 0.f;
#pragma unroll
        for (int c = 0; c < 4; c++) {
            if (c < n) {
                dots[at + py.noff[l - 1] + child[c]] = dp[c];
                if (l == 1) norms[at + child[c]] = cn[c];
            }
        }
    }
}

// Levels 1 and 2 in one pass over the cells: one warp per node of level 2 holds its (up to) 4 x 4 cells,
// forms its level-1 children and itself, and takes all the norms and dot products of the three levels
// (same sums in the same order as two passes of k_gen_pool; level 1 is not read back).
template <typename T>
__global__ void __launch_bounds__(128)
k_gen_pool2(const T* __restrict__ feats, float* __restrict__ pooled, Geo g, Pyr py, float* __restrict__ norms,
            float* __restrict__ dots) {
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const int per = py.H[2] * py.W[2];
    if (warp >= (long long)g.B * g.T * per) return;
    const long long bt = warp / per;
    const int idx2 = (int)(warp % per), i2 = idx2 / py.W[2], j2 = idx2 % py.W[2];
    int kid[4], nk = 0;                 // level-1 children of the node
    int cell[4][4], nc[4];              // their cells
    for (int a = 0; a < 2; a++)
        for (int b = 0; b < 2; b++) {
            const int i1 = 2 * i2 + a, j1 = 2 * j2 + b;
            if (i1 >= py.H[1] || j1 >= py.W[1]) continue;
            kid[nk] = i1 * py.W[1] + j1;
            nc[nk] = 0;
            for (int a0 = 0; a0 < 2; a0++)
                for (int b0 = 0; b0 < 2; b0++)
                    if (2 * i1 + a0 < py.H[0] && 2 * j1 + b0 < py.W[0]) cell[nk][nc[nk]++] = (2 * i1 + a0) * py.W[0] + 2 * j1 + b0;
            nk++;
        }
    float n2 = 0.f, n1[4] = {0.f, 0.f, 0.f, 0.f}, d1[4] = {0.f, 0.f, 0.f, 0.f};
    float cn[4][4], d0[4][4];
#pragma unroll
    for (int k = 0; k < 4; k++)
#pragma unroll
        for (int c = 0; c < 4; c++) cn[k][c] = d0[k][c] = 0.f;
    float* dst2 = pooled + (bt * py.upper + py.uoff[2] + idx2) * (long long)g.D;
    for (int d = lane * VEC; d < g.D; d += 32 * VEC) {
        float s2[VEC] = {0.f, 0.f, 0.f, 0.f};
        float s1[4][VEC];
#pragma unroll
        for (int k = 0; k < 4; k++) {
            if (k < nk) {
                float x[4][VEC];
#pragma unroll
                for (int v = 0; v < VEC; v++) s1[k][v] = 0.f;
#pragma unroll
                for (int c = 0; c < 4; c++) {
                    if (c < nc[k]) {
                        load4(feats + ((bt * g.HW + cell[k][c]) * (long long)g.D + d), x[c]);
#pragma unroll
                        for (int v = 0; v < VEC; v++) s1[k][v] += x[c][v];
                    }
                }
                const float inv1 = 1.f / (float)nc[k];
#pragma unroll
                for (int v = 0; v < VEC; v++) s1[k][v] *= inv1;
                store4(pooled + ((bt * py.upper + py.uoff[1] + kid[k]) * (long long)g.D + d), s1[k]);
#pragma unroll
                for (int v = 0; v < VEC; v++) n1[k] = fmaf(s1[k][v], s1[k][v], n1[k]);
#pragma unroll
                for (int c = 0; c < 4; c++) {
                    if (c < nc[k]) {
#pragma unroll
                        for (int v = 0; v < VEC; v++) {
                            d0[k][c] = fmaf(x[c][v], s1[k][v], d0[k][c]);
                            cn[k][c] = fmaf(x[c][v], x[c][v], cn[k][c]);
                        }
                    }
                }
#pragma unroll
                for (int v = 0; v < VEC; v++) s2[v] += s1[k][v];
            }
        }
        const float inv2 = 1.f / (float)nk;
#pragma unroll
        for (int v = 0; v < VEC; v++) s2[v] *= inv2;
        store4(dst2 + d, s2);
#pragma unroll
        for (int v = 0; v < VEC; v++) n2 = fmaf(s2[v], s2[v], n2);
#pragma unroll
        for (int k = 0; k < 4; k++) {
            if (k < nk) {
#pragma unroll
                for (int v = 0; v < VEC; v++) d1[k] = fmaf(s1[k][v], s2[v], d1[k]);
            }
        }
    }
    n2 = warp_sum(n2);
#pragma unroll
    for (int k = 0; k < 4; k++) {
        n1[k] = warp_sum(n1[k]);
        d1[k] = warp_sum(d1[k]);
#pragma unroll
        for (int c = 0; c < 4; c++) { cn[k][c] = warp_sum(cn[k][c]); d0[k][c] = warp_sum(d0[k][c]); }
    }
    if (lane == 0) {
        const long long at = bt * py.nodes;
        norms[at + py.noff[2] + idx2] = n2;
        if (py.L == 3) dots[at + py.noff[2] + idx2] = 0.f;
#pragma unroll
        for (int k = 0; k < 4; k++) {
            if (k < nk) {
                norms[at + py.noff[1] + kid[k]] = n1[k];
                dots[at + py.noff[1] + kid[k]] = d1[k];
#pragma unroll
                for (int c = 0; c < 4; c++) {
                    if (c < nc[k]) {
                        norms[at + cell[k][c]] = cn[k][c];
                        dots[at + cell[k][c]] = d0[k][c];
                    }
                }
            }
        }
    }
}

// does every existing child of a node exceed tau_s in cosine to it?  One thread per node of a
// level >= 1.
__global__ void __launch_bounds__(256)
k_gen_allpass(Geo g, Pyr py, Taus taus, const float* __restrict__ norms, const float* __restrict__ dots,
              int8_t* __restrict__ allpass) {
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i0 >= (long long)g.B * g.T * py.nodes) return;
    const long long bt = i0 / py.nodes;
    const int node = (int)(i0 % py.nodes);
    int l = 0;
    while (l + 1 < py.L && node >= py.noff[l + 1]) l++;
    if (l == 0) { allpass[i0] = 0; return; }
    const int idx = node - py.noff[l], i = idx / py.W[l], j = idx % py.W[l];
    const float tau = taus.s[bt / g.T];
    const float np = norms[i0];
    bool all = true;
    for (int a = 0; a < 2; a++)
        for (int b = 0; b < 2; b++)
            if (2 * i + a < py.H[l - 1] && 2 * j + b < py.W[l - 1]) {
                const long long c = bt * py.nodes + py.noff[l - 1] + (2 * i + a) * py.W[l - 1] + 2 * j + b;
                all = all && cos_from(dots[c], norms[c], np) > tau;
            }
    allpass[i0] = all ? 1 : 0;
}

// Section 3.2, the search read per cell: the coarsest ancestor all of whose children pass, met
// from the top, covers the cell.
__global__ void __launch_bounds__(256)
k_gen_cover(Geo g, Pyr py, const int8_t* __restrict__ allpass, int8_t* __restrict__ cover) {
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i0 >= (long long)g.B * g.N) return;
    const long long bt = i0 / g.HW;
    const int cell = (int)(i0 % g.HW), y = cell / g.W, x = cell % g.W;
    int lv = 0;
    for (int l = py.L - 1; l >= 1; l--)
        if (allpass[bt * py.nodes + py.noff[l] + (y >> l) * py.W[l] + (x >> l)]) { lv = l; break; }
    cover[i0] = (int8_t)lv;
}

// Section 3.3: one warp per kept node of a frame t >= 1 (met at its top-left cell): every kept
// node of frame t-1 that overlaps it is compared once, at the first cell of the overlap.
template <typename T>
__global__ void __launch_bounds__(256)
k_gen_temporal(const T* __restrict__ feats, const float* __restrict__ pooled, Geo g, Pyr py, Taus taus,
               const int8_t* __restrict__ cover, const float* __restrict__ norms, int32_t* __restrict__ link,
               int match_best) {
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= (long long)g.B * g.N) return;
    const long long bt = warp / g.HW;
    const int t = (int)(bt % g.T);
    const int cell = (int)(warp % g.HW), y0 = cell / g.W, x0 = cell % g.W;
    const int lv = cover[warp], m = (1 << lv) - 1;
    if (t == 0 || ((y0 & m) | (x0 & m)) != 0) return;
    const int y1 = min(y0 + (1 << lv), g.H), x1 = min(x0 + (1 << lv), g.W);
    const int vidx = (y0 >> lv) * py.W[lv] + (x0 >> lv);
    const float nv = norms[bt * py.nodes + py.noff[lv] + vidx];
    const float tau = taus.t[bt / g.T];
    const int8_t* cprev = cover + (warp - cell) - g.HW;
    int best_u = -1;
    float best_s = 0.f;
    for (int yy = y0; yy < y1; yy++)
        for (int xx = x0; xx < x1; xx++) {
            const int lu = cprev[yy * g.W + xx], mu = (1 << lu) - 1;
            const int uy = yy & ~mu, ux = xx & ~mu;
            if (yy != max(uy, y0) || xx != max(ux, x0)) continue;      // this candidate was met before
            const int uidx = (uy >> lu) * py.W[lu] + (ux >> lu);
            float dp = 0.f;
            for (int d = lane * VEC; d < g.D; d += 32 * VEC) {
                float a[VEC], b[VEC];
                node4(feats, pooled, g, py, bt, lv, vidx, d, a);
                node4(feats, pooled, g, py, bt - 1, lu, uidx, d, b);
#pragma unroll
                for (int v = 0; v < VEC; v++) dp = fmaf(a[v], b[v], dp);
            }
            dp = warp_sum(dp);
            const float s = cos_from(dp, nv, norms[(bt - 1) * py.nodes + py.noff[lu] + uidx]);
            if (!(s > tau)) continue;
            const int u_id = (t - 1) * g.HW + uy * g.W + ux;
            if (best_u < 0 || (match_best ? (s > best_s || (s == best_s && u_id < best_u)) : u_id < best_u)) {
                best_u = u_id;
                best_s = s;
            }
        }
    if (lane == 0) link[warp] = best_u;
}

// Section 3.3, common root: top-left cells first point at their link (or at themselves), then
// pointer jumping; the other cells of a node copy from its top-left cell at the end.
__global__ void __launch_bounds__(256)
k_gen_root_init(Geo g, const int8_t* __restrict__ cover, const int32_t* __restrict__ link, int32_t* __restrict__ root) {
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i0 >= (long long)g.B * g.N) return;
    const int c = (int)(i0 % g.N), cell = c % g.HW, y = cell / g.W, x = cell % g.W;
    const int m = (1 << cover[i0]) - 1;
    if (((y & m) | (x & m)) != 0) { root[i0] = -1; return; }
    const int lk = link[i0];
    root[i0] = lk < 0 ? c : lk;
}
__global__ void __launch_bounds__(256)
k_gen_root_jump(Geo g, int32_t* root) {
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i0 >= (long long)g.B * g.N) return;
    const long long vb = i0 / g.N * g.N;
    const int r = root[i0];
    if (r < 0) return;
    const int rr = root[vb + r];
    if (rr != r) root[i0] = rr;
}
__global__ void __launch_bounds__(256)
k_gen_root_fill(Geo g, const int8_t* __restrict__ cover, int32_t* root) {
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i0 >= (long long)g.B * g.N) return;
    const int c = (int)(i0 % g.N), t = c / g.HW, cell = c % g.HW, y = cell / g.W, x = cell % g.W;
    const int m = (1 << cover[i0]) - 1;
    if (((y & m) | (x & m)) == 0) return;
    root[i0] = root[i0 / g.N * g.N + t * g.HW + (y & ~m) * g.W + (x & ~m)];
}

// Section 3.3, merge.  Every output row gets the list of its kept nodes (counted, placed by a prefix
// sum over the rows, put into index order), then kGenParts warps per row add the weighted features
// in that order and divide once: the sums do not depend on scheduling.
__device__ __forceinline__ bool gen_kept_anchor(const Geo& g, long long i0, int lv) {
    const int cell = (int)(i0 % g.HW), y0 = cell / g.W, x0 = cell % g.W, m = (1 << lv) - 1;
    return ((y0 & m) | (x0 & m)) == 0;
}
__global__ void __launch_bounds__(256)
k_gen_count(Geo g, const int8_t* __restrict__ cover, const int32_t* __restrict__ cell_row, int32_t* __restrict__ cnt,
            long long capacity) {
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i0 >= (long long)g.B * g.N || !gen_kept_anchor(g, i0, cover[i0])) return;
    const long long row = cell_row[i0];
    if (row < capacity) atomicAdd(cnt + row, 1);
}
// one block: start[r] = number of list entries before row r, start[rows] = their total
__global__ void __launch_bounds__(1024)
k_gen_scan_rows(Geo g, const long long* __restrict__ vid_off, long long capacity, const int32_t* __restrict__ cnt,
                int32_t* __restrict__ start) {
    __shared__ int sm[33];
    const long long rows = min(vid_off[g.B], capacity);
    int carry = 0;
    for (long long r0 = 0; r0 < rows; r0 += blockDim.x) {
        const long long r = r0 + threadIdx.x;
        const int v = r < rows ? cnt[r] : 0;
        int total;
        const int ex = block_exclusive_scan(v, total, sm);
        if (r < rows) start[r] = carry + ex;
        carry += total;
        __syncthreads();
    }
    if (threadIdx.x == 0) start[rows] = carry;
}
// (the counts are used up as cursors: a row's entries land in any order and are put in order next)
__global__ void __launch_bounds__(256)
k_gen_fill(Geo g, const int8_t* __restrict__ cover, const int32_t* __restrict__ cell_row, int32_t* __restrict__ cnt,
           const int32_t* __restrict__ start, int32_t* __restrict__ list, long long capacity) {
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i0 >= (long long)g.B * g.N || !gen_kept_anchor(g, i0, cover[i0])) return;
    const long long row = cell_row[i0];
    if (row >= capacity) return;
    const int at = atomicSub(cnt + row, 1) - 1;
    list[start[row] + at] = (int32_t)i0;
}
// one warp per row: its entries in increasing order (rank by counting; rows are short)
__global__ void __launch_bounds__(256)
k_gen_sort(Geo g, const long long* __restrict__ vid_off, long long capacity, const int32_t* __restrict__ start,
           const int32_t* __restrict__ list, int32_t* __restrict__ sorted) {
    const long long row = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= min(vid_off[g.B], capacity)) return;
    const int base = start[row], n = start[row + 1] - base;
    for (int i = lane; i < n; i += 32) {
        const int mine = list[base + i];
        int rank = 0;
        for (int k = 0; k < n; k++) rank += list[base + k] < mine ? 1 : 0;
        sorted[base + rank] = mine;
    }
}
constexpr int kGenParts = 8;
template <typename T, typename OutT>
__global__ void __launch_bounds__(256)
k_gen_gather(const T* __restrict__ feats, const float* __restrict__ pooled, Geo g, Pyr py,
             const long long* __restrict__ vid_off, const int8_t* __restrict__ cover,
             const int32_t* __restrict__ start, const int32_t* __restrict__ sorted,
             const int32_t* __restrict__ row_weight, OutT* __restrict__ out, long long capacity, int weight_mode) {
    const long long unit = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const long long row = unit / kGenParts;
    const int part = (int)(unit % kGenParts);
    if (row >= min(vid_off[g.B], capacity)) return;
    const int base = start[row], n = start[row + 1] - base;
    const float inv = 1.f / (float)row_weight[row];
    const int nf4 = g.D / VEC;
    const int lo = (int)((long long)nf4 * part / kGenParts), hi = (int)((long long)nf4 * (part + 1) / kGenParts);
    for (int f0 = lo + lane; f0 < hi; f0 += 4 * 32) {
        float sum[4][VEC];
#pragma unroll
        for (int u = 0; u < 4; u++)
#pragma unroll
            for (int v = 0; v < VEC; v++) sum[u][v] = 0.f;
        // two members' loads are issued before anything is added; the additions keep the list's order
        for (int k0 = 0; k0 < n; k0 += 2) {
            float x[2][4][VEC], w[2];
#pragma unroll
            for (int k = 0; k < 2; k++) {
                if (k0 + k < n) {
                    const long long i0 = sorted[base + k0 + k];
                    const long long bt = i0 / g.HW;
                    const int cell = (int)(i0 % g.HW), y0 = cell / g.W, x0 = cell % g.W;
                    const int lv = cover[i0];
                    w[k] = weight_mode ? (float)(min(1 << lv, g.H - y0) * min(1 << lv, g.W - x0)) : 1.f;
                    const int vidx = (y0 >> lv) * py.W[lv] + (x0 >> lv);
#pragma unroll
                    for (int u = 0; u < 4; u++)
                        if (f0 + u * 32 < hi) node4(feats, pooled, g, py, bt, lv, vidx, (f0 + u * 32) * VEC, x[k][u]);
                }
            }
#pragma unroll
            for (int k = 0; k < 2; k++) {
                if (k0 + k < n) {
#pragma unroll
                    for (int u = 0; u < 4; u++)
                        if (f0 + u * 32 < hi) {
#pragma unroll
                            for (int v = 0; v < VEC; v++) sum[u][v] = fmaf(w[k], x[k][u][v], sum[u][v]);
                        }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < 4; u++)
            if (f0 + u * 32 < hi) {
#pragma unroll
                for (int v = 0; v < VEC; v++) sum[u][v] *= inv;
                store4(out + row * g.D + (long long)(f0 + u * 32) * VEC, sum[u]);
            }
    }
}

}  // namespace sttm
