// General path for quadtrees of more than three levels (grids of more than 16 cells a side
// with a 4x4 coarsest map, or the 2x2 coarsest map of the paper's ablation on a 13x13 / 14x14 /
// 16x16 grid).  Plain kernels, one step of Section 3 each, pooled features kept in fp32 in the
// workspace; nothing here is tuned: the fused kernel covers the shapes that matter for speed.
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
// that exist).  One warp per node of level l.
template <typename T>
__global__ void __launch_bounds__(256)
k_gen_pool(const T* __restrict__ feats, float* __restrict__ pooled, Geo g, Pyr py, int l) {
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
    for (int d = lane * VEC; d < g.D; d += 32 * VEC) {
        float s[VEC] = {0.f, 0.f, 0.f, 0.f};
        for (int c = 0; c < n; c++) {
            float x[VEC];
            node4(feats, pooled, g, py, bt, l - 1, child[c], d, x);
#pragma unroll
            for (int v = 0; v < VEC; v++) s[v] += x[v];
        }
#pragma unroll
        for (int v = 0; v < VEC; v++) s[v] *= inv;
        store4(dst + d, s);
    }
}

// squared norm of every node and its dot product with its parent.  One warp per node.
template <typename T>
__global__ void __launch_bounds__(256)
k_gen_norm_dot(const T* __restrict__ feats, const float* __restrict__ pooled, Geo g, Pyr py,
               float* __restrict__ norms, float* __restrict__ dots) {
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= (long long)g.B * g.T * py.nodes) return;
    const long long bt = warp / py.nodes;
    const int node = (int)(warp % py.nodes);
    int l = 0;
    while (l + 1 < py.L && node >= py.noff[l + 1]) l++;
    const int idx = node - py.noff[l], i = idx / py.W[l], j = idx % py.W[l];
    const bool has_parent = l + 1 < py.L;
    const int pidx = has_parent ? (i >> 1) * py.W[l + 1] + (j >> 1) : 0;
    float nn = 0.f, dp = 0.f;
    for (int d = lane * VEC; d < g.D; d += 32 * VEC) {
        float x[VEC], q[VEC];
        node4(feats, pooled, g, py, bt, l, idx, d, x);
#pragma unroll
        for (int v = 0; v < VEC; v++) nn = fmaf(x[v], x[v], nn);
        if (has_parent) {
            node4(feats, pooled, g, py, bt, l + 1, pidx, d, q);
#pragma unroll
            for (int v = 0; v < VEC; v++) dp = fmaf(x[v], q[v], dp);
        }
    }
    nn = warp_sum(nn);
    dp = warp_sum(dp);
    if (lane == 0) {
        norms[bt * py.nodes + node] = nn;
        dots[bt * py.nodes + node] = dp;
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

// Section 3.3, merge: every kept node adds its weighted feature to its row (fp32 atomics: the
// order of the additions, hence the last bits, may differ from run to run), then one division.
template <typename T>
__global__ void __launch_bounds__(256)
k_gen_accumulate(const T* __restrict__ feats, const float* __restrict__ pooled, Geo g, Pyr py,
                 const int8_t* __restrict__ cover, const int32_t* __restrict__ cell_row, float* __restrict__ acc,
                 long long capacity, int weight_mode) {
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= (long long)g.B * g.N) return;
    const long long bt = warp / g.HW;
    const int cell = (int)(warp % g.HW), y0 = cell / g.W, x0 = cell % g.W;
    const int lv = cover[warp], m = (1 << lv) - 1;
    if (((y0 & m) | (x0 & m)) != 0) return;
    const long long row = cell_row[warp];
    if (row >= capacity) return;
    const float w = weight_mode ? (float)(min(1 << lv, g.H - y0) * min(1 << lv, g.W - x0)) : 1.f;
    const int vidx = (y0 >> lv) * py.W[lv] + (x0 >> lv);
    for (int d = lane * VEC; d < g.D; d += 32 * VEC) {
        float x[VEC];
        node4(feats, pooled, g, py, bt, lv, vidx, d, x);
#pragma unroll
        for (int v = 0; v < VEC; v++) atomicAdd(acc + row * g.D + d + v, w * x[v]);
    }
}
template <typename OutT>
__global__ void __launch_bounds__(256)
k_gen_finish(Geo g, const long long* __restrict__ vid_off, const float* __restrict__ acc,
             const int32_t* __restrict__ row_weight, OutT* __restrict__ out, long long capacity) {
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long rows = min(vid_off[g.B], capacity);
    const int per = g.D / VEC;
    if (i0 >= rows * per) return;
    const long long row = i0 / per;
    const int d = (int)(i0 % per) * VEC;
    const float inv = 1.f / (float)row_weight[row];
    float x[VEC];
    load4(acc + row * g.D + d, x);
#pragma unroll
    for (int v = 0; v < VEC; v++) x[v] *= inv;
    store4(out + row * g.D + d, x);
}

}  // namespace sttm
