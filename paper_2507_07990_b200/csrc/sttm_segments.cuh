// One long video cut into segments of consecutive frames, one segment per GPU (Section 3.3:
// the temporal links form chains over frames, so a chain may cross a cut).  Every segment is
// merged on its own with the frame before it (the halo) in front; the kernels here fold what a
// later segment merged into the halo's nodes into the rows of the segment that owns them.
//
// Vocabulary: a segment's LOCAL result is what sttm_merge_ex returns for halo + segment; its
// first n_h rows are rooted in the halo frame (one row per kept node of the halo, in order) and
// belong to an earlier segment; the other rows are OWNED.  A row is held as (mean m, weight W);
// a contribution to a row is (sum S, weight V): the row becomes (W m + S) / (W + V).
#pragma once
#include "sttm_device.cuh"
#include "sttm_kernels.cuh"

namespace sttm {

enum : int { kStatusBadIndex = 1 << 1 };

// W of every local row: the weights of its member nodes (1 per node, or its cells), found at
// the nodes' top-left cells.  weights starts at zero.
__global__ void __launch_bounds__(256)
k_row_weights(Geo g, const int8_t* __restrict__ cover, const int32_t* __restrict__ merge_map,
              const int64_t* __restrict__ out_offsets, float* __restrict__ weights, long long capacity,
              int weight_mode) {
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i0 >= (long long)g.B * g.N) return;
    const int b = (int)(i0 / g.N);
    const int cell = (int)(i0 % g.HW), y = cell / g.W, x = cell % g.W;
    const int lv = cover[i0], m = (1 << lv) - 1;
    if (((y & m) | (x & m)) != 0) return;
    const long long row = out_offsets[b] + merge_map[i0];
    if (row >= capacity) return;
    const float w = weight_mode ? (float)(min(1 << lv, g.H - y) * min(1 << lv, g.W - x)) : 1.f;
    atomicAdd(weights + row, w);
}

// Contributions that arrived from the next segment, keyed by the cell (within this segment's
// last frame) of the node they belong to: add each to the row that node went into.  Several
// nodes of one frame may share a row, hence atomics.  One warp per entry.
__global__ void __launch_bounds__(256)
k_segment_fold(const int32_t* __restrict__ map_last, const int32_t* __restrict__ anchors, const float* __restrict__ v,
               const float* __restrict__ s, const int32_t* __restrict__ n_dev, int n_max, int HW, int D,
               float* __restrict__ extra, float* __restrict__ extra_w, long long capacity,
               int32_t* __restrict__ device_status) {
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const int n = min(*n_dev, n_max);
    if (warp >= n) return;
    const float vi = v[warp];
    if (vi == 0.f) return;
    const int a = anchors[warp];
    if (a < 0 || a >= HW) {
        if (lane == 0 && device_status) atomicOr(device_status, kStatusBadIndex);
        return;
    }
    const long long row = map_last[a];
    if (row < 0 || row >= capacity) {
        if (lane == 0 && device_status) atomicOr(device_status, kStatusCapacity);
        return;
    }
    for (int d = lane; d < D; d += 32) atomicAdd(extra + row * D + d, s[warp * (long long)D + d]);
    if (lane == 0) atomicAdd(extra_w + row, vi);
}

// What this segment merged into the halo's nodes, without the nodes themselves (they are in the
// owner's rows already): S_b = W_b m_b + extra_b - w_u F(u), V_b = W_b + extra_w_b - w_u for the
// b-th halo-rooted row and the b-th kept node u of the halo frame.  One warp per row.
__global__ void __launch_bounds__(256)
k_segment_emit(const float* __restrict__ feats, const float* __restrict__ weights, const float* __restrict__ extra,
               const float* __restrict__ extra_w, const float* __restrict__ halo_feats,
               const float* __restrict__ halo_w, const int32_t* __restrict__ n_h_dev, int n_max, int D,
               float* __restrict__ v_out, float* __restrict__ s_out) {
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= min(*n_h_dev, n_max)) return;
    const float W = weights[warp], wu = halo_w[warp];
    const float V = W + extra_w[warp] - wu;
    if (lane == 0) v_out[warp] = V;
    const long long o = warp * (long long)D;
    for (int d = lane; d < D; d += 32)
        s_out[o + d] = V == 0.f ? 0.f : fmaf(W, feats[o + d], extra[o + d]) - wu * halo_feats[o + d];
}

// Owned rows with what later segments added, and their ids in the whole video.
template <typename OutT>
__global__ void __launch_bounds__(256)
k_segment_finish(const float* __restrict__ feats, const int32_t* __restrict__ pos, const float* __restrict__ weights,
                 const float* __restrict__ extra, const float* __restrict__ extra_w,
                 const int32_t* __restrict__ count_dev, const int32_t* __restrict__ n_h_dev, int D,
                 long long capacity, long long pos_shift, int reassigned, OutT* __restrict__ out_feats,
                 int32_t* __restrict__ out_pos, int32_t* __restrict__ owned_count) {
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int n_h = n_h_dev ? *n_h_dev : 0;
    const long long rows = min((long long)*count_dev, capacity) - n_h;
    if (i0 == 0) *owned_count = *count_dev - n_h;
    const int per = D / VEC;
    if (i0 >= rows * per) return;
    const long long r = i0 / per, src = r + n_h;
    const int d = (int)(i0 % per) * VEC;
    float m[VEC], e[VEC];
    load4(feats + src * D + d, m);
    const float ew = extra_w[src];
    if (ew != 0.f) {
        const float W = weights[src], inv = 1.f / (W + ew);
        load4(extra + src * D + d, e);
#pragma unroll
        for (int k = 0; k < VEC; k++) m[k] = fmaf(W, m[k], e[k]) * inv;
    }
    store4(out_feats + r * D + d, m);
    if (d == 0) out_pos[r] = (int32_t)((reassigned ? r : (long long)pos[src]) + pos_shift);
}

}  // namespace sttm
