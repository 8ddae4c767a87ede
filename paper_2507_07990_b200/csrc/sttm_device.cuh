// Device-side building blocks shared by the STTM kernels (sm_100a).
//
// Work decomposition.  With L quadtree levels a frame splits into "columns": the
// regions of the coarsest nodes (side 2^(L-1) cells).  Everything that touches
// features stays inside one column through time: the coarse-to-fine search of
// Section 3.2 only looks at a coarsest node's own subtree, kept nodes never cross a
// column border, and the temporal candidates of Section 3.3 overlap the node, hence
// lie in the same column of the previous frame.  Only the final ordering (Section 3.4)
// looks across columns, and that is integer work.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sttm {

constexpr int kMaxBatch = 64;
constexpr int VEC = 4;              // channels per lane per step
constexpr int kSliceCh = 32 * VEC;  // channels one warp covers per step

struct Geo {
    int B, T, H, W, D;
    int L;         // quadtree levels, 1..3
    int side;      // 1 << (L-1): cells per column side
    int Hc, Wc;    // columns per frame (= size of the coarsest map)
    int ncol;
    int HW, N;     // cells per frame, per video
    int H1, W1;    // size of the level-1 map
    int nsim;      // parent-child similarities per frame
};

struct Taus {
    float s[kMaxBatch];
    float t[kMaxBatch];
};

// Node numbering inside a column.  L=3: cells 0..15 (row-major in the 4x4 region),
// level-1 nodes 16..19, the coarsest node 20.  L=2: cells 0..3, coarsest node 4.
// L=1: the cell itself.
template <int LEVELS>
struct Col {
    static constexpr int SIDE = 1 << (LEVELS - 1);
    static constexpr int NC = SIDE * SIDE;
    static constexpr int NQ = LEVELS == 3 ? 4 : 0;
    static constexpr int NN = NC + NQ + (LEVELS > 1 ? 1 : 0);
    __host__ __device__ static constexpr int dy(int c) { return c / SIDE; }
    __host__ __device__ static constexpr int dx(int c) { return c % SIDE; }
    // level-1 node (quad) of a cell, L=3 only
    __host__ __device__ static constexpr int quad(int c) { return (dy(c) >> 1) * 2 + (dx(c) >> 1); }
    // k-th cell of quad q, L=3 only
    __host__ __device__ static constexpr int quad_cell(int q, int k) {
        return ((q >> 1) * 2 + (k >> 1)) * SIDE + (q & 1) * 2 + (k & 1);
    }
    // index (in the column's node numbering) of the level-`lv` node that holds cell c
    __host__ __device__ static constexpr int node_of(int c, int lv) {
        return lv == 0 ? c : (LEVELS == 3 && lv == 1 ? NC + quad(c) : NC + NQ);
    }
};

// First statement of a kernel that may be launched with programmatic stream serialization
// (its blocks may become resident while the kernel before it in the stream still runs): waits
// until that kernel has completed and its writes are visible.  Returns at once otherwise.
__device__ __forceinline__ void wait_for_prior_kernel() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the kernel launched after this one (with the same attribute) become resident now instead of
// when this kernel ends.  That kernel still sees this one's writes only after its own
// wait_for_prior_kernel(), or through flags written with store_release() and read with load_acquire().
__device__ __forceinline__ void let_next_kernel_start() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void store_release(int32_t* p, int32_t v) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int32_t load_acquire(const int32_t* p) {
    int32_t v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// cos from a dot product and two squared norms; 0 when a vector is all zero
__device__ __forceinline__ float cos_from(float dot, float na, float nb) {
    if (na == 0.f || nb == 0.f) return 0.f;
    return dot / (sqrtf(na) * sqrtf(nb));
}

// 4 consecutive channels -> fp32
__device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&x)[VEC]) {
    const uint2 r = __ldg(reinterpret_cast<const uint2*>(p));
    x[0] = __uint_as_float(r.x << 16);
    x[1] = __uint_as_float(r.x & 0xffff0000u);
    x[2] = __uint_as_float(r.y << 16);
    x[3] = __uint_as_float(r.y & 0xffff0000u);
}
__device__ __forceinline__ void load4(const float* p, float (&x)[VEC]) {
    const float4 r = __ldg(reinterpret_cast<const float4*>(p));
    x[0] = r.x; x[1] = r.y; x[2] = r.z; x[3] = r.w;
}

__device__ __forceinline__ void store4(__nv_bfloat16* p, const float (&x)[VEC]) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(x[0], x[1]);
    const __nv_bfloat162 hi = __floats2bfloat162_rn(x[2], x[3]);
    uint2 r;
    r.x = *reinterpret_cast<const uint32_t*>(&lo);
    r.y = *reinterpret_cast<const uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p) = r;
}
__device__ __forceinline__ void store4(float* p, const float (&x)[VEC]) {
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
}

// Validity of a column's cells on a clipped grid, and the reciprocal child counts of
// its parents (2x2 average pooling divides by the children that exist).
template <int LEVELS>
struct ColShape {
    uint32_t valid;                 // bit c: cell c lies inside the grid
    float inv1[Col<LEVELS>::NQ > 0 ? Col<LEVELS>::NQ : 1];
    float inv2;
    __device__ __forceinline__ void init(int rows, int cols) {
        using C = Col<LEVELS>;
        valid = 0;
#pragma unroll
        for (int c = 0; c < C::NC; c++)
            if (C::dy(c) < rows && C::dx(c) < cols) valid |= 1u << c;
        if constexpr (LEVELS == 3) {
            int nq = 0;
#pragma unroll
            for (int q = 0; q < 4; q++) {
                int n = 0;
#pragma unroll
                for (int k = 0; k < 4; k++) n += (valid >> C::quad_cell(q, k)) & 1;
                inv1[q] = n ? 1.f / (float)n : 0.f;
                nq += n ? 1 : 0;
            }
            inv2 = 1.f / (float)nq;
        } else if constexpr (LEVELS == 2) {
            inv1[0] = 0.f;
            inv2 = 1.f / (float)__popc(valid);
        } else {
            inv1[0] = 0.f;
            inv2 = 1.f;
        }
    }
    __device__ __forceinline__ bool cell(int c) const { return (valid >> c) & 1u; }
    __device__ __forceinline__ bool quad(int q) const { return inv1[q] != 0.f; }
};

// Pooled features of a column for VEC channels: p1 = level-1 nodes (L=3), p2 = the
// coarsest node (L>=2).  Cells outside the grid hold zeros.
template <int LEVELS>
__device__ __forceinline__ void pool_column(const float (&x)[Col<LEVELS>::NC][VEC], const ColShape<LEVELS>& sh,
                                            float (&p1)[4][VEC], float (&p2)[VEC]) {
    using C = Col<LEVELS>;
    if constexpr (LEVELS == 3) {
#pragma unroll
        for (int q = 0; q < 4; q++)
#pragma unroll
            for (int v = 0; v < VEC; v++)
                p1[q][v] = ((x[C::quad_cell(q, 0)][v] + x[C::quad_cell(q, 1)][v]) +
                            (x[C::quad_cell(q, 2)][v] + x[C::quad_cell(q, 3)][v])) * sh.inv1[q];
#pragma unroll
        for (int v = 0; v < VEC; v++) p2[v] = ((p1[0][v] + p1[1][v]) + (p1[2][v] + p1[3][v])) * sh.inv2;
    } else if constexpr (LEVELS == 2) {
#pragma unroll
        for (int v = 0; v < VEC; v++) p2[v] = ((x[0][v] + x[1][v]) + (x[2][v] + x[3][v])) * sh.inv2;
    }
}

// feature of the level-`lv` node holding cell c (lv is warp-uniform, c is a constant)
template <int LEVELS>
__device__ __forceinline__ float node_feat(int lv, int c, int v, const float (&x)[Col<LEVELS>::NC][VEC],
                                           const float (&p1)[4][VEC], const float (&p2)[VEC]) {
    if constexpr (LEVELS == 3) return lv == 0 ? x[c][v] : (lv == 1 ? p1[Col<3>::quad(c)][v] : p2[v]);
    else if constexpr (LEVELS == 2) return lv == 0 ? x[c][v] : p2[v];
    else return x[c][v];
}

// is cell c the top-left cell of its level-lv node
template <int LEVELS>
__device__ __forceinline__ bool is_anchor(int c, int lv) {
    const int m = (1 << lv) - 1;
    return ((Col<LEVELS>::dy(c) & m) | (Col<LEVELS>::dx(c) & m)) == 0;
}

}  // namespace sttm
