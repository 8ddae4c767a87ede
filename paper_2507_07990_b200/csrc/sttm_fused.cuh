// Fused single-read STTM kernel (sm_100a): spatial search, temporal linking and averaging
// in one pass over the features.
//
// Decomposition.  A frame is cut into 4x4-cell tiles (the region of a coarsest quadtree
// node when the tree has three levels; four / sixteen independent regions when it has two
// / one).  Everything that touches features stays inside one tile through time, so a work
// item is (video, tile, run of consecutive frames).  A thread-block cluster of C CTAs owns
// an item; each CTA owns D/C channels of the tile and streams them frame by frame through
// a shared-memory ring filled by bulk asynchronous copies (one per cell).
//
// Per frame j of an item:
//   1. tensor-core warps form the tile's Gram matrix G_j = X_j X_j^T and the cross matrix
//      C_j = X_j X_{j-1}^T over the CTA's channels (X = the 16 cells of the tile); every
//      cosine of Sections 3.2 and 3.3 is a short linear combination of entries of G and C
//      because parents are averages of cells.  The products of bf16 inputs are exact and
//      the sums are kept in fp32.
//   2. worker threads contract the partial matrices to the 128 numbers the decisions need
//      (per cell: its squared norm, its products with its parent and with the coarsest node,
//      and its products with the nodes of the previous frame that contain it or that it
//      contains) and add them across warps (shared memory) and across the cluster
//      (distributed shared memory), in a fixed order.
//   3. one decision warp per CTA turns the totals into the cover map, the links and the
//      bookkeeping of the running chains (every CTA of the cluster repeats this on the
//      same numbers and gets the same answer), and leaves a small command record.
//   4. two frames later the worker threads execute the record on the frame that is still
//      in the ring: each thread owns two channels, keeps the running sums of up to 16
//      chains in registers, adds the nodes of the frame and writes out chains that ended.
// Finished chains go to a staging row indexed by the root's cell id (their final row is
// only known after the global ordering); chains cut by the end of an item go to an fp32
// piece buffer and are put together by the gather kernel.
#pragma once

#include "sttm_device.cuh"
#include "sttm_kernels.cuh"

namespace sttm {

constexpr int kMaxTiles = 64;
constexpr int kMaxCluster = 8;
constexpr int kRecRing = 4;
constexpr int kGramVals = 512;          // G (16x16) then C (16x16)
constexpr int kSumVals = 128;           // 8 numbers per cell, see combine_sums()
constexpr int kPieceSlots = 32;         // per item: 16 keyed by a cell of the frame before the item, 16 by chain slot
constexpr int kFusedMaxWorkerWarps = 16;
constexpr int kFusedMaxThreads = (kFusedMaxWorkerWarps + 1) * 32;
constexpr int kSpinLimit = 1 << 20;   // after the first wait that runs out, later waits are skipped

enum : int { kStatusWaitTimeout = 1 << 6 };

struct FlushCmd { int slot, kind, dst; float weight; };     // kind 0: finished row, 1: piece
struct NodeCmd { int cell, lv, slot; float w; };
struct FrameRec {
    int n_pre, n_nodes, n_post, pad;
    FlushCmd pre[16];
    NodeCmd node[16];
    FlushCmd post[16];
};

struct FusedParams {
    const __nv_bfloat16* feats;
    int B, T, H, W, D, L;
    int HW, N;
    int Wt, ntiles;
    int C, S, Wn, NM;        // cluster size, channels per CTA, worker warps, tensor-core warps
    int row_bytes, slot_bytes, R;
    int F, nseg, nitems;
    int weight_mode, out_f32;
    int8_t* cover;
    int32_t* link;
    int32_t* chain_key;      // [B*N] per cell: root cell id of its chain as far as the item knows it
    void* staging;           // [B*N][D] rows of the output dtype
    float* pieces;           // [nitems][kPieceSlots][D]
    int2* piece_meta;        // [nitems][kPieceSlots] {key cell id or -1, weight}
    int* queue;
    int* status;
    unsigned char tile_order[kMaxTiles];
};

// ---------------------------------------------------------------------------------
// PTX helpers
// ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
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
// global -> this CTA's shared memory, completion counted in bytes on an mbarrier
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
    uint32_t out;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(addr), "r"(rank));
    return out;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void st_cluster_u32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void named_sync(int id, int count) {
    asm volatile("barrier.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// D (16x8, fp32) += A (16x16 bf16, row) * B (16x8 bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ int ld_acquire_cta(const int* p) {
    int v;
    asm volatile("ld.acquire.cta.shared.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_cta(int* p, int v) {
    asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}

// tile-local cell c = dy*4 + dx; top-left cell of the level-lv node that holds c
__device__ __forceinline__ int tile_anchor(int c, int lv) {
    const int m = ~((1 << lv) - 1);
    return (((c >> 2) & m) << 2) | ((c & 3) & m);
}
__device__ __forceinline__ uint32_t quad_mask(int c) { return 0x33u << (8 * (c >> 3) + 2 * ((c >> 1) & 1)); }
__device__ __forceinline__ uint32_t region_mask(int c, int lv) {
    return lv == 0 ? (1u << c) : (lv == 1 ? quad_mask(c) : 0xffffu);
}

// running sums of the chains: 16 slots x 2 channels, in registers; the slot index is
// uniform over the block, so the switch does not diverge
struct ChainAcc {
    float2 a[16];
    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int i = 0; i < 16; i++) a[i] = make_float2(0.f, 0.f);
    }
#define STTM_ACC_CASE(i) case i: a[i].x += f.x; a[i].y += f.y; break;
    __device__ __forceinline__ void add(int slot, float2 f) {
        switch (slot) {
            STTM_ACC_CASE(0) STTM_ACC_CASE(1) STTM_ACC_CASE(2) STTM_ACC_CASE(3) STTM_ACC_CASE(4) STTM_ACC_CASE(5)
            STTM_ACC_CASE(6) STTM_ACC_CASE(7) STTM_ACC_CASE(8) STTM_ACC_CASE(9) STTM_ACC_CASE(10) STTM_ACC_CASE(11)
            STTM_ACC_CASE(12) STTM_ACC_CASE(13) STTM_ACC_CASE(14) default: a[15].x += f.x; a[15].y += f.y; break;
        }
    }
#undef STTM_ACC_CASE
#define STTM_TAKE_CASE(i) case i: v = a[i]; a[i] = make_float2(0.f, 0.f); break;
    __device__ __forceinline__ float2 take(int slot) {
        float2 v;
        switch (slot) {
            STTM_TAKE_CASE(0) STTM_TAKE_CASE(1) STTM_TAKE_CASE(2) STTM_TAKE_CASE(3) STTM_TAKE_CASE(4)
            STTM_TAKE_CASE(5) STTM_TAKE_CASE(6) STTM_TAKE_CASE(7) STTM_TAKE_CASE(8) STTM_TAKE_CASE(9)
            STTM_TAKE_CASE(10) STTM_TAKE_CASE(11) STTM_TAKE_CASE(12) STTM_TAKE_CASE(13) STTM_TAKE_CASE(14)
            default: v = a[15]; a[15] = make_float2(0.f, 0.f); break;
        }
        return v;
    }
#undef STTM_TAKE_CASE
};

__device__ __forceinline__ float2 unpack_bf16x2(uint32_t w) {
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float2 v) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(v.x, v.y);
    return *reinterpret_cast<const uint32_t*>(&h);
}

// sum over lanes that share (lane & 16): every lane of a half gets its half's total
__device__ __forceinline__ float half_warp_sum(float v) {
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

struct ItemGeo {
    int item, b, t0, t1, tstart, n, halo, last_seg;
    int y0, x0;
    uint32_t vmask;     // bit c: cell c of the tile lies inside the grid
    int nvalid;
};

// What the decision warp carries from frame to frame (lane c < 16: cell c of the tile).
struct DecState {
    int prev_lv, prev_slot;      // level / chain slot of the kept node covering the cell in the previous frame
    float prev_nk;               // its squared norm
    uint32_t active;             // uniform: slots in use
};

// Chain slots of the decision warp (shared memory, private to it).
struct SlotTable {
    int key[16], weight[16], virt[16], cell[16];
};

// The 8 numbers of cell c that the decisions need, as linear functions of the tile's Gram
// matrix G = X_t X_t^T and cross matrix Cm = X_t X_{t-1}^T (row: cell of frame t).  With
// q(c) the cell's 2x2 block, w1 / w2 the averaging weights of level 1 / level 2:
//   k=0  |x_c|^2                       k=1  x_c . parent(c)            k=2  x_c . top
//   k=3  x_c(t) . x_c(t-1)             k=4  x_c(t) . parent(c)(t-1)    k=5  x_c(t) . top(t-1)
//   k=6  parent(c)(t) . x_c(t-1)       k=7  top(t) . x_c(t-1)
// `m` points at NM partial matrices of kGramVals floats each; they are added in order.
__device__ __forceinline__ float combine_sums(const float* m, int NM, int c, int k, const float* W1s,
                                              const float* W2s) {
    const int qb = tile_anchor(c, 1);
    float acc = 0.f;
    for (int w = 0; w < NM; w++) {
        const float* G = m + w * kGramVals;
        const float* Cm = G + 256;
        float v = 0.f;
        switch (k) {
            case 0: v = G[c * 16 + c]; break;
            case 1: v = ((G[c * 16 + qb] + G[c * 16 + qb + 1]) + (G[c * 16 + qb + 4] + G[c * 16 + qb + 5])) * W1s[c]; break;
            case 2:
#pragma unroll
                for (int i = 0; i < 16; i++) v = fmaf(W2s[i], G[c * 16 + i], v);
                break;
            case 3: v = Cm[c * 16 + c]; break;
            case 4: v = ((Cm[c * 16 + qb] + Cm[c * 16 + qb + 1]) + (Cm[c * 16 + qb + 4] + Cm[c * 16 + qb + 5])) * W1s[c]; break;
            case 5:
#pragma unroll
                for (int i = 0; i < 16; i++) v = fmaf(W2s[i], Cm[c * 16 + i], v);
                break;
            case 6: v = ((Cm[qb * 16 + c] + Cm[(qb + 1) * 16 + c]) + (Cm[(qb + 4) * 16 + c] + Cm[(qb + 5) * 16 + c])) * W1s[c]; break;
            default:
#pragma unroll
                for (int i = 0; i < 16; i++) v = fmaf(W2s[i], Cm[i * 16 + c], v);
                break;
        }
        acc += v;
    }
    return acc;
}

// sum over the four cells of the lane's 2x2 block (lanes of the same half warp)
__device__ __forceinline__ float quad_sum(float v, int lane) {
    const int hb = lane & 16, qb = tile_anchor(lane & 15, 1);
    return (__shfl_sync(0xffffffffu, v, hb + qb) + __shfl_sync(0xffffffffu, v, hb + qb + 1)) +
           (__shfl_sync(0xffffffffu, v, hb + qb + 4) + __shfl_sync(0xffffffffu, v, hb + qb + 5));
}

// ---------------------------------------------------------------------------------
// Decisions of one frame (Sections 3.2 and 3.3) from the cluster totals of the 8 numbers
// per cell (v[0..7], lane c = cell c; lanes 16..31 mirror lanes 0..15).
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void decide_frame(const FusedParams& p, const ItemGeo& it, int j, float tau_s, float tau_t,
                                             const float (&v)[8], const float* W1s, const float* W2s, DecState& st,
                                             SlotTable* tab, FrameRec* rec, uint32_t rank, int lane) {
    const unsigned full = 0xffffffffu;
    const int c = lane & 15;
    const bool low = lane < 16;
    const int L = p.L;
    const int t = it.tstart + j;
    const bool has_prev = j > 0;
    const bool is_halo = it.halo && j == 0;
    const bool is_last = j == it.n - 1;
    const bool valid = (it.vmask >> c) & 1u;
    const uint32_t qm = quad_mask(c);
    const float w1 = W1s[c], w2 = W2s[c];

    // Section 3.2: cosine of every node with its parent, then the coarse-to-fine search
    const float n0 = v[0], d0 = v[1], rr = v[2];
    const float n1 = w1 * quad_sum(d0, lane);          // |parent|^2
    const float d1 = w1 * quad_sum(rr, lane);          // parent . top
    const float n2 = half_warp_sum(w2 * rr);           // |top|^2
    const float s0 = cos_from(d0, n0, n1);
    const float s1 = cos_from(d1, n1, n2);
    int lv = 0;
    if (L >= 2) {
        const bool p0 = !valid || s0 > tau_s;
        const uint32_t pm0 = __ballot_sync(full, p0) & 0xffffu;
        const bool quad_pass = (pm0 & qm) == qm;
        if (L == 3) {
            const bool quad_exists = (it.vmask & qm) != 0;
            const bool p1 = !quad_exists || s1 > tau_s;
            const uint32_t pm1 = __ballot_sync(full, p1) & 0xffffu;
            lv = pm1 == 0xffffu ? 2 : (quad_pass ? 1 : 0);
        } else {
            lv = quad_pass ? 1 : 0;
        }
    }
    const float nk = lv == 0 ? n0 : (lv == 1 ? n1 : n2);

    // Section 3.3: the node covering the cell against the overlapping kept node of the
    // previous frame; a pair is evaluated at the top-left cell of its finer node
    int link_local = -1;
    if (has_prev) {
        const int lu = st.prev_lv;
        const float t11 = w1 * quad_sum(v[4], lane), t12 = w1 * quad_sum(v[5], lane);
        const float t21 = w1 * quad_sum(v[7], lane), t22 = half_warp_sum(w2 * v[5]);
        float dot;
        if (lv == 0) dot = lu == 0 ? v[3] : (lu == 1 ? v[4] : v[5]);
        else if (lv == 1) dot = lu == 0 ? v[6] : (lu == 1 ? t11 : t12);
        else dot = lu == 0 ? v[7] : (lu == 1 ? t21 : t22);
        const bool rep = valid && tile_anchor(c, min(lv, lu)) == c;
        const float s = cos_from(dot, nk, st.prev_nk);
        const bool pass = rep && s > tau_t;
        const uint32_t passm = __ballot_sync(full, pass) & 0xffffu;
        const uint32_t cand = passm & region_mask(c, lv);
        const int cstar = cand ? __ffs(cand) - 1 : 0;         // first in row-major order: the top-left one
        const int lu_star = __shfl_sync(full, lu, cstar);
        link_local = cand ? tile_anchor(cstar, lu_star) : -1;
    }

    // chains: nodes with a link join the chain of their target; chains without a member in
    // this frame have ended; the remaining nodes start new chains in free slots
    const bool anchor = valid && tile_anchor(c, lv) == c;
    const bool linked = anchor && link_local >= 0;
    const bool fresh = anchor && link_local < 0;
    const int slot_linked = __shfl_sync(full, st.prev_slot, link_local < 0 ? 0 : link_local);
    const uint32_t memb = __reduce_or_sync(full, linked ? 1u << slot_linked : 0u);
    const uint32_t dead = st.active & ~memb;
    const uint32_t freem = ~memb & 0xffffu;
    const uint32_t freshm = __ballot_sync(full, fresh && low);
    const int slot_fresh = __fns(freem, 0, __popc(freshm & ((1u << c) - 1)) + 1);
    const int node_slot = linked ? slot_linked : slot_fresh;
    const int cur_slot = __shfl_sync(full, node_slot, (lane & 16) + tile_anchor(c, lv));
    const int wint = p.weight_mode ? __popc(it.vmask & region_mask(c, lv)) : 1;
    const long long gc = (long long)it.b * p.N + (long long)t * p.HW + (it.y0 + (c >> 2)) * p.W + it.x0 + (c & 3);

    // chains that ended: lane s looks at slot s (before the slot is given away again)
    const bool my_dead = low && ((dead >> lane) & 1u);
    if (my_dead) {
        const int at = __popc(dead & ((1u << lane) - 1));
        if (tab->virt[lane]) {
            const int pc = it.item * kPieceSlots + tab->cell[lane];
            rec->pre[at] = FlushCmd{lane, 1, pc, 0.f};
            if (rank == 0) p.piece_meta[pc] = make_int2(tab->key[lane], tab->weight[lane]);
        } else {
            rec->pre[at] = FlushCmd{lane, 0, tab->key[lane], (float)tab->weight[lane]};
        }
    }
    __syncwarp();
    if (low && fresh) {
        tab->key[slot_fresh] = (int)gc;
        tab->weight[slot_fresh] = is_halo ? 0 : wint;
        tab->virt[slot_fresh] = is_halo ? 1 : 0;
        tab->cell[slot_fresh] = c;
    }
    if (low && linked) atomicAdd(&tab->weight[slot_linked], wint);
    const uint32_t anchorm = __ballot_sync(full, anchor && low);
    if (low && anchor && !is_halo) {
        const float wn = lv == 1 ? w1 * (float)wint : (float)wint;
        rec->node[__popc(anchorm & ((1u << c) - 1))] = NodeCmd{c, lv, node_slot, wn};
    }
    const uint32_t active = memb | __reduce_or_sync(full, fresh ? 1u << slot_fresh : 0u);
    __syncwarp();

    if (rank == 0 && !is_halo && low && valid) {
        p.cover[gc] = (int8_t)lv;
        p.link[gc] = link_local < 0 ? -1
                                    : (t - 1) * p.HW + (it.y0 + (link_local >> 2)) * p.W + it.x0 + (link_local & 3);
        p.chain_key[gc] = tab->key[cur_slot] - it.b * p.N;
    }

    int npost = 0;
    if (is_last) {
        npost = __popc(active);
        if (low && ((active >> lane) & 1u)) {
            const int at = __popc(active & ((1u << lane) - 1));
            if (!tab->virt[lane] && it.last_seg) {
                rec->post[at] = FlushCmd{lane, 0, tab->key[lane], (float)tab->weight[lane]};
            } else {
                const int pc = it.item * kPieceSlots + 16 + lane;
                rec->post[at] = FlushCmd{lane, 1, pc, 0.f};
                if (rank == 0) p.piece_meta[pc] = make_int2(tab->key[lane], tab->weight[lane]);
            }
        }
    }
    if (lane == 0) {
        rec->n_pre = __popc(dead);
        rec->n_nodes = is_halo ? 0 : __popc(anchorm);
        rec->n_post = npost;
    }
    st.active = is_last ? 0u : active;
    st.prev_lv = lv;
    st.prev_slot = cur_slot;
    st.prev_nk = nk;
    __syncwarp();
}

// ---------------------------------------------------------------------------------
// The kernel.  blockDim.x = (Wn + 1) * 32: Wn worker warps, then the decision warp.
// ---------------------------------------------------------------------------------
template <int MAX_THREADS>
__global__ void __launch_bounds__(MAX_THREADS, 1)
k_fused(const __grid_constant__ FusedParams p, const __grid_constant__ Taus taus) {
    extern __shared__ __align__(128) unsigned char smem[];
    // carve-up
    unsigned char* ring = smem;
    size_t off = (size_t)p.R * p.slot_bytes;
    float* red = reinterpret_cast<float*>(smem + off);      off += (size_t)p.NM * kGramVals * 4;
    float* xchg = reinterpret_cast<float*>(smem + off);     off += (size_t)2 * p.C * kSumVals * 4;
    float* W1s = reinterpret_cast<float*>(smem + off);      off += 16 * 4;
    float* W2s = reinterpret_cast<float*>(smem + off);      off += 16 * 4;
    SlotTable* tab = reinterpret_cast<SlotTable*>(smem + off); off += sizeof(SlotTable);
    FrameRec* recs = reinterpret_cast<FrameRec*>(smem + off); off += kRecRing * sizeof(FrameRec);
    unsigned long long* full_bar = reinterpret_cast<unsigned long long*>(smem + off); off += 16 * 8;
    int* ctl = reinterpret_cast<int*>(smem + off);          // [0] current item, [1] records published

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nworkers = p.Wn * 32;
    const bool is_dec = warp == p.Wn;
    const uint32_t rank = cluster_rank();
    const uint32_t ring_base = smem_u32(ring);

    if (tid == 0) {
        for (int s = 0; s < p.R; s++) mbar_init(smem_u32(full_bar + s), 1);
        ctl[0] = 0;
        ctl[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    ChainAcc acc;
    acc.clear();
    __syncthreads();

    int qbase = 0;          // frames consumed so far (same in every thread of the cluster)
    bool timed_out = false;

    while (true) {
        // next item: rank 0 draws it and tells the cluster
        if (rank == 0 && tid == 0) {
            const int item = atomicAdd(p.queue, 1);
            for (int r = 0; r < p.C; r++) st_cluster_u32(map_to_rank(smem_u32(ctl), r), (uint32_t)item);
        }
        cluster_arrive();
        cluster_wait();
        ItemGeo it;
        it.item = *reinterpret_cast<volatile int*>(ctl);
        if (it.item >= p.nitems) break;
        {
            const int seg = it.item % p.nseg;
            const int bt = it.item / p.nseg;
            const int tile = p.tile_order[bt % p.ntiles];
            it.b = bt / p.ntiles;
            it.t0 = seg * p.F;
            it.t1 = min(p.T, it.t0 + p.F);
            it.halo = it.t0 > 0;
            it.tstart = it.t0 - it.halo;
            it.n = it.t1 - it.tstart;
            it.last_seg = it.t1 == p.T;
            it.y0 = (tile / p.Wt) * 4;
            it.x0 = (tile % p.Wt) * 4;
            const int rows = min(4, p.H - it.y0), cols = min(4, p.W - it.x0);
            it.vmask = 0;
            for (int c = 0; c < 16; c++)
                if ((c >> 2) < rows && (c & 3) < cols) it.vmask |= 1u << c;
            it.nvalid = __popc(it.vmask);
        }
        // per-item set-up: zero the rows of cells outside the grid, pooling weights, piece table
        if (!is_dec) {
            for (int s = 0; s < p.R; s++)
                for (int c = 0; c < 16; c++)
                    if (!((it.vmask >> c) & 1u))
                        for (int k = tid * 4; k < p.row_bytes; k += nworkers * 4)
                            *reinterpret_cast<uint32_t*>(ring + (size_t)s * p.slot_bytes + c * p.row_bytes + k) = 0u;
        } else {
            if (lane < 16) {
                const int c = lane;
                const uint32_t qm = quad_mask(c);
                const int nq = __popc(it.vmask & qm);
                int quads = 0;
                for (int q = 0; q < 4; q++) quads += (it.vmask & (0x33u << (8 * (q >> 1) + 2 * (q & 1)))) ? 1 : 0;
                const bool valid = (it.vmask >> c) & 1u;
                const float inv1 = nq ? 1.f / (float)nq : 0.f;
                W1s[c] = p.L >= 2 ? inv1 : 0.f;      // per quad: also on lanes of cells outside the grid
                W2s[c] = p.L == 3 && valid ? inv1 * (1.f / (float)quads) : 0.f;
            }
            if (rank == 0) p.piece_meta[(long long)it.item * kPieceSlots + lane] = make_int2(-1, 0);
        }
        __syncthreads();

        auto issue = [&](int j) {      // called by the whole warp 0
            const int q = qbase + j, s = q % p.R;
            const uint32_t bar = smem_u32(full_bar + s);
            if (lane == 0) mbar_expect_tx(bar, (uint32_t)(it.nvalid * p.S * 2));
            __syncwarp();
            if (lane < 16 && ((it.vmask >> lane) & 1u)) {
                const long long cell = ((long long)it.b * p.T + it.tstart + j) * p.HW + (it.y0 + (lane >> 2)) * p.W +
                                       it.x0 + (lane & 3);
                bulk_g2s(ring_base + s * p.slot_bytes + lane * p.row_bytes, p.feats + cell * p.D + rank * p.S,
                         (uint32_t)(p.S * 2), bar);
            }
        };
        if (warp == 0)
            for (int j = 0; j < min(p.R, it.n); j++) issue(j);

        if (!is_dec) {
            // ------------------------------ worker warps ------------------------------
            const int pair = tid;                       // channels 2*pair, 2*pair+1 of this CTA's slice
            const bool active = 2 * pair < p.S;
            for (int j = 0; j < it.n + 2; j++) {
                if (j < it.n) {
                    const int q = qbase + j, s = q % p.R;
                    const uint32_t bar = smem_u32(full_bar + s), parity = (uint32_t)((q / p.R) & 1);
                    int spins = 0;
                    while (!timed_out && !mbar_try_wait(bar, parity)) {
                        if (++spins > kSpinLimit) timed_out = true;
                    }
                    if (warp < p.NM) {
                        // Gram and cross matrices over this warp's share of the channels
                        // two independent accumulator sets keep twice as many tensor-core operations in flight
                        float g0[4] = {0.f, 0.f, 0.f, 0.f}, g1[4] = {0.f, 0.f, 0.f, 0.f};
                        float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
                        float h0[4] = {0.f, 0.f, 0.f, 0.f}, h1[4] = {0.f, 0.f, 0.f, 0.f};
                        float e0[4] = {0.f, 0.f, 0.f, 0.f}, e1[4] = {0.f, 0.f, 0.f, 0.f};
                        const uint32_t lrow = (lane & 7) + ((lane >> 3) & 1) * 8, lk = (lane >> 4) * 8;
                        const uint32_t cur = ring_base + s * p.slot_bytes + lrow * p.row_bytes + lk * 2;
                        const int sp = (q - 1 + p.R) % p.R;
                        const uint32_t prv = ring_base + sp * p.slot_bytes + lrow * p.row_bytes + lk * 2;
                        const int ksteps = p.S >> 4;
                        if (j > 0) {
                            for (int ks = warp; ks < ksteps; ks += 2 * p.NM) {
                                uint32_t a[4], b[4];
                                ldmatrix_x4(cur + ks * 32, a);
                                ldmatrix_x4(prv + ks * 32, b);
                                mma_bf16(g0, a, a[0], a[2]);
                                mma_bf16(g1, a, a[1], a[3]);
                                mma_bf16(c0, a, b[0], b[2]);
                                mma_bf16(c1, a, b[1], b[3]);
                                if (ks + p.NM < ksteps) {
                                    ldmatrix_x4(cur + (ks + p.NM) * 32, a);
                                    ldmatrix_x4(prv + (ks + p.NM) * 32, b);
                                    mma_bf16(h0, a, a[0], a[2]);
                                    mma_bf16(h1, a, a[1], a[3]);
                                    mma_bf16(e0, a, b[0], b[2]);
                                    mma_bf16(e1, a, b[1], b[3]);
                                }
                            }
                        } else {
                            for (int ks = warp; ks < ksteps; ks += 2 * p.NM) {
                                uint32_t a[4];
                                ldmatrix_x4(cur + ks * 32, a);
                                mma_bf16(g0, a, a[0], a[2]);
                                mma_bf16(g1, a, a[1], a[3]);
                                if (ks + p.NM < ksteps) {
                                    ldmatrix_x4(cur + (ks + p.NM) * 32, a);
                                    mma_bf16(h0, a, a[0], a[2]);
                                    mma_bf16(h1, a, a[1], a[3]);
                                }
                            }
                        }
#pragma unroll
                        for (int i = 0; i < 4; i++) { g0[i] += h0[i]; g1[i] += h1[i]; c0[i] += e0[i]; c1[i] += e1[i]; }
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
                }
                named_sync(1, nworkers);
                if (j < it.n) {
                    // contract the warps' partial matrices to the 8 numbers per cell and hand the CTA's
                    // share to every CTA of the cluster
                    for (int i = tid; i < kSumVals; i += nworkers) {
                        const float sum = combine_sums(red, p.NM, i & 15, i >> 4, W1s, W2s);
                        const uint32_t a = smem_u32(xchg + ((qbase + j) & 1) * p.C * kSumVals + rank * kSumVals + i);
                        for (int r = 0; r < p.C; r++) st_cluster_f32(map_to_rank(a, r), sum);
                    }
                }
                cluster_arrive();
                if (j >= 2) {
                    // execute the record of frame j-2 on the frame still in the ring
                    const int jj = j - 2;
                    const int need = qbase + jj + 1;
                    int spins = 0;
                    while (!timed_out && ld_acquire_cta(ctl + 1) < need) {
                        if (++spins > kSpinLimit) timed_out = true;
                    }
                    const FrameRec* rec = recs + ((qbase + jj) % kRecRing);
                    const int s = (qbase + jj) % p.R;
                    const uint32_t fb = ring_base + s * p.slot_bytes + pair * 4;
                    const long long ch2 = ((long long)rank * p.S >> 1) + pair;      // index in units of 2 channels
                    const long long D2 = p.D >> 1;
                    auto flush = [&](const FlushCmd& fc) {
                        float2 v = acc.take(fc.slot);
                        if (!active) return;
                        if (fc.kind == 0) {
                            v.x = v.x / fc.weight;
                            v.y = v.y / fc.weight;
                            if (p.out_f32) reinterpret_cast<float2*>(p.staging)[(long long)fc.dst * D2 + ch2] = v;
                            else reinterpret_cast<uint32_t*>(p.staging)[(long long)fc.dst * D2 + ch2] = pack_bf16x2(v);
                        } else {
                            reinterpret_cast<float2*>(p.pieces)[(long long)fc.dst * D2 + ch2] = v;
                        }
                    };
                    const int n_pre = rec->n_pre, n_nodes = rec->n_nodes, n_post = rec->n_post;
                    for (int i = 0; i < n_pre; i++) flush(rec->pre[i]);
                    for (int i = 0; i < n_nodes; i++) {
                        const NodeCmd nc = rec->node[i];
                        float2 f = make_float2(0.f, 0.f);
                        if (active) {
                            const uint32_t a0 = fb + nc.cell * p.row_bytes;
                            if (nc.lv == 0) {
                                f = unpack_bf16x2(lds_u32(a0));
                            } else if (nc.lv == 1) {
                                const float2 u0 = unpack_bf16x2(lds_u32(a0)), u1 = unpack_bf16x2(lds_u32(a0 + p.row_bytes));
                                const float2 u2 = unpack_bf16x2(lds_u32(a0 + 4 * p.row_bytes));
                                const float2 u3 = unpack_bf16x2(lds_u32(a0 + 5 * p.row_bytes));
                                f.x = (u0.x + u1.x) + (u2.x + u3.x);
                                f.y = (u0.y + u1.y) + (u2.y + u3.y);
                            } else {
#pragma unroll
                                for (int c = 0; c < 16; c++) {
                                    const float2 u = unpack_bf16x2(lds_u32(fb + c * p.row_bytes));
                                    f.x = fmaf(W2s[c], u.x, f.x);
                                    f.y = fmaf(W2s[c], u.y, f.y);
                                }
                            }
                            f.x *= nc.w;
                            f.y *= nc.w;
                        }
                        acc.add(nc.slot, f);
                    }
                    for (int i = 0; i < n_post; i++) flush(rec->post[i]);
                }
                cluster_wait();
                named_sync(1, nworkers);
                if (warp == 0 && j >= 2 && j - 2 + p.R < it.n) issue(j - 2 + p.R);
            }
        } else {
            // ------------------------------ decision warp ------------------------------
            DecState st;
            st.prev_lv = 0; st.prev_slot = 0; st.prev_nk = 0.f;
            st.active = 0;
            const float tau_s = taus.s[it.b], tau_t = taus.t[it.b];
            cluster_arrive();
            for (int j = 0; j < it.n + 2; j++) {
                cluster_wait();
                // take this frame's totals out of the exchange buffer, then let the cluster go on:
                // the decisions themselves run beside the workers' next frame
                float v[8];
                if (j < it.n) {
                    const float* xch = xchg + ((qbase + j) & 1) * p.C * kSumVals;
#pragma unroll
                    for (int k = 0; k < 8; k++) {
                        float sum = 0.f;
                        for (int r = 0; r < p.C; r++) sum += xch[r * kSumVals + k * 16 + (lane & 15)];
                        v[k] = sum;
                    }
                }
                if (j + 1 < it.n + 2) cluster_arrive();
                if (j < it.n) {
                    FrameRec* rec = recs + ((qbase + j) % kRecRing);
                    decide_frame(p, it, j, tau_s, tau_t, v, W1s, W2s, st, tab, rec, rank, lane);
                    if (lane == 0) st_release_cta(ctl + 1, qbase + j + 1);
                }
            }
        }
        qbase += it.n;
        __syncthreads();
    }
    if (timed_out && p.status != nullptr) atomicOr(p.status, kStatusWaitTimeout);
}

// ---------------------------------------------------------------------------------
// Roots (Section 3.3, "common root node").  Inside an item the fused kernel already follows
// every chain to its first node; a chain that enters an item from the frame before it is
// known there by that earlier node, whose own entry names a node further back.  One thread
// per cell walks these hand-overs (at most one per item border).
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
k_resolve_roots(Geo g, int max_hops, const int32_t* __restrict__ chain_key, int32_t* __restrict__ root,
                int32_t* status) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)g.B * g.N) return;
    const long long vb = i / g.N * g.N;
    int r = chain_key[i];
    int hops = 0;
    while (true) {
        const int up = chain_key[vb + r];
        if (up == r) break;
        r = up;
        if (++hops > max_hops) {
            if (status != nullptr) atomicOr(status, kStatusNotConverged);
            break;
        }
    }
    root[i] = r;
}

// ---------------------------------------------------------------------------------
// After the ordering: chains cut by item borders.  One thread per piece: find the row of
// the piece's chain, add its weight, push it on the row's list.
// ---------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
k_piece_link(Geo g, int npieces, const int2* __restrict__ piece_meta, const int32_t* __restrict__ root,
             const int32_t* __restrict__ row_at_root, const long long* __restrict__ vid_off,
             int32_t* __restrict__ row_head, int32_t* __restrict__ piece_next, int32_t* __restrict__ row_weight) {
    const int pc = blockIdx.x * blockDim.x + threadIdx.x;
    if (pc >= npieces) return;
    const int2 m = piece_meta[pc];
    if (m.x < 0) return;
    const int b = m.x / g.N;
    const long long vb = (long long)b * g.N;
    const int r = root[vb + (m.x - b * g.N)];
    const long long row = vid_off[b] + row_at_root[vb + r];
    piece_next[pc] = atomicExch(row_head + row, pc);
    atomicAdd(row_weight + row, m.y);
}

// One warp per output row: copy the staged row, or add the row's pieces in the order of
// their index (a fixed order, so the result does not depend on scheduling).
template <typename OutT>
__global__ void __launch_bounds__(256)
k_gather(Geo g, const long long* __restrict__ vid_off, const int32_t* __restrict__ row_anchor,
         const int32_t* __restrict__ row_head, const int32_t* __restrict__ piece_next,
         const int32_t* __restrict__ row_weight, const OutT* __restrict__ staging, const float* __restrict__ pieces,
         OutT* __restrict__ out, long long capacity) {
    const int lane = threadIdx.x & 31;
    const long long nrows = min(vid_off[g.B], capacity);
    const long long nwarps = (long long)gridDim.x * (blockDim.x >> 5);
    const int n16 = (int)((size_t)g.D * sizeof(OutT) / 16);
    for (long long r = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); r < nrows; r += nwarps) {
        const int head = row_head[r];
        if (head < 0) {
            int b = 0;                                  // video of the row: vid_off is short, walk it
            while (b + 1 < g.B && vid_off[b + 1] <= r) b++;
            const long long src = (long long)b * g.N + row_anchor[r];
            const uint4* s4 = reinterpret_cast<const uint4*>(staging + src * g.D);
            uint4* d4 = reinterpret_cast<uint4*>(out + r * g.D);
            for (int i0 = 0; i0 < n16; i0 += 8 * 32) {  // eight loads in flight per lane
                uint4 v[8];
#pragma unroll
                for (int k = 0; k < 8; k++) {
                    const int i = i0 + k * 32 + lane;
                    if (i < n16) v[k] = __ldcs(s4 + i);
                }
#pragma unroll
                for (int k = 0; k < 8; k++) {
                    const int i = i0 + k * 32 + lane;
                    if (i < n16) __stcs(d4 + i, v[k]);
                }
            }
        } else {
            const float wsum = (float)row_weight[r];
            for (int d = lane * VEC; d < g.D; d += kSliceCh) {
                float sum[VEC] = {0.f, 0.f, 0.f, 0.f};
                int last = -1;
                while (true) {          // next larger piece index on the row's (short) list
                    int best = 0x7fffffff;
                    for (int pc = head; pc >= 0; pc = piece_next[pc])
                        if (pc > last && pc < best) best = pc;
                    if (best == 0x7fffffff) break;
                    const float4 v = *reinterpret_cast<const float4*>(pieces + (long long)best * g.D + d);
                    sum[0] += v.x; sum[1] += v.y; sum[2] += v.z; sum[3] += v.w;
                    last = best;
                }
#pragma unroll
                for (int v = 0; v < VEC; v++) sum[v] = sum[v] / wsum;
                store4(out + r * g.D + d, sum);
            }
        }
    }
}

// merge map alone (per cell: row of the cell's chain inside its video)
__global__ void __launch_bounds__(256)
k_merge_map(Geo g, const int32_t* __restrict__ root, const int32_t* __restrict__ row_at_root,
            int32_t* __restrict__ merge_map) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)g.B * g.N) return;
    const long long vb = i / g.N * g.N;
    merge_map[i] = row_at_root[vb + root[i]];
}

}  // namespace sttm
