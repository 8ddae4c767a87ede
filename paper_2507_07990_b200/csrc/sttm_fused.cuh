// Fused single-read STTM kernel (sm_100a): spatial search, temporal linking and averaging
// in one pass over the features.
//
// Decomposition.  A frame is cut into 4x4-cell tiles (the region of a coarsest quadtree
// node when the tree has three levels; four / sixteen independent regions when it has two
// / one).  Everything that touches features stays inside one tile through time, so a work
// item is (video, tile, run of consecutive frames).  The partial tiles at the right and
// bottom border of a grid whose sides are not multiples of four are packed, several at a
// time, into the 16 rows of one "tile" of the kernel (they never interact: every lane knows
// which of its neighbours belong to its own 2x2 block and coarsest node).  A thread-block cluster of C CTAs owns
// a fixed list of items; each CTA owns D/C channels of the tile and streams them frame by
// frame through a shared-memory ring filled by bulk asynchronous copies (one per cell).
//
// The warps of a CTA are specialised and hand frames to each other through mbarriers, so
// that every stage works on a different frame at the same time:
//   producer warp   issues the bulk copies of the next frames as ring slots come free;
//   Gram warps      form the tile's Gram matrix G = X_t X_t^T and cross matrix
//                   C = X_t X_{t-1}^T over the CTA's channels on the tensor cores (X = the 16
//                   cells of the tile; products of bf16 inputs are exact, sums are fp32);
//   combine warps   add the Gram warps' parts, contract them to the 128 numbers the decisions
//                   need (every cosine of Sections 3.2 and 3.3 is a short linear combination
//                   of entries of G and C because parents are averages of cells) and send
//                   them to every CTA of the cluster (one bulk copy from shared memory to the other CTA's
//                   shared memory each, completing on that CTA's mbarrier);
//   similarity warp adds the cluster's shares in a fixed order and takes the decisions of
//                   Section 3.2 (cover map) and Section 3.3 (links), the same in every CTA;
//   chain warp      follows the chains through time: which running sum each kept node
//                   joins, which chains ended; leaves a command record per frame;
//   sum warps       execute the records on the frame that is still in the ring.  The record
//                   holds a 16x16 matrix W (chain slot x cell: the weight of the cell in the
//                   running sum of that chain), so the update of all running sums is one
//                   small matrix product  sums[16 x channels] += W X  on the tensor cores,
//                   with the sums living in the accumulator registers of the warps.
// Finished chains go to a staging row indexed by the root's cell id (their final row is
// only known after the global ordering); chains cut by the end of an item go to an fp32
// piece buffer and are put together by the gather kernel.
#pragma once

#include "sttm_device.cuh"
#include "sttm_kernels.cuh"

namespace sttm {

constexpr int kMaxTiles = 64;
constexpr int kMaxCluster = 8;
constexpr int kRecRing = 4;             // command records, hand-over slots and exchange buffers in flight
constexpr int kGramVals = 512;          // G (16x16) then C (16x16)
constexpr int kSumVals = 128;           // 8 numbers per cell, see combine_sums()
constexpr int kPieceSlots = 32;         // per item: 16 keyed by a cell of the frame before the item, 16 by chain slot
constexpr int kMaxRing = 12;
constexpr int kPrefetchAhead = 2;        // frames between a frame's L2 prefetch and its copy into the ring
constexpr int kPrefetchMinFrames = 128;  // items shorter than this do without (measured: no gain, small loss)
constexpr int kMaxGramWarps = 4;
constexpr int kCombineWarps = 4;
constexpr int kMaxSumWarps = 8;         // 128 channels each: at most 1024 channels per CTA
constexpr int kTailWarps = 4;           // similarity, chain, two producers
constexpr int kFusedMaxThreads = (kMaxGramWarps + kCombineWarps + kMaxSumWarps + kTailWarps) * 32;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // a wait gives up after two seconds

enum : int { kStatusWaitTimeout = 1 << 7 };         // 1 << STTM_ERR_TIMEOUT
// launch shape of the instantiation with constant shape (D = 3584 bf16)
constexpr int kFlagshipC = 4, kFlagshipS = 896, kFlagshipNM = 4, kFlagshipNA = 7;

struct FlushCmd { int slot, kind, dst; float weight; };     // kind 0: finished row, 1: piece
// Commands of one frame for the sum warps: first write out and clear the chain sums of the
// slots in flush_mask, flush[s] saying where slot s goes (chains that got no member in this
// frame; at the first frame of an item: everything the previous item left; all of them are
// written in one go, each slot by the lanes that hold it), then add W X to the running sums, W[slot][cell] (bf16; the weights
// are small integers times powers of two, hence exact) = weight of the cell in its kept node
// if that node belongs to the chain in `slot`, else 0.
struct FrameRec {
    uint32_t flush_mask, pad0, pad1, pad2;
    FlushCmd flush[16];
    uint16_t wmat[256];
};

// One tile of the kernel: up to 16 cells of a frame, row l of the tile = lane l of the
// decision warps.  y == 255: no cell.  bits: low nibble = which lane-index bits join the lanes
// of one 2x2 block (1: the lane to the right, 4: the lane below), high nibble = the same for
// the coarsest node (1, 2: along the row, 4, 8: down the column).  A full tile has 0xf5.
struct TileDesc {
    unsigned char y[16], x[16], bits[16];
};

struct FusedParams {
    const __nv_bfloat16* feats;
    int B, T, H, W, D, L;
    int HW, N;
    int Wt, ntiles;
    int C, S, NM, NA;        // cluster size, channels per CTA, Gram warps, sum warps
    int row_bytes, slot_bytes;
    int R, RB, lead;         // slots of the Gram warps' ring and of the sum warps' ring; see the second producer
    int F, nseg, nitems;
    int weight_mode, out_f32, match_best;
    int8_t* cover;
    int32_t* link;
    int32_t* chain_key;      // [B*N] per cell: root cell id of its chain as far as the item knows it
    int32_t* frame_roots;    // [B*T] chains that start in a frame (= its output rows), zero on entry
    float* tmax;             // budget mode, may be null: [B*N] per cell, at the top-left cell of a kept node the
                             // largest cosine to its candidates in the frame before, -2 elsewhere / without one
    const float* tau_t_dev;  // budget mode, may be null: [B] temporal thresholds in device memory
    void* staging;           // [B*N][D] rows of the output dtype
    float* pieces;           // [nitems][kPieceSlots][D]
    int2* piece_meta;        // [nitems][kPieceSlots] {key cell id or -1, weight}
    int* status;
    TileDesc tiles[kMaxTiles];   // most cells first
};

// ---------------------------------------------------------------------------------
// PTX helpers
// ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// arrive on an mbarrier of another CTA of the cluster (address from map_to_rank)
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// has the phase with this parity completed?  (no waiting: the callers spin on it, which hands a
// frame from warp to warp faster than a suspending wait does; measured 1.5 % of the kernel's time)
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait for the `use`-th completion (0-based) of an mbarrier: false when it has not
// come within kWaitLimitNs (or an earlier wait of this thread ran out).  The caller then
// leaves its loops without touching the data it waited for; the warps that depend on it
// run out in turn, every CTA still reaches the end of the kernel, and the host sees
// kStatusWaitTimeout in the status word.
__device__ __forceinline__ bool mbar_wait_lane(uint32_t bar, int use, bool& timed_out) {
    if (timed_out) return false;
    const uint32_t parity = (uint32_t)(use & 1);
    if (mbar_test(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    int tries = 0;
    while (!mbar_test(bar, parity)) {
        if ((++tries & 63) == 0 && global_timer_ns() - t0 > kWaitLimitNs) {
            timed_out = true;
            return false;
        }
    }
    return true;
}
// The same for a whole warp (every caller is one): the lanes agree on the outcome, so that a warp
// never splits at the time limit with some lanes leaving and the others entering a warp-wide
// primitive.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, int use, bool& timed_out) {
    const bool ok = mbar_wait_lane(bar, use, timed_out);
    const bool all = __all_sync(0xffffffffu, ok);
    if (!all) timed_out = true;
    return all;
}
// waits until a progress counter in shared memory (written by another warp of the CTA; only
// a timing hint, no data hangs on it) has reached `target`; time-bounded like mbar_wait
__device__ __forceinline__ bool hint_wait(const int* counter, int target, bool& timed_out) {
    bool ok = !timed_out;
    const volatile int* c = counter;
    if (ok && *c < target) {
        const unsigned long long t0 = global_timer_ns();
        while (*c < target) {
            __nanosleep(64);
            if (global_timer_ns() - t0 > kWaitLimitNs) { ok = false; break; }
        }
    }
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) timed_out = true;
    return ok;
}
// this CTA's shared memory -> shared memory of a CTA of the cluster, completion counted in
// bytes on that CTA's mbarrier (both given as cluster addresses)
__device__ __forceinline__ void bulk_s2s(uint32_t dst_cluster, uint32_t src, uint32_t bytes, uint32_t bar_cluster) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_cluster), "r"(src), "r"(bytes), "r"(bar_cluster)
                 : "memory");
}
// orders this thread's earlier writes to shared memory before later reads of the async proxy
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// asks for a piece of global memory to be brought into L2 (no completion, nothing to wait for)
__device__ __forceinline__ void bulk_prefetch_l2(const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
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
__device__ __forceinline__ uint32_t cluster_id() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_count() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
    uint32_t out;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(addr), "r"(rank));
    return out;
}
__device__ __forceinline__ void named_sync(int id, int count) {
    asm volatile("barrier.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
// named barrier that also returns the OR of a flag over its `count` threads
__device__ __forceinline__ bool named_sync_or(int id, int count, bool flag) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "barrier.red.or.pred q, %2, %3, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)flag), "r"(id), "r"(count)
        : "memory");
    return r != 0;
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
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
__device__ __forceinline__ float lds_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ float4 lds_f32x4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 lds_u32x4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds_u64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}

// What lane c of a decision warp knows about its cell: the lanes of its 2x2 block and of its
// coarsest node (bit masks over the 16 lanes, cells inside the grid only), the averaging
// weights (w1: of a cell in its block; w2: of a cell in the coarsest node = mean of the
// existing blocks' means), its position in the frame.
struct LaneGeo {
    bool valid;
    int qbits, tbits;
    uint32_t qmask, tmask;
    float w1, w2;
    int cell;               // y * W + x
};
// Pure function of the tile description: any thread can ask for any lane.
__device__ __forceinline__ LaneGeo lane_geo(const TileDesc& td, int c, int L, int W) {
    LaneGeo g;
    g.valid = td.y[c] != 255;
    g.qbits = L >= 2 ? (td.bits[c] & 15) : 0;
    g.tbits = L == 3 ? (td.bits[c] >> 4) : 0;
    g.qmask = 0;
    g.tmask = 0;
    int blocks = 0;
    for (int l = 0; l < 16; l++) {
        if (td.y[l] == 255) continue;
        const int ql = L >= 2 ? (td.bits[l] & 15) : 0, tl = L == 3 ? (td.bits[l] >> 4) : 0;
        if ((l & ~ql) == (c & ~g.qbits)) g.qmask |= 1u << l;
        if ((l & ~tl) == (c & ~g.tbits)) {
            g.tmask |= 1u << l;
            blocks += (l & ~ql) == l ? 1 : 0;         // top-left cells of the blocks of the node
        }
    }
    if (!g.valid) { g.qmask = 0; g.tmask = 0; }
    g.w1 = g.valid && L >= 2 ? 1.f / (float)__popc(g.qmask) : 0.f;
    g.w2 = g.valid && L == 3 ? g.w1 / (float)blocks : 0.f;
    g.cell = g.valid ? td.y[c] * W + td.x[c] : 0;
    return g;
}
// top-left lane of the level-lv node of lane c
__device__ __forceinline__ int lane_anchor(const LaneGeo& g, int c, int lv) {
    return lv == 0 ? c : (lv == 1 ? (c & ~g.qbits) : (c & ~g.tbits));
}
__device__ __forceinline__ uint32_t lane_region(const LaneGeo& g, int c, int lv) {
    return lv == 0 ? (g.valid ? 1u << c : 0u) : (lv == 1 ? g.qmask : g.tmask);
}
// position of the k-th (0-based) set bit of a 16-bit mask that has more than k bits set
__device__ __forceinline__ int kth_set_bit16(uint32_t m, int k) {
    int pos = 0;
    int n = __popc(m & 0xffu);
    if (k >= n) { k -= n; pos = 8; }
    n = __popc((m >> pos) & 0xfu);
    if (k >= n) { k -= n; pos += 4; }
    n = __popc((m >> pos) & 0x3u);
    if (k >= n) { k -= n; pos += 2; }
    n = (int)((m >> pos) & 1u);
    if (k >= n) pos += 1;
    return pos;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float x, float y) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
    return *reinterpret_cast<const uint32_t*>(&h);
}

// sum over the lanes of the lane's coarsest node (lanes 0..15 and 16..31 separately): a butterfly
// over the lane-index bits that stay inside the node
__device__ __forceinline__ float top_sum(float v, int tbits) {
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) {
        const float t = __shfl_xor_sync(0xffffffffu, v, o);
        v += (tbits & o) ? t : 0.f;
    }
    return v;
}
// sum over the lanes of the lane's 2x2 block
__device__ __forceinline__ float quad_sum(float v, int qbits) {
    float t = __shfl_xor_sync(0xffffffffu, v, 1);
    v += (qbits & 1) ? t : 0.f;
    t = __shfl_xor_sync(0xffffffffu, v, 4);
    v += (qbits & 4) ? t : 0.f;
    return v;
}
// cos(a, b) > tau from a.b, |a|^2, |b|^2 without a division; a zero vector has cosine 0
__device__ __forceinline__ float sqrt_fast(float x) {
    float r;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));      // a few ulp: far inside the decision margins
    return r;
}
__device__ __forceinline__ bool cos_above(float dot, float na, float nb, float tau) {
    if (na == 0.f || nb == 0.f) return 0.f > tau;
    return dot > tau * (sqrt_fast(na) * sqrt_fast(nb));
}

struct ItemGeo {
    int item, b, tstart, n, halo, last_seg;
    int tile;           // index into FusedParams::tiles
    uint32_t vmask;     // bit l: row l of the tile holds a cell
    int nvalid;
};

// The round-th item of this cluster: items are numbered from the most expensive tile to the
// cheapest and dealt to the clusters back and forth.  Returns false past the last round;
// `skip` says that this cluster has no item in the round.
__device__ __forceinline__ bool next_item(const FusedParams& p, int round, uint32_t cid, uint32_t ncl, ItemGeo& it,
                                          bool& skip) {
    const long long base = (long long)round * ncl;
    if (base >= p.nitems) return false;
    const long long idx = base + ((round & 1) ? (long long)(ncl - 1 - cid) : (long long)cid);
    skip = idx >= p.nitems;
    if (skip) return true;
    it.item = (int)idx;
    const int seg = it.item % p.nseg;
    const int tb = it.item / p.nseg;
    it.b = tb % p.B;
    it.tile = tb / p.B;
    const int t0 = seg * p.F, t1 = min(p.T, t0 + p.F);
    it.halo = t0 > 0;
    it.tstart = t0 - it.halo;
    it.n = t1 - it.tstart;
    it.last_seg = t1 == p.T;
    it.vmask = 0;
    for (int l = 0; l < 16; l++)
        if (p.tiles[it.tile].y[l] != 255) it.vmask |= 1u << l;
    it.nvalid = __popc(it.vmask);
    return true;
}

// The 8 numbers of cell c that the decisions need, as linear functions of the tile's Gram
// matrix G = X_t X_t^T and cross matrix Cm = X_t X_{t-1}^T (row: cell of frame t).  With
// q(c) the cell's 2x2 block, w1 / w2 the averaging weights of level 1 / level 2:
//   k=0  |x_c|^2                       k=1  x_c . parent(c)            k=2  x_c . top
//   k=3  x_c(t) . x_c(t-1)             k=4  x_c(t) . parent(c)(t-1)    k=5  x_c(t) . top(t-1)
//   k=6  parent(c)(t) . x_c(t-1)       k=7  top(t) . x_c(t-1)
// Ring rows without a cell hold stale finite data: such columns are masked here, and the
// similarity warp drops the numbers of such rows.  W2s: the 16 lanes' weights w2 in shared memory.
__device__ __forceinline__ float combine_sums(uint32_t G, int c, int k, const LaneGeo& g, uint32_t W2s) {
    const uint32_t Cm = G + 256 * 4;
    float v = 0.f;
    if (k == 0) {
        v = lds_f32(G + (c * 16 + c) * 4);
    } else if (k == 3) {
        v = lds_f32(Cm + (c * 16 + c) * 4);
    } else if (k == 1 || k == 4 || k == 6) {
        // the (up to) four cells of the 2x2 block: along the row of c (k = 1, 4) or down its column (k = 6)
        const uint32_t M = k == 1 ? G : Cm;
        const int qb = c & ~g.qbits;
        const int step = k == 6 ? 16 : 1;
        const uint32_t a = M + (k == 6 ? (qb * 16 + c) : (c * 16 + qb)) * 4;
        const float m0 = (g.qmask >> qb) & 1u ? 1.f : 0.f, m1 = (g.qbits & 1) && ((g.qmask >> (qb + 1)) & 1u) ? 1.f : 0.f;
        const float m2 = (g.qbits & 4) && ((g.qmask >> (qb + 4)) & 1u) ? 1.f : 0.f;
        const float m3 = (g.qbits & 5) == 5 && ((g.qmask >> (qb + 5)) & 1u) ? 1.f : 0.f;
        const float x0 = lds_f32(a), x1 = lds_f32(a + step * 4), x2 = lds_f32(a + 4 * step * 4),
                    x3 = lds_f32(a + 5 * step * 4);
        v = ((m0 * x0 + m1 * x1) + (m2 * x2 + m3 * x3)) * g.w1;
    } else {
        // weighted sum over the cells of the coarsest node: along the row of c (k = 2, 5) or down its column (k = 7)
        const uint32_t M = k == 2 ? G : Cm;
        if (k == 7) {
#pragma unroll
            for (int i = 0; i < 16; i++) {
                const float w = (g.tmask >> i) & 1u ? lds_f32(W2s + i * 4) : 0.f;
                v = fmaf(w, lds_f32(M + (i * 16 + c) * 4), v);
            }
        } else {
#pragma unroll
            for (int i = 0; i < 16; i += 4) {
                const float4 w = lds_f32x4(W2s + i * 4), x = lds_f32x4(M + (c * 16 + i) * 4);
                v = fmaf((g.tmask >> i) & 1u ? w.x : 0.f, x.x, v);
                v = fmaf((g.tmask >> (i + 1)) & 1u ? w.y : 0.f, x.y, v);
                v = fmaf((g.tmask >> (i + 2)) & 1u ? w.z : 0.f, x.z, v);
                v = fmaf((g.tmask >> (i + 3)) & 1u ? w.w : 0.f, x.w, v);
            }
        }
    }
    return v;
}

// Chain slots of the chain warp (shared memory, private to it).
struct SlotTable {
    int key[16], weight[16], virt[16], cell[16], row[16];
};

// ---------------------------------------------------------------------------------
// The kernel.  Warps: [0, NM) Gram, then 4 combine, NA sum, similarity, chain, two producers.
// ---------------------------------------------------------------------------------
// kLean: the common set-up (top-left destination, bf16 rows, one ring, thresholds from the host)
// with the options compiled out -- the budget mode's additions (best candidate cosine per kept
// node written to p.tmax with the sums left out; tau_t read from p.tau_t_dev), the second ring,
// fp32 rows, the most-similar destination.  The kernel is a chain of dependent instructions in
// seven code streams per SM: the unused branches cost 3 % of its time when they are present.
template <bool kLean, bool kFlagship>
__global__ void __launch_bounds__(kFusedMaxThreads, 1)
k_fused(const __grid_constant__ FusedParams p, const __grid_constant__ Taus taus) {
    extern __shared__ __align__(128) unsigned char smem[];
    // cluster size, channels per CTA, Gram and sum warps, levels: constants in the instantiation for
    // D = 3584 on three-level grids (the loops over the cluster's CTAs and a warp's channels unroll: 5 % faster)
    const int nC = kFlagship ? kFlagshipC : p.C, nS = kFlagship ? kFlagshipS : p.S;
    const int nNM = kFlagship ? kFlagshipNM : p.NM, nNA = kFlagship ? kFlagshipNA : p.NA;
    const int nL = kFlagship ? 3 : p.L;        // quadtree levels (13x13 ... 16x16 grids)
    const int nD = kFlagship ? kFlagshipC * kFlagshipS : p.D;
    const int RB2 = kLean ? 0 : p.RB;          // slots of the second ring
    unsigned char* ring = smem;
    size_t off = (size_t)(p.R + RB2) * p.slot_bytes;
    float* red = reinterpret_cast<float*>(smem + off);       off += (size_t)nNM * kGramVals * 4;
    float* redsum = reinterpret_cast<float*>(smem + off);    off += kGramVals * 4;
    float* xchg = reinterpret_cast<float*>(smem + off);      off += (size_t)kRecRing * nC * kSumVals * 4;
    float* wtab = reinterpret_cast<float*>(smem + off);      off += 128;              // the 16 lanes' weights w2 of the current item
    float* xsend = reinterpret_cast<float*>(smem + off);     off += kRecRing * kSumVals * 4;   // this CTA's share, staged for the bulk copies
    int* hand = reinterpret_cast<int*>(smem + off);          off += kRecRing * 16 * 4;
    SlotTable* tab = reinterpret_cast<SlotTable*>(smem + off); off += sizeof(SlotTable);
    FrameRec* recs = reinterpret_cast<FrameRec*>(smem + off); off += kRecRing * sizeof(FrameRec);
    int* hint = reinterpret_cast<int*>(smem + off);          off += 16;               // frames the similarity warp has finished
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + off);
    const uint32_t bar0 = smem_u32(bars);
    const uint32_t full_bar = bar0, empty_bar = bar0 + 8 * kMaxRing;
    const uint32_t fullb_bar = bar0 + 16 * kMaxRing, emptyb_bar = bar0 + 24 * kMaxRing;
    const uint32_t xfull_bar = bar0 + 32 * kMaxRing, xempty_bar = xfull_bar + 8 * kRecRing;
    const uint32_t hfull_bar = xempty_bar + 8 * kRecRing, hempty_bar = hfull_bar + 8 * kRecRing;
    const uint32_t rfull_bar = hempty_bar + 8 * kRecRing, rempty_bar = rfull_bar + 8 * kRecRing;
    const uint32_t gfull_bar = rempty_bar + 8 * kRecRing, gempty_bar = gfull_bar + 16;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_rank(), cid = cluster_id(), ncl = cluster_count();
    const uint32_t ring_base = smem_u32(ring), ringb_base = ring_base + p.R * p.slot_bytes;
    const int w_comb = nNM, w_sum = nNM + kCombineWarps, w_sim = w_sum + nNA, w_chain = w_sim + 1, w_prod = w_sim + 2;

    // set-up: barriers, a ring without NaN patterns
    if (tid == 0) {
        for (int s = 0; s < p.R; s++) {
            mbar_init(full_bar + 8 * s, 1);
            mbar_init(empty_bar + 8 * s, nNM + (RB2 == 0 ? nNA : 0));
        }
        for (int s = 0; s < RB2; s++) {
            mbar_init(fullb_bar + 8 * s, 1);
            mbar_init(emptyb_bar + 8 * s, nNA);
        }
        *hint = 0;
        for (int s = 0; s < kRecRing; s++) {
            mbar_init(xfull_bar + 8 * s, 1);
            mbar_init(xempty_bar + 8 * s, nC);
            mbar_init(hfull_bar + 8 * s, 1);
            mbar_init(hempty_bar + 8 * s, 1);
            mbar_init(rfull_bar + 8 * s, 1);
            mbar_init(rempty_bar + 8 * s, nNA);
        }
        for (int s = 0; s < 2; s++) {
            mbar_init(gfull_bar + 8 * s, nNM);
            mbar_init(gempty_bar + 8 * s, kCombineWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int k = tid * 16; k < (p.R + RB2) * p.slot_bytes; k += blockDim.x * 16)
        *reinterpret_cast<uint4*>(ring + k) = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    cluster_arrive();
    cluster_wait();         // every CTA of the cluster has its barriers before anyone signals them

    bool timed_out = false;
    ItemGeo it;
    bool skip;
    int q = 0;              // frames of this cluster so far (the same in every role)

    if (warp < nNM) {
        // ------------------------------------ Gram warps ------------------------------------
        const uint32_t lrow = (lane & 7) + ((lane >> 3) & 1) * 8, lk = (lane >> 4) * 8;
        const uint32_t loff = lrow * p.row_bytes + lk * 2;
        const int ksteps = nS >> 4;
        const int k0 = ksteps * warp / nNM, k1 = ksteps * (warp + 1) / nNM;     // this warp's channel steps
        int s = 0, use = 0;         // ring slot of frame q and how often it has been filled before (q = use * R + s)
        for (int round = 0; !timed_out && next_item(p, round, cid, ncl, it, skip); round++) {
            if (skip) continue;
            for (int j = 0; j < it.n; j++, q++) {
                if (!mbar_wait(full_bar + 8 * s, use, timed_out)) break;
                __syncwarp();
                float g0[4] = {0.f, 0.f, 0.f, 0.f}, g1[4] = {0.f, 0.f, 0.f, 0.f};
                float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
                float h0[4] = {0.f, 0.f, 0.f, 0.f}, h1[4] = {0.f, 0.f, 0.f, 0.f};
                float e0[4] = {0.f, 0.f, 0.f, 0.f}, e1[4] = {0.f, 0.f, 0.f, 0.f};
                const uint32_t cur = ring_base + s * p.slot_bytes + loff;
                const int sp = s == 0 ? p.R - 1 : s - 1;
                const uint32_t prv = ring_base + sp * p.slot_bytes + loff;
                // two accumulator sets; the fragments of a step are loaded before the products of the
                // step before it are issued (the index is clamped at the end: a repeated load, no branch)
                uint32_t a[4], b[4], a2[4], b2[4];
                const int kl = k1 - 1;
                ldmatrix_x4(cur + k0 * 32, a);
                ldmatrix_x4(prv + k0 * 32, b);
                int ks = k0;
                for (; ks + 1 < k1; ks += 2) {
                    ldmatrix_x4(cur + (ks + 1) * 32, a2);
                    ldmatrix_x4(prv + (ks + 1) * 32, b2);
                    mma_bf16(g0, a, a[0], a[2]);
                    mma_bf16(g1, a, a[1], a[3]);
                    mma_bf16(c0, a, b[0], b[2]);
                    mma_bf16(c1, a, b[1], b[3]);
                    const int kn = min(ks + 2, kl);
                    ldmatrix_x4(cur + kn * 32, a);
                    ldmatrix_x4(prv + kn * 32, b);
                    mma_bf16(h0, a2, a2[0], a2[2]);
                    mma_bf16(h1, a2, a2[1], a2[3]);
                    mma_bf16(e0, a2, b2[0], b2[2]);
                    mma_bf16(e1, a2, b2[1], b2[3]);
                }
                if (ks < k1) {
                    mma_bf16(g0, a, a[0], a[2]);
                    mma_bf16(g1, a, a[1], a[3]);
                    mma_bf16(c0, a, b[0], b[2]);
                    mma_bf16(c1, a, b[1], b[3]);
                }
                // the combine warps have taken the previous frame's parts out of the buffer?
                if (q >= 1 && !mbar_wait(gempty_bar, q - 1, timed_out)) break;
                __syncwarp();
                {
                    float* r = red + warp * kGramVals;
                    const int gr = lane >> 2, gc = (lane & 3) * 2;
                    *reinterpret_cast<float2*>(r + gr * 16 + gc) = make_float2(g0[0] + h0[0], g0[1] + h0[1]);
                    *reinterpret_cast<float2*>(r + (gr + 8) * 16 + gc) = make_float2(g0[2] + h0[2], g0[3] + h0[3]);
                    *reinterpret_cast<float2*>(r + gr * 16 + 8 + gc) = make_float2(g1[0] + h1[0], g1[1] + h1[1]);
                    *reinterpret_cast<float2*>(r + (gr + 8) * 16 + 8 + gc) = make_float2(g1[2] + h1[2], g1[3] + h1[3]);
                    *reinterpret_cast<float2*>(r + 256 + gr * 16 + gc) = make_float2(c0[0] + e0[0], c0[1] + e0[1]);
                    *reinterpret_cast<float2*>(r + 256 + (gr + 8) * 16 + gc) = make_float2(c0[2] + e0[2], c0[3] + e0[3]);
                    *reinterpret_cast<float2*>(r + 256 + gr * 16 + 8 + gc) = make_float2(c1[0] + e1[0], c1[1] + e1[1]);
                    *reinterpret_cast<float2*>(r + 256 + (gr + 8) * 16 + 8 + gc) =
                        make_float2(c1[2] + e1[2], c1[3] + e1[3]);
                }
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(gfull_bar);
                    // done with the previous frame's slot (the current one stays for the next frame)
                    if (q >= 1) mbar_arrive(empty_bar + 8 * sp);
                }
                if (++s == p.R) { s = 0; use++; }
            }
        }
    } else if (warp < w_sum) {
        // ----------------------------------- combine warps -----------------------------------
        const int ctid = tid - w_comb * 32, nthr = kCombineWarps * 32;
        const uint32_t red_a = smem_u32(red), redsum_a = smem_u32(redsum);
        // this thread's entry of the exchange buffers and the matching barrier in every CTA of the cluster
        // (entry i = 8 numbers x 16 cells, stored [cell][number]; a CTA with fewer than 128 combine
        // threads would loop, so the addresses are per entry index ctid only when nthr == 128)
        // Thread r < C sends the whole share (128 numbers) to CTA r with one bulk copy from shared
        // memory to that CTA's shared memory: one completion on the receiver's barrier instead of 128.
        const uint32_t peer_x = map_to_rank(smem_u32(xchg + rank * kSumVals), ctid < nC ? ctid : 0);
        const uint32_t peer_bar = map_to_rank(xfull_bar, ctid < nC ? ctid : 0);
        const uint32_t xsend_a = smem_u32(xsend);
        for (int round = 0; !timed_out && next_item(p, round, cid, ncl, it, skip); round++) {
            if (skip) continue;
            // this thread's cell and the weights of all 16 lanes for the sums over the coarsest node
            const LaneGeo lg = lane_geo(p.tiles[it.tile], ctid & 15, nL, p.W);
            const uint32_t W2s = smem_u32(wtab);
            named_sync(1, nthr);                       // the previous item's weights are not read any more
            if (ctid < 16) wtab[ctid] = lg.w2;
            named_sync(1, nthr);
            for (int j = 0; j < it.n; j++, q++) {
                // the first combine warp waits; the named barriers hand the outcome to the others
                if (warp == w_comb) mbar_wait(gfull_bar, q, timed_out);
                if (named_sync_or(3, nthr, timed_out)) { timed_out = true; break; }
                // add the Gram warps' parts, each thread a share of the 512 entries
                for (int i = ctid * 4; i < kGramVals; i += nthr * 4) {
                    float4 sum = lds_f32x4(red_a + i * 4);
                    for (int w = 1; w < nNM; w++) {
                        const float4 v = lds_f32x4(red_a + (w * kGramVals + i) * 4);
                        sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
                    }
                    *reinterpret_cast<float4*>(redsum + i) = sum;
                }
                named_sync(1, nthr);
                if (lane == 0) mbar_arrive(gempty_bar);
                // contract to 8 numbers per cell and send this CTA's share to every CTA of the cluster
                const int xb = q % kRecRing;
                if (warp == w_comb && q >= kRecRing) mbar_wait(xempty_bar + 8 * xb, q / kRecRing - 1, timed_out);
                if (named_sync_or(2, nthr, timed_out)) { timed_out = true; break; }
                {
                    // (the staging buffer of this frame was last used four frames ago, and the wait above
                    // says that every CTA has consumed that frame)
                    xsend[xb * kSumVals + (ctid & 15) * 8 + (ctid >> 4)] = combine_sums(redsum_a, ctid & 15, ctid >> 4, lg, W2s);
                    fence_async_smem();                 // the copies below read what was just written normally
                    named_sync(1, nthr);
                    if (ctid < nC)
                        bulk_s2s(peer_x + xb * nC * kSumVals * 4, xsend_a + xb * kSumVals * 4, kSumVals * 4, peer_bar + 8 * xb);
                }
            }
        }
    } else if (warp < w_sim) {
        // ------------------------------------ sum warps ------------------------------------
        // Warp a owns channels [128 a, 128 a + 128) of the CTA's slice: 16 tiles of 8 channels.
        // sums[nt][0..3] is the accumulator fragment of tile nt: chain slots g and g + 8
        // (g = lane / 4), channels 2 t and 2 t + 1 of the tile (t = lane % 4).
        float sums[16][4];
#pragma unroll
        for (int nt = 0; nt < 16; nt++)
#pragma unroll
            for (int k = 0; k < 4; k++) sums[nt][k] = 0.f;
        const int ch0 = (warp - w_sum) * 128;
        const int g = lane >> 2, t4 = lane & 3;
        const uint32_t recs_a = smem_u32(recs);
        // B fragments (cells x 16 channels) by transposing loads: lane l addresses row (cell) l%8 + 8*((l>>3)&1)
        // of the 8-channel column block l>>4
        const uint32_t xoff = ((lane & 7) + ((lane >> 3) & 1) * 8) * p.row_bytes + (ch0 + (lane >> 4) * 8) * 2;
        // A fragment (16 slots x 16 cells) straight from the record
        const uint32_t woff = 16 + 256 + ((lane & 7) + ((lane >> 3) & 1) * 8) * 32 + (lane >> 4) * 16;
        const long long chan = (long long)rank * nS + ch0 + 2 * t4;
        const int ntmax = min(16, (nS - ch0) >> 3);         // 8-channel tiles of this warp inside the slice
        int total = 0;
        for (int round = 0; next_item(p, round, cid, ncl, it, skip); round++)
            if (!skip) total += it.n;
        // the frames come from a ring of their own, or (RB == 0) from the Gram warps' ring
        const bool own = RB2 > 0;
        const uint32_t sfull_bar = own ? fullb_bar : full_bar, sempty_bar = own ? emptyb_bar : empty_bar;
        const uint32_t sbase = own ? ringb_base : ring_base;
        const int SR = own ? RB2 : p.R;
        // one record per frame, and a last one that only writes out what the last item left
        int s = 0, use = 0;         // ring slot of frame q and how often it has been filled before
        for (; q <= total; q++) {
            const int rk = q % kRecRing;
            if (!mbar_wait(rfull_bar + 8 * rk, q / kRecRing, timed_out)) break;
            if (q < total && !mbar_wait(sfull_bar + 8 * s, use, timed_out)) break;
            __syncwarp();
            const uint32_t rec = recs_a + rk * (uint32_t)sizeof(FrameRec);
            // (first pass of the budget mode: only the decisions are wanted, nothing is summed or written)
            const bool dry = !kLean && p.tmax != nullptr;
            const uint32_t flush_mask = dry ? 0u : lds_u32x4(rec).x;
            // Slots g and g + 8 live in the four lanes of group g: all slots of one half of the
            // fragment are written in the same pass, every group following its own command.  One
            // loop per kind of destination and per half keeps register indices and offsets static.
#pragma unroll 1
            for (int hi = 0; hi < 2; hi++) {
                const uint32_t m8 = (flush_mask >> (8 * hi)) & 0xffu;
                if (m8 == 0) continue;
                const bool mine = (m8 >> g) & 1u;
                const uint4 fc = lds_u32x4(rec + 16 + (g + 8 * hi) * 16);       // slot, kind, dst, weight
                const float inv = mine && fc.y == 0 ? 1.f / __uint_as_float(fc.w) : 1.f;
                const long long row = (long long)(int)fc.z * nD + chan;
#define STTM_FLUSH_LOOP(I0, I1, STORE)                                        \
    _Pragma("unroll") for (int nt = 0; nt < 16; nt++) {                       \
        const float x = sums[nt][I0] * inv, y = sums[nt][I1] * inv;           \
        sums[nt][I0] = 0.f;                                                   \
        sums[nt][I1] = 0.f;                                                   \
        if (nt < ntmax) { STORE; }                                            \
    }
#define STTM_FLUSH_KINDS(I0, I1)                                                                              \
    if (fc.y != 0) {                                                                                          \
        float* dst = p.pieces + row;                                                                          \
        STTM_FLUSH_LOOP(I0, I1, *reinterpret_cast<float2*>(dst + nt * 8) = make_float2(x, y))                 \
    } else if ((!kLean && p.out_f32)) {                                                                                   \
        float* dst = reinterpret_cast<float*>(p.staging) + row;                                               \
        STTM_FLUSH_LOOP(I0, I1, *reinterpret_cast<float2*>(dst + nt * 8) = make_float2(x, y))                 \
    } else {                                                                                                  \
        /* bf16 rows: two 8-channel tiles per store, so that the four lanes of a slot write one whole  */    \
        /* 32-byte sector (the words of a 16-channel block are left in the order lane, tile; the        */    \
        /* gather kernel puts them back in channel order)                                               */    \
        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.staging) + row + 2 * t4;                      \
        _Pragma("unroll") for (int j = 0; j < 8; j++) {                                                       \
            const uint32_t lo = pack_bf16x2(sums[2 * j][I0] * inv, sums[2 * j][I1] * inv);                    \
            const uint32_t up = pack_bf16x2(sums[2 * j + 1][I0] * inv, sums[2 * j + 1][I1] * inv);            \
            sums[2 * j][I0] = 0.f; sums[2 * j][I1] = 0.f;                                                     \
            sums[2 * j + 1][I0] = 0.f; sums[2 * j + 1][I1] = 0.f;                                             \
            if (2 * j < ntmax) *reinterpret_cast<uint2*>(dst + j * 16) = make_uint2(lo, up);                  \
        }                                                                                                     \
    }
                if (mine) {
                    if (hi) { STTM_FLUSH_KINDS(2, 3) } else { STTM_FLUSH_KINDS(0, 1) }
                }
#undef STTM_FLUSH_KINDS
#undef STTM_FLUSH_LOOP
            }
            __syncwarp();
            if (q < total && !dry) {
                uint32_t wa[4];
                ldmatrix_x4(rec + woff, wa);
                const uint32_t xb = sbase + s * p.slot_bytes + xoff;
#pragma unroll
                for (int pr = 0; pr < 8; pr++) {
                    if (ch0 + pr * 16 < nS) {
                        uint32_t xb4[4];
                        ldmatrix_x4_trans(xb + pr * 32, xb4);
                        mma_bf16(sums[2 * pr], wa, xb4[0], xb4[1]);
                        mma_bf16(sums[2 * pr + 1], wa, xb4[2], xb4[3]);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(rempty_bar + 8 * rk);
                if (q < total) mbar_arrive(sempty_bar + 8 * s);
            }
            if (++s == SR) { s = 0; use++; }
        }
    } else if (warp == w_sim) {
        // --------------------------------- similarity warp ---------------------------------
        // Two frames per pass: lanes 0..15 take frame q, lanes 16..31 frame q + 1; lane c and
        // lane c + 16 are cell c of the tile.
        const unsigned full = 0xffffffffu;
        const int c = lane & 15, half = lane >> 4;
        const int L = nL;
        const uint32_t xchg_a = smem_u32(xchg);
        for (int round = 0; !timed_out && next_item(p, round, cid, ncl, it, skip); round++) {
            if (skip) continue;
            const float tau_s = taus.s[it.b], tau_t = (!kLean && p.tau_t_dev != nullptr) ? p.tau_t_dev[it.b] : taus.t[it.b];
            const LaneGeo lg = lane_geo(p.tiles[it.tile], c, L, p.W);
            const float w1 = lg.w1, w2 = lg.w2;
            const bool valid = lg.valid;
            int carry_lv = 0;               // cover level / squared norm of the node covering cell c in the
            float carry_nk = 0.f;           // last frame of the previous pass
            for (int j = 0; j < it.n; j += 2) {
                const bool two = j + 1 < it.n;
                const int myq = q + half, xb = myq % kRecRing;
                const bool mine = half == 0 || two;                 // this half has a frame
                if (lane == 0) {
                    mbar_expect_tx(xfull_bar + 8 * (q % kRecRing), (uint32_t)(nC * kSumVals * 4));
                    if (two) mbar_expect_tx(xfull_bar + 8 * ((q + 1) % kRecRing), (uint32_t)(nC * kSumVals * 4));
                }
                if (!mbar_wait(xfull_bar + 8 * (q % kRecRing), q / kRecRing, timed_out)) break;
                if (two && !mbar_wait(xfull_bar + 8 * ((q + 1) % kRecRing), (q + 1) / kRecRing, timed_out)) break;
                __syncwarp();
                float v[8];
                {
                    const uint32_t xch = xchg_a + (xb * nC * kSumVals + c * 8) * 4;
                    float4 lo = lds_f32x4(xch), hi = lds_f32x4(xch + 16);
                    for (int r = 1; r < nC; r++) {          // the CTAs' shares, in rank order
                        const float4 l2 = lds_f32x4(xch + r * kSumVals * 4), h2 = lds_f32x4(xch + r * kSumVals * 4 + 16);
                        lo.x += l2.x; lo.y += l2.y; lo.z += l2.z; lo.w += l2.w;
                        hi.x += h2.x; hi.y += h2.y; hi.z += h2.z; hi.w += h2.w;
                    }
                    // cells outside the grid (stale ring rows) and a half without a frame: dropped
                    const bool keep = valid && mine;
                    v[0] = keep ? lo.x : 0.f; v[1] = keep ? lo.y : 0.f; v[2] = keep ? lo.z : 0.f; v[3] = keep ? lo.w : 0.f;
                    v[4] = keep ? hi.x : 0.f; v[5] = keep ? hi.y : 0.f; v[6] = keep ? hi.z : 0.f; v[7] = keep ? hi.w : 0.f;
                }
                __syncwarp();
                if (c < nC && mine) mbar_arrive_remote(map_to_rank(xempty_bar + 8 * xb, c));

                // Section 3.2: cosine of every node with its parent, then the coarse-to-fine search
                const float n0 = v[0], d0 = v[1], rr = v[2];
                const float n1 = w1 * quad_sum(d0, lg.qbits);    // |parent|^2
                const float d1 = w1 * quad_sum(rr, lg.qbits);    // parent . top
                const float n2 = top_sum(w2 * rr, lg.tbits);     // |top|^2
                int lv = 0;
                if (L >= 2) {
                    const bool p0 = !valid || cos_above(d0, n0, n1, tau_s);
                    const uint32_t pm0 = (__ballot_sync(full, p0) >> (16 * half)) & 0xffffu;
                    const bool quad_pass = (pm0 & lg.qmask) == lg.qmask;
                    if (L == 3) {
                        const bool p1 = !valid || cos_above(d1, n1, n2, tau_s);
                        const uint32_t pm1 = (__ballot_sync(full, p1) >> (16 * half)) & 0xffffu;
                        lv = (pm1 & lg.tmask) == lg.tmask ? 2 : (quad_pass ? 1 : 0);
                    } else {
                        lv = quad_pass ? 1 : 0;
                    }
                }
                const float nk = lv == 0 ? n0 : (lv == 1 ? n1 : n2);

                // Section 3.3: the node covering the cell against the overlapping kept node of the
                // previous frame (for the upper half: the lower half's frame); a pair is evaluated
                // at the top-left cell of its finer node
                const int lv_lo = __shfl_sync(full, lv, c), lv_hi = __shfl_sync(full, lv, 16 + c);
                const float nk_lo = __shfl_sync(full, nk, c), nk_hi = __shfl_sync(full, nk, 16 + c);
                const int lu = half ? lv_lo : carry_lv;
                const float pnk = half ? nk_lo : carry_nk;
                int link_local = -1;
                {
                    const float t11 = w1 * quad_sum(v[4], lg.qbits), t12 = w1 * quad_sum(v[5], lg.qbits);
                    const float t21 = w1 * quad_sum(v[7], lg.qbits), t22 = top_sum(w2 * v[5], lg.tbits);
                    float dot;
                    if (lv == 0) dot = lu == 0 ? v[3] : (lu == 1 ? v[4] : v[5]);
                    else if (lv == 1) dot = lu == 0 ? v[6] : (lu == 1 ? t11 : t12);
                    else dot = lu == 0 ? v[7] : (lu == 1 ? t21 : t22);
                    const bool has_prev = j + half > 0;
                    const bool rep = valid && has_prev && lane_anchor(lg, c, min(lv, lu)) == c;
                    const bool pass = rep && cos_above(dot, nk, pnk, tau_t);
                    const uint32_t passm = (__ballot_sync(full, pass) >> (16 * half)) & 0xffffu;
                    const uint32_t cand = passm & lane_region(lg, c, lv);
                    int cstar = cand ? __ffs(cand) - 1 : 0;           // first in row-major order: the top-left one
                    if (!kLean && p.match_best) {
                        // the most similar of them instead (equal ones: the first); the cosine itself is
                        // needed here, every lane looks at the 16 lanes of its half
                        const float cosv = pass ? dot / (sqrtf(nk) * sqrtf(pnk)) : -2.f;
                        float best = -2.f;
#pragma unroll
                        for (int i = 0; i < 16; i++) {
                            const float si = __shfl_sync(full, cosv, 16 * half + i);
                            if (((cand >> i) & 1u) && si > best) { best = si; cstar = i; }
                        }
                    }
                    if (!kLean && p.tmax != nullptr) {
                        // budget mode: the number of rows as a function of tau_t only needs, per kept node,
                        // the largest cosine to its candidates (the node is linked iff that exceeds tau_t)
                        const float cosv = rep ? ((nk == 0.f || pnk == 0.f) ? 0.f : dot / (sqrtf(nk) * sqrtf(pnk))) : -2.f;
                        const uint32_t candm = ((__ballot_sync(full, rep) >> (16 * half)) & 0xffffu) & lane_region(lg, c, lv);
                        float most = -2.f;
#pragma unroll
                        for (int i = 0; i < 16; i++) {
                            const float si = __shfl_sync(full, cosv, 16 * half + i);
                            if (((candm >> i) & 1u) && si > most) most = si;
                        }
                        if (rank == 0 && mine && valid && !(it.halo && j + half == 0))
                            p.tmax[(long long)it.b * p.N + (long long)(it.tstart + j + half) * p.HW + lg.cell] =
                                lane_anchor(lg, c, lv) == c ? most : -2.f;
                    }
                    const int lu_star = __shfl_sync(full, lu, 16 * half + cstar);
                    link_local = cand ? lane_anchor(lg, cstar, lu_star) : -1;      // same sub-tile: same bits
                }
                carry_lv = two ? lv_hi : lv_lo;
                carry_nk = two ? nk_hi : nk_lo;

                // hand the cover level and the link of every cell to the chain warp
                if (q >= kRecRing && !mbar_wait(hempty_bar + 8 * (q % kRecRing), q / kRecRing - 1, timed_out)) break;
                if (two && q + 1 >= kRecRing &&
                    !mbar_wait(hempty_bar + 8 * ((q + 1) % kRecRing), (q + 1) / kRecRing - 1, timed_out))
                    break;
                __syncwarp();
                if (mine) hand[xb * 16 + c] = lv | ((link_local + 1) << 8);
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(hfull_bar + 8 * (q % kRecRing));
                    if (two) mbar_arrive(hfull_bar + 8 * ((q + 1) % kRecRing));
                }
                // cover map and links go out from here, after the hand-over: this warp has more slack
                // than the chain warp, whose time per frame weighs most on the pipeline
                {
                    const int lcell = __shfl_sync(full, lg.cell, 16 * half + (link_local < 0 ? 0 : link_local));
                    const int tt = it.tstart + j + half;
                    if (rank == 0 && mine && valid && !(it.halo && j + half == 0)) {
                        const long long gcc = (long long)it.b * p.N + (long long)tt * p.HW + lg.cell;
                        p.cover[gcc] = (int8_t)lv;
                        p.link[gcc] = link_local < 0 ? -1 : (tt - 1) * p.HW + lcell;
                    }
                }
                q += two ? 2 : 1;
                if (lane == 0) *reinterpret_cast<volatile int*>(hint) = q;
            }
        }
    } else if (warp == w_chain) {
        // ------------------------------------ chain warp ------------------------------------
        const unsigned full = 0xffffffffu;
        const int c = lane & 15;
        const bool low = lane < 16;
        // what the previous item left running when it ended: written out by the next record
        FlushCmd carry = FlushCmd{0, 0, 0, 0.f};     // lane s < 16: slot s
        uint32_t carry_mask = 0;
        for (int round = 0; !timed_out && next_item(p, round, cid, ncl, it, skip); round++) {
            if (skip) continue;
            const LaneGeo lg = lane_geo(p.tiles[it.tile], c, nL, p.W);
            const bool valid = lg.valid;
            const float w1 = lg.w1, w2 = lg.w2;
            if (rank == 0) p.piece_meta[(long long)it.item * kPieceSlots + lane] = make_int2(-1, 0);
            int prev_slot = 0;
            uint32_t active_slots = 0;
            for (int j = 0; j < it.n; j++, q++) {
                const int hb = q % kRecRing;
                if (!mbar_wait(hfull_bar + 8 * hb, q / kRecRing, timed_out)) break;
                __syncwarp();
                const int packed = hand[hb * 16 + c];
                __syncwarp();
                if (lane == 0) mbar_arrive(hempty_bar + 8 * hb);
                const int lv = packed & 3, link_local = (packed >> 8) - 1;
                if (q >= kRecRing && !mbar_wait(rempty_bar + 8 * hb, q / kRecRing - 1, timed_out)) break;
                __syncwarp();
                FrameRec* rec = recs + hb;
                const int t = it.tstart + j;
                const bool is_halo = it.halo && j == 0;
                const bool is_last = j == it.n - 1;

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
                // every new chain is an output row of this frame (the ordering needs the count per frame)
                if (rank == 0 && lane == 0 && !is_halo && freshm != 0) atomicAdd(p.frame_roots + it.b * p.T + t, __popc(freshm));
                const int slot_fresh = kth_set_bit16(freem, __popc(freshm & ((1u << c) - 1)));
                const int node_slot = linked ? slot_linked : slot_fresh;
                const int cur_slot = __shfl_sync(full, node_slot, (lane & 16) + lane_anchor(lg, c, lv));
                const uint32_t cells = lane_region(lg, c, lv);
                const int wint = p.weight_mode ? __popc(cells) : 1;
                const long long gc = (long long)it.b * p.N + (long long)t * p.HW + lg.cell;

                // chains that ended: lane s looks at slot s (before the slot is given away again); at
                // the first frame of an item nothing of the item runs yet and the list is the carry
                if (low && ((dead >> lane) & 1u)) {
                    if (tab->virt[lane]) {
                        const int pc = it.item * kPieceSlots + tab->cell[lane];
                        rec->flush[lane] = FlushCmd{lane, 1, pc, 0.f};
                        if (rank == 0) p.piece_meta[pc] = make_int2(tab->key[lane], tab->weight[lane]);
                    } else {
                        rec->flush[lane] = FlushCmd{lane, 0, tab->key[lane], (float)tab->weight[lane]};
                    }
                }
                // (nothing of the item runs at its first frame: dead and the carry never meet)
                if (low && ((carry_mask >> lane) & 1u)) rec->flush[lane] = carry;
                const uint32_t flush_mask = dead | carry_mask;
                carry_mask = 0;
                __syncwarp();
                if (low && fresh) {
                    tab->key[slot_fresh] = (int)gc;
                    tab->weight[slot_fresh] = is_halo ? 0 : wint;
                    tab->virt[slot_fresh] = is_halo ? 1 : 0;
                    tab->cell[slot_fresh] = c;
                }
                if (low && linked) atomicAdd(&tab->weight[slot_linked], wint);
                // the frame's weight matrix: row = chain slot, column = cell
                reinterpret_cast<uint4*>(rec->wmat)[lane] = make_uint4(0u, 0u, 0u, 0u);
                const int wnode = __shfl_sync(full, wint, (lane & 16) + lane_anchor(lg, c, lv));
                __syncwarp();
                if (low && valid && !is_halo) {
                    const float wc = (lv == 0 ? 1.f : (lv == 1 ? w1 : w2)) * (float)wnode;
                    rec->wmat[cur_slot * 16 + c] = __bfloat16_as_ushort(__float2bfloat16_rn(wc));
                }
                if (lane == 0) rec->flush_mask = flush_mask;
                const uint32_t active = memb | __reduce_or_sync(full, fresh ? 1u << slot_fresh : 0u);
                __syncwarp();
                // the record is complete: the sum warps may start while the rest of the frame's
                // bookkeeping (global arrays, the carry of an ending item) is still written
                if (lane == 0) mbar_arrive(rfull_bar + 8 * hb);

                if (rank == 0 && !is_halo && low && valid) {
                    p.chain_key[gc] = tab->key[cur_slot] - it.b * p.N;
                }
                if (is_last) {
                    // the item ends: everything still running is written out by the next record
                    carry_mask = active;
                    if (low && ((active >> lane) & 1u)) {
                        if (!tab->virt[lane] && it.last_seg) {
                            carry = FlushCmd{lane, 0, tab->key[lane], (float)tab->weight[lane]};
                        } else {
                            const int pc = it.item * kPieceSlots + 16 + lane;
                            carry = FlushCmd{lane, 1, pc, 0.f};
                            if (rank == 0) p.piece_meta[pc] = make_int2(tab->key[lane], tab->weight[lane]);
                        }
                    }
                }
                active_slots = is_last ? 0u : active;
                prev_slot = cur_slot;
                __syncwarp();
            }
        }
        if (q < kRecRing || mbar_wait(rempty_bar + 8 * (q % kRecRing), q / kRecRing - 1, timed_out)) {
            // last record: only the carry of the last item
            const int hb = q % kRecRing;
            __syncwarp();
            FrameRec* rec = recs + hb;
            if (low && ((carry_mask >> lane) & 1u)) rec->flush[lane] = carry;
            if (lane == 0) rec->flush_mask = carry_mask;
            __syncwarp();
            if (lane == 0) mbar_arrive(rfull_bar + 8 * hb);
        }
    } else if (warp == w_prod || (warp == w_prod + 1 && RB2 == 0)) {
        // ---------------------------------- producer warps ----------------------------------
        // Issuing one bulk copy costs a warp some 80 cycles, and a frame is 16 of them, so two
        // warps share the rows (with a second ring the second warp has that ring to fill, and
        // this one issues all 16).
        const int nprod = RB2 == 0 ? 2 : 1, which = warp - w_prod;
        const int row = lane * nprod + which;              // the tile row this lane copies
        int s = 0, use = 0;         // ring slot of frame q and how often it has been filled before
        for (int round = 0; !timed_out && next_item(p, round, cid, ncl, it, skip); round++) {
            if (skip) continue;
            for (int j = 0; j < it.n; j++, q++) {
                const uint32_t bar = full_bar + 8 * s;
                if (use >= 1 && !mbar_wait(empty_bar + 8 * s, use - 1, timed_out)) break;
                __syncwarp();
                // (one warp announces the bytes of the whole frame; a copy of the other warp that lands
                // before that only makes the count run negative for a moment)
                if (lane == 0 && which == 0) mbar_expect_tx(bar, (uint32_t)(it.nvalid * nS * 2));
                __syncwarp();
                if (row < 16 && ((it.vmask >> row) & 1u)) {
                    const long long cell = ((long long)it.b * p.T + it.tstart + j) * p.HW +
                                           p.tiles[it.tile].y[row] * p.W + p.tiles[it.tile].x[row];
                    bulk_g2s(ring_base + s * p.slot_bytes + row * p.row_bytes, p.feats + cell * nD + rank * nS,
                             (uint32_t)(nS * 2), bar);
                    // the frame kPrefetchAhead frames on is called into L2 now (its copy then takes less of
                    // the slot's time); the CTAs of the cluster share the cells out and ask for whole rows
                    if (p.F >= kPrefetchMinFrames && j + kPrefetchAhead < it.n && row % nC == (int)rank)
                        bulk_prefetch_l2(p.feats + (cell + (long long)kPrefetchAhead * p.HW) * nD, (uint32_t)(nD * 2));
                }
                if (++s == p.R) { s = 0; use++; }
            }
        }
        // the CTA must not end with copies in flight: the last R frames issued have landed?
        // (immediate in a normal run; after a wait ran out, each of these waits is bounded again)
        for (int qq = max(0, q - p.R); qq < q; qq++) {
            bool late = false;
            mbar_wait(full_bar + 8 * (qq % p.R), qq / p.R, late);
            timed_out |= late;
        }
    } else if (warp == w_prod + 1 && RB2 > 0) {
        // ---------------------------------- second producer ----------------------------------
        // The sum warps need a frame only once its record exists, long after the Gram warps are
        // done with it.  Holding the frame in shared memory all that time would let too few frames
        // be in flight, so it is fetched a second time (from L2, where the first copy left it) into
        // a ring of its own, timed by the similarity warp's progress so that it lands about when
        // the chain warp posts the record.  (With RB == 0 there is one ring for both and this warp
        // has nothing to do.)
        int s = 0, use = 0;
        for (int round = 0; !timed_out && next_item(p, round, cid, ncl, it, skip); round++) {
            if (skip) continue;
            for (int j = 0; j < it.n; j++, q++) {
                const uint32_t bar = fullb_bar + 8 * s;
                if (!hint_wait(hint, q + 1 - p.lead, timed_out)) break;
                if (use >= 1 && !mbar_wait(emptyb_bar + 8 * s, use - 1, timed_out)) break;
                __syncwarp();
                if (lane == 0) mbar_expect_tx(bar, (uint32_t)(it.nvalid * nS * 2));
                __syncwarp();
                if (lane < 16 && ((it.vmask >> lane) & 1u)) {
                    const long long cell = ((long long)it.b * p.T + it.tstart + j) * p.HW +
                                           p.tiles[it.tile].y[lane] * p.W + p.tiles[it.tile].x[lane];
                    bulk_g2s(ringb_base + s * p.slot_bytes + lane * p.row_bytes, p.feats + cell * nD + rank * nS,
                             (uint32_t)(nS * 2), bar);
                }
                if (++s == RB2) { s = 0; use++; }
            }
        }
        const int rb = kLean ? 1 : RB2;       // (this role does not exist in the lean kernel)
        for (int qq = max(0, q - RB2); qq < q; qq++) {
            bool late = false;
            mbar_wait(fullb_bar + 8 * (qq % rb), qq / rb, late);
            timed_out |= late;
        }
    }
    // nobody leaves while a CTA of the cluster may still store into it or signal its barriers
    __syncwarp();
    cluster_arrive();
    cluster_wait();
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
    wait_for_prior_kernel();
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
// After the ordering: chains cut by item borders.  A row that is put together from pieces is
// named by its smallest piece index, the leader.  k_piece_link (one thread per piece) finds the
// piece's row, adds its weight and proposes itself as the row's leader; k_piece_group (after it)
// enters every piece in its leader's list.
// ---------------------------------------------------------------------------------
constexpr int kRowPieces = 64;          // pieces listed per row; a row with more is found by a scan of all pieces

__global__ void __launch_bounds__(256)
k_piece_link(Geo g, int npieces, int max_hops, const int2* __restrict__ piece_meta, const int32_t* __restrict__ chain_key,
             const int32_t* __restrict__ row_at_root, const long long* __restrict__ vid_off,
             int32_t* __restrict__ row_head, int32_t* __restrict__ piece_row, int32_t* __restrict__ lead_n,
             int32_t* __restrict__ row_weight, int32_t* status) {
    wait_for_prior_kernel();
    const int pc = blockIdx.x * blockDim.x + threadIdx.x;
    if (pc >= npieces) return;
    lead_n[pc] = 0;
    if (pc == 0) lead_n[npieces] = 0;                   // number of leaders, counted by k_piece_group
    const int2 m = piece_meta[pc];
    if (m.x < 0) { piece_row[pc] = -1; return; }
    const int b = m.x / g.N;
    const long long vb = (long long)b * g.N;
    // the root of the piece's chain: the hand-over walk of k_resolve_roots, for this one cell
    int r = chain_key[m.x];
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
    const long long row = vid_off[b] + row_at_root[vb + r];
    piece_row[pc] = (int32_t)row;
    atomicMax(row_head + row, npieces - pc);           // (0: no piece yet; the smallest index gives the largest entry)
    atomicAdd(row_weight + row, m.y);
}

__global__ void __launch_bounds__(256)
k_piece_group(int npieces, const int32_t* __restrict__ piece_row, const int32_t* __restrict__ row_head,
              int32_t* __restrict__ lead_n, int32_t* __restrict__ lead_ids, int32_t* __restrict__ lead_list) {
    wait_for_prior_kernel();
    const int pc = blockIdx.x * blockDim.x + threadIdx.x;
    if (pc >= npieces) return;
    const int row = piece_row[pc];
    if (row < 0) return;
    const int leader = npieces - row_head[row];
    const int at = atomicAdd(lead_n + leader, 1);
    if (at < kRowPieces) lead_ids[(long long)leader * kRowPieces + at] = pc;
    // the leaders, in any order (every row is added up on its own): the gather walks this list only
    if (pc == leader) lead_list[atomicAdd(lead_n + npieces, 1)] = pc;
}

// Gather: kGatherParts warps per output row, each a contiguous share of the channels.  Two
// kernels over the same rows, because the two kinds of row want different register budgets:
// k_gather_rows copies the rows that are one finished staging row (bandwidth: many warps, few
// registers), k_gather_pieces adds the pieces of the rows whose chains were cut by item borders,
// in the order of their index (a fixed order, so the result does not depend on scheduling).  A row
// of pieces is bound by the latency of its dependent loads (list head -> piece ids -> data), so
// every warp issues all loads of its share before it adds anything.
constexpr int kGatherParts = 4;
template <typename OutT>
__global__ void __launch_bounds__(256)
k_gather_rows(Geo g, const long long* __restrict__ vid_off, const int32_t* __restrict__ row_anchor,
              const int32_t* __restrict__ row_head, const OutT* __restrict__ staging, OutT* __restrict__ out,
              long long capacity) {
    wait_for_prior_kernel();
    const int lane = threadIdx.x & 31;
    const long long nunits = min(vid_off[g.B], capacity) * kGatherParts;
    const long long nwarps = (long long)gridDim.x * (blockDim.x >> 5);
    const int n16 = (int)((size_t)g.D * sizeof(OutT) / 16);         // 16-byte pieces of a row
    for (long long unit = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); unit < nunits; unit += nwarps) {
        const long long r = unit / kGatherParts;
        const int part = (int)(unit % kGatherParts);
        if (row_head[r] != 0) continue;                 // a row of pieces
        int b = 0;                                      // video of the row: vid_off is short, walk it
        while (b + 1 < g.B && vid_off[b + 1] <= r) b++;
        const long long src = (long long)b * g.N + row_anchor[r];
        const uint4* s4 = reinterpret_cast<const uint4*>(staging + src * g.D);
        uint4* d4 = reinterpret_cast<uint4*>(out + r * g.D);
        // (shares begin on whole 32-byte blocks: an even index goes to an even lane)
        const int lo = (int)((long long)(n16 / 2) * part / kGatherParts) * 2;
        const int hi = part + 1 == kGatherParts ? n16 : (int)((long long)(n16 / 2) * (part + 1) / kGatherParts) * 2;
        for (int i0 = lo; i0 < hi; i0 += 4 * 32) {      // four loads in flight per lane
            uint4 v[4];
#pragma unroll
            for (int k = 0; k < 4; k++) {
                const int i = i0 + k * 32 + lane;
                v[k] = make_uint4(0u, 0u, 0u, 0u);
                if (i < hi) v[k] = __ldcs(s4 + i);
            }
            if constexpr (sizeof(OutT) == 2) {
                // bf16 staging rows hold the eight words of every 16-channel block in the order
                // 0 4 1 5 | 2 6 3 7 (the fused kernel's store pattern): two neighbouring lanes hold one
                // block and swap two words each
                const bool odd = lane & 1;
#pragma unroll
                for (int k = 0; k < 4; k++) {
                    const uint32_t r0 = __shfl_xor_sync(0xffffffffu, odd ? v[k].x : v[k].y, 1);
                    const uint32_t r1 = __shfl_xor_sync(0xffffffffu, odd ? v[k].z : v[k].w, 1);
                    v[k] = odd ? make_uint4(r0, r1, v[k].y, v[k].w) : make_uint4(v[k].x, v[k].z, r0, r1);
                }
            }
#pragma unroll
            for (int k = 0; k < 4; k++) {
                const int i = i0 + k * 32 + lane;
                if (i < hi) __stcs(d4 + i, v[k]);
            }
        }
    }
}

// Rows put together from pieces: kPieceParts warps per such row, the rows taken from the list of
// leader pieces.  The pieces are added in the order of their index (a fixed order, so the result
// does not depend on scheduling); such a row is bound by the latency of its dependent loads
// (leader -> list -> data), so the grid holds as many warps as the GPU keeps resident and two pieces'
// loads are issued before anything is added.
constexpr int kPieceParts = 8;
template <typename OutT>
__global__ void __launch_bounds__(256, 3)
k_gather_pieces(Geo g, int npieces, const int32_t* __restrict__ piece_row, const int32_t* __restrict__ lead_n,
                const int32_t* __restrict__ lead_ids, const int32_t* __restrict__ lead_list,
                const int32_t* __restrict__ row_weight, const float* __restrict__ pieces, OutT* __restrict__ out,
                long long capacity) {
    wait_for_prior_kernel();
    __shared__ int s_ids[8][2 * kRowPieces];
    const int lane = threadIdx.x & 31;
    const long long nunits = (long long)lead_n[npieces] * kPieceParts;
    const long long nwarps = (long long)gridDim.x * (blockDim.x >> 5);
    const int nf4 = g.D / VEC;                                      // 4-channel groups of a row
    int* ids = s_ids[threadIdx.x >> 5];
    int* sorted = ids + kRowPieces;
    for (long long unit = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); unit < nunits; unit += nwarps) {
        const int leader = lead_list[unit / kPieceParts], part = (int)(unit % kPieceParts);
        const int n_all = lead_n[leader];
        const long long r = piece_row[leader];
        if (r >= capacity) continue;
        const int n = min(n_all, kRowPieces);
        __syncwarp();
        for (int i = lane; i < n; i += 32) ids[i] = lead_ids[(long long)leader * kRowPieces + i];
        const float wsum = (float)row_weight[r];
        __syncwarp();
        for (int i = lane; i < n; i += 32) {
            const int mine = ids[i];
            int rank = 0;
            for (int k = 0; k < n; k++) rank += ids[k] < mine ? 1 : 0;
            sorted[rank] = mine;
        }
        __syncwarp();
        const int lo = (int)((long long)nf4 * part / kPieceParts), hi = (int)((long long)nf4 * (part + 1) / kPieceParts);
        for (int f0 = lo + lane; f0 < hi; f0 += 4 * 32) {
            float sum[4][VEC];
#pragma unroll
            for (int u = 0; u < 4; u++)
#pragma unroll
                for (int v = 0; v < VEC; v++) sum[u][v] = 0.f;
            if (n_all <= kRowPieces) {
                for (int k0 = 0; k0 < n; k0 += 2) {
                    float4 v[2][4];
#pragma unroll
                    for (int k = 0; k < 2; k++) {
                        if (k0 + k < n) {
                            const float4* src = reinterpret_cast<const float4*>(pieces + (long long)sorted[k0 + k] * g.D);
#pragma unroll
                            for (int u = 0; u < 4; u++)
                                if (f0 + u * 32 < hi) v[k][u] = __ldcs(src + f0 + u * 32);
                        }
                    }
#pragma unroll
                    for (int k = 0; k < 2; k++) {
                        if (k0 + k < n) {
#pragma unroll
                            for (int u = 0; u < 4; u++)
                                if (f0 + u * 32 < hi) {
                                    sum[u][0] += v[k][u].x; sum[u][1] += v[k][u].y; sum[u][2] += v[k][u].z; sum[u][3] += v[k][u].w;
                                }
                        }
                    }
                }
            } else {
                // more pieces than a list holds: all pieces are looked through, in index order
                for (int q = leader; q < npieces; q++) {
                    if (piece_row[q] != (int32_t)r) continue;
                    const float4* src = reinterpret_cast<const float4*>(pieces + (long long)q * g.D);
#pragma unroll
                    for (int u = 0; u < 4; u++)
                        if (f0 + u * 32 < hi) {
                            const float4 v = src[f0 + u * 32];
                            sum[u][0] += v.x; sum[u][1] += v.y; sum[u][2] += v.z; sum[u][3] += v.w;
                        }
                }
            }
#pragma unroll
            for (int u = 0; u < 4; u++)
                if (f0 + u * 32 < hi) {
#pragma unroll
                    for (int v = 0; v < VEC; v++) sum[u][v] = sum[u][v] / wsum;
                    store4(out + r * g.D + (long long)(f0 + u * 32) * VEC, sum[u]);
                }
        }
    }
}

// merge map alone (per cell: row of the cell's chain inside its video)
__global__ void __launch_bounds__(256)
k_merge_map(Geo g, const int32_t* __restrict__ root, const int32_t* __restrict__ row_at_root,
            int32_t* __restrict__ merge_map) {
    wait_for_prior_kernel();
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)g.B * g.N) return;
    const long long vb = i / g.N * g.N;
    merge_map[i] = row_at_root[vb + root[i]];
}

// ---------------------------------------------------------------------------------
// Budget mode: the temporal threshold that leaves at most `budget` rows.  With the cover maps
// fixed (tau_s), a kept node is merged into the frame before iff the largest cosine m to its
// candidates exceeds tau_t, so rows(tau_t) = nodes - #{m > tau_t}: the threshold is put in the
// middle of the gap between the k-th and the (k+1)-th largest m, k = nodes - budget.  One block
// per video; the k-th largest value by three histogram passes over the order-preserving bit
// pattern of the floats.
// ---------------------------------------------------------------------------------
struct Budgets { long long rows[kMaxBatch]; };

__device__ __forceinline__ uint32_t float_key(float f) {
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// One block: k-th largest (k >= 1) of the values > -1.5 among v[0..n), or -2 when there are fewer
// than k; *cand receives their number.  Three histogram passes (11 + 11 + 10 bits of the key).
__device__ float block_kth_largest(const float* __restrict__ v, long long n, long long k, uint32_t* hist,
                                   long long* cand) {
    __shared__ uint32_t s_prefix, s_mask;
    __shared__ long long s_k, s_total;
    if (threadIdx.x == 0) { s_prefix = 0; s_mask = 0; s_k = k; }
    __syncthreads();
    const int shifts[3] = {21, 10, 0}, bits[3] = {11, 11, 10};
    for (int pass = 0; pass < 3; pass++) {
        const int nb = 1 << bits[pass];
        for (int i = threadIdx.x; i < 2048; i += blockDim.x) hist[i] = 0;
        __syncthreads();
        const uint32_t prefix = s_prefix, mask = s_mask;
#pragma unroll 8
        for (long long i = threadIdx.x; i < n; i += blockDim.x) {
            const float f = v[i];
            if (f > -1.5f) {
                const uint32_t key = float_key(f);
                if ((key & mask) == prefix) atomicAdd(&hist[(key >> shifts[pass]) & (nb - 1)], 1u);
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            if (pass == 0) {
                long long total = 0;
                for (int b = 0; b < nb; b++) total += hist[b];
                s_total = total;
            }
            long long kk = s_k;
            int b = nb - 1;
            for (; b > 0; b--) {               // from the largest bin down
                if ((long long)hist[b] >= kk) break;
                kk -= hist[b];
            }
            s_k = kk;
            s_prefix = prefix | ((uint32_t)b << shifts[pass]);
            s_mask = mask | ((uint32_t)(nb - 1) << shifts[pass]);
        }
        __syncthreads();
        if (pass == 0 && s_total < k) break;    // fewer candidates than k (the same for every thread)
    }
    *cand = s_total;
    return s_total < k ? -2.f : key_float(s_prefix);
}

__global__ void __launch_bounds__(1024)
k_budget_tau(long long N, const float* __restrict__ tmax, const int32_t* __restrict__ nodes, Budgets budgets,
             float* __restrict__ tau_t) {
    wait_for_prior_kernel();
    __shared__ uint32_t hist[2048];
    __shared__ unsigned long long s_above, s_equal;
    __shared__ uint32_t s_below;            // key of the largest value below the k-th largest
    const int b = blockIdx.x;
    const float* v = tmax + (long long)b * N;
    const long long k = (long long)nodes[b] - budgets.rows[b];          // nodes that have to be merged away
    float tau;
    if (k <= 0) {
        tau = 2.f;                                                      // fits without temporal merging
    } else {
        long long cand;
        const float mk = block_kth_largest(v, N, k, hist, &cand);
        if (k > cand) {
            tau = -2.f;                                                 // not reachable: link whatever can be linked
        } else {
            // the (k+1)-th largest: mk again if enough values equal it, else the largest value below it
            if (threadIdx.x == 0) { s_above = 0; s_equal = 0; s_below = 0; }
            __syncthreads();
            unsigned long long above = 0, equal = 0;
            uint32_t below = 0;
#pragma unroll 8
            for (long long i = threadIdx.x; i < N; i += blockDim.x) {
                const float f = v[i];
                if (f > -1.5f) {
                    above += f > mk;
                    equal += f == mk;
                    if (f < mk) below = max(below, float_key(f));
                }
            }
            atomicAdd(&s_above, above);
            atomicAdd(&s_equal, equal);
            atomicMax(&s_below, below);
            __syncthreads();
            float mk1;
            if (k + 1 <= (long long)(s_above + s_equal)) mk1 = mk;
            else if (k + 1 <= cand) mk1 = key_float(s_below);
            else mk1 = mk - 2e-3f;
            tau = 0.5f * (mk + mk1);
        }
    }
    if (threadIdx.x == 0) tau_t[b] = tau;
}

}  // namespace sttm
