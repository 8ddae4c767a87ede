// Gram stage of the two-stream kernels on the fifth-generation tensor cores (tcgen05, sm_100a).
//
// Same task and same result as k_flow<false>: per (tile, frame, channel slice) the 128 numbers of
// combine_sums(), i.e. linear combinations of G = X_t X_t^T and C = X_t X_{t-1}^T over the slice's
// channels (Sections 3.2 and 3.3: all cosines of a tile are such combinations).  What differs is
// where the sums over channels are formed.  Four consecutive frames of a tile are the 64 rows of
// the A operand, the same four frames with the frame before them the 80 rows of B:
//     D[64 x 80] += A[64 x 16 channels] B[80 x 16 channels]^T        (tcgen05.mma, M = 64, N = 80, K = 16)
// over all 16-channel steps of the slice, with D in tensor memory.  Frame q's rows meet the columns
// of frame q - 1 in block (q, q): that is C; and its own columns in block (q, q + 1): that is G.
// One thread issues the products; nothing is added across warps and no barrier stands between the
// frames.  An M = 64 accumulator keeps rows 16 q ... 16 q + 15 in lanes 32 q ... 32 q + 15, which are
// the lanes warp q of a warpgroup may read: warp q reads out frame q, contracts it and stores it.
//
// One tensor copy brings five frames of a tile and NB 64-channel blocks into a ring slot as
// [block][frame][cell][64 channels] under the 128-byte swizzle (the tensor map has the frame axis
// inside the block axis), which is the K-major operand layout of the products: rows of 128 bytes,
// groups of eight rows 1024 bytes apart.  The frame before the group is loaded again with it (it
// comes out of L2); copies of this size stream at the full rate with one CTA per SM.
#pragma once

#include "sttm_flow.cuh"

namespace sttm {

constexpr int kTcFrames = 4;                         // frames per product: the 64 rows of A
constexpr int kTcBoxFrames = kTcFrames + 1;          // with the frame before them: the 80 rows of B
constexpr int kTcMaxNB = 7;                          // 64-channel blocks per slice
constexpr int kTcRing = 3;
constexpr int kTcReaders = 4;                        // read-out warps: one per frame of a group
constexpr int kTcThreads = (2 + kTcReaders) * 32;    // producer warp, product warp, read-out warps
constexpr uint32_t kTcCols = 256;                    // tensor-memory columns: two accumulators, 128 apart
constexpr uint32_t kTcAccStride = 128;
constexpr int kTcBlkBytes = kTcBoxFrames * kBlkBytes;

// instruction descriptor of tcgen05.mma kind::f16: fp32 accumulator (bits 4-5 = 1), bf16 A and B
// (bits 7-9 and 10-12 = 1), both K-major (bits 15, 16 = 0), N / 8 in bits 17-22, M / 16 in bits 24-28
constexpr uint32_t kTcIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTcBoxFrames * 16 / 8) << 17) |
                              ((uint32_t)(kTcFrames * 16 / 16) << 24);

// shared-memory operand descriptor, K-major, 128-byte swizzle: start address / 16 in bits 0-13,
// leading offset (unused for this layout) 1 in bits 16-29, 1024 bytes between groups of eight rows
// (/ 16) in bits 32-45, descriptor version 1 in bits 46-47, swizzle mode 2 in bits 61-63
__device__ __forceinline__ uint64_t tc_operand(uint32_t smem_addr) {
    return (uint64_t)((smem_addr & 0x3ffffu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}
// (the two descriptors differ from product to product only in their address field, the low word:
// the one thread that issues the products should have little else to do per product)
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
        ::"r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(kTcIdesc), "r"(accumulate)
        : "memory");
}
// the mbarrier gets one arrival when every product issued so far by this thread has completed
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// 32 consecutive columns of this warp's 32 lanes: lane i receives row i
__device__ __forceinline__ void tc_load32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// five frames of one tile, NB 64-channel blocks from block `blk0` on (coordinates: channel, x, y, frame, block)
__device__ __forceinline__ void tc_load_group(uint32_t dst, const CUtensorMap* map, int x, int y, int frame, int blk0,
                                              uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(x), "r"(y), "r"(frame), "r"(blk0), "r"(bar)
        : "memory");
}

// Groups of four frames of an item.  The frame before a run is not among them: it is only the
// "frame before" of the first group (the decision stage takes its own numbers from the run before).
__device__ __forceinline__ int tc_groups(const FlowItem& it) { return (it.n - it.halo + kTcFrames - 1) / kTcFrames; }

__host__ __device__ inline size_t tc_smem_bytes(int NBg) {
    return (size_t)kTcRing * NBg * kTcBlkBytes + (size_t)kTcReaders * kGramVals * 4 + kTcReaders * 64 + 16 +
           (2 * kTcRing + 4) * 8 + 1024;
}

// p.NSg slices of p.NCg x p.NBg blocks; tasks = (item, slice); partial is [nitems][F+1][NSg][128]
__global__ void __launch_bounds__(kTcThreads, 1)
k_flow_gram_tc(const __grid_constant__ FlowParams p, const __grid_constant__ FlowMaps maps) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const uint32_t slot_bytes = (uint32_t)p.NBg * kTcBlkBytes;
    size_t off = (size_t)kTcRing * slot_bytes;
    float* sums = reinterpret_cast<float*>(smem + off);            off += (size_t)kTcReaders * kGramVals * 4;
    float* wtab = reinterpret_cast<float*>(smem + off);            off += kTcReaders * 64;
    uint32_t* tmem_word = reinterpret_cast<uint32_t*>(smem + off); off += 16;
    const uint32_t bar0 = smem_u32(smem + off);
    const uint32_t full_bar = bar0, empty_bar = bar0 + 8 * kTcRing;
    const uint32_t acc_full = bar0 + 16 * kTcRing, acc_empty = acc_full + 16;
    const uint32_t ring_base = smem_u32(smem);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < kTcRing; s++) {
            mbar_init(full_bar + 8 * s, 1);
            mbar_init(empty_bar + 8 * s, 1);
        }
        for (int b = 0; b < 2; b++) {
            mbar_init(acc_full + 8 * b, 1);
            mbar_init(acc_empty + 8 * b, kTcReaders);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_word)), "r"(kTcCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_word);

    const int ntasks = p.nitems * p.NSg;
    bool timed_out = false;
    int q = 0, qc = 0;              // groups (copies) taken up so far by this CTA, see the roles

    if (warp == 0) {
        // ------------------------------------- producer -------------------------------------
        for (int task = blockIdx.x; task < ntasks && !timed_out; task += gridDim.x) {
            const FlowItem it = flow_item(p, task / p.NSg);
            const int slice = task % p.NSg;
            const TileBox bx = p.boxes[it.tile];
            const int ngroups = tc_groups(it);
            // one copy per group and part of the slice's channels: q counts copies here
            for (int gh = 0; gh < ngroups * p.NCg && !timed_out; gh++, q++) {
                const int g = gh / p.NCg, h = gh % p.NCg;
                const int s = q % kTcRing;
                // (this warp and the next have nothing else to do: they poll, which sees a completed phase
                // sooner than a suspended wait is woken, and a slot that waits is bandwidth lost)
                if (q >= kTcRing && !mbar_wait(empty_bar + 8 * s, q / kTcRing - 1, timed_out)) break;
                if (lane == 0) {
                    mbar_expect_tx(full_bar + 8 * s, slot_bytes);
                    tc_load_group(ring_base + s * slot_bytes, &maps.m[bx.kind], bx.x0, bx.y0,
                                  it.b * p.T + it.tstart + it.halo + g * kTcFrames - 1, (slice * p.NCg + h) * p.NBg,
                                  full_bar + 8 * s);
                }
                __syncwarp();
            }
        }
        // the CTA must not end with copies in flight
        for (int qq = max(0, q - kTcRing); qq < q; qq++) {
            bool late = false;
            mbar_wait_sleep(full_bar + 8 * (qq % kTcRing), qq / kTcRing, late);
            timed_out |= late;
        }
    } else if (warp == 1) {
        // ------------------------------------- products -------------------------------------
        for (int task = blockIdx.x; task < ntasks && !timed_out; task += gridDim.x) {
            const FlowItem it = flow_item(p, task / p.NSg);
            const int ngroups = tc_groups(it);
            // q counts groups (accumulator q % 2), qc copies (ring slot qc % kTcRing): the parts of a
            // slice's channels arrive in NCg copies and are added into the same accumulator
            for (int g = 0; g < ngroups && !timed_out; g++, q++) {
                const int b = q & 1;
                if (q >= 2 && !mbar_wait(acc_empty + 8 * b, (q >> 1) - 1, timed_out)) break;
                for (int h = 0; h < p.NCg; h++, qc++) {
                    const int s = qc % kTcRing;
                    if (!mbar_wait(full_bar + 8 * s, qc / kTcRing, timed_out)) break;
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t d = tmem_base + b * kTcAccStride;
                        const uint64_t b0 = tc_operand(ring_base + s * slot_bytes);
                        const uint32_t hi = (uint32_t)(b0 >> 32);
                        uint32_t b_lo = (uint32_t)b0, a_lo = b_lo + (kBlkBytes >> 4);   // A: without the frame before
                        for (int blk = 0; blk < p.NBg; blk++, a_lo += kTcBlkBytes >> 4, b_lo += kTcBlkBytes >> 4) {
#pragma unroll
                            for (int k = 0; k < 4; k++) tc_mma(d, a_lo + 2 * k, b_lo + 2 * k, hi, (h | blk | k) != 0);
                        }
                        tc_commit(empty_bar + 8 * s);                           // the slot has been read
                        if (h + 1 == p.NCg) tc_commit(acc_full + 8 * b);        // the sums are complete
                    }
                    __syncwarp();
                }
            }
        }
        // (the last products have completed before the tensor memory is given back)
        for (int qq = max(0, q - 2); qq < q; qq++) {
            bool late = false;
            mbar_wait_sleep(acc_full + 8 * (qq & 1), qq >> 1, late);
            timed_out |= late;
        }
    } else {
        // ------------------------------------- read-out -------------------------------------
        const int fq = warp & 3;                            // the lanes this warp may read hold frame fq of a group
        float* mine = sums + (warp - 2) * kGramVals;
        float* wt = wtab + (warp - 2) * 16;
        const uint32_t mine_a = smem_u32(mine), W2s = smem_u32(wt);
        for (int task = blockIdx.x; task < ntasks && !timed_out; task += gridDim.x) {
            const FlowItem it = flow_item(p, task / p.NSg);
            const int slice = task % p.NSg;
            const LaneGeo lg = lane_geo(p.tiles[it.tile], lane & 15, p.L, p.W);
            __syncwarp();
            if (lane < 16) wt[lane] = lg.w2;
            __syncwarp();
            float* dst = p.partial + ((long long)it.item * (p.F + 1) * p.NSg + slice) * kSumVals;
            const int ngroups = tc_groups(it);
            for (int g = 0; g < ngroups; g++, q++) {
                const int b = q & 1;
                if (!mbar_wait(acc_full + 8 * b, q >> 1, timed_out)) break;
                tc_fence_after();
                // columns 16 fq ... 16 fq + 15: the frame before (C); the next 16: the frame itself (G)
                uint32_t v[32];
                tc_load32(tmem_base + ((uint32_t)(32 * fq) << 16) + b * kTcAccStride + 16 * fq, v);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(acc_empty + 8 * b);
                const int j = it.halo + g * kTcFrames + fq;
                if (j < it.n) {
                    if (lane < 16) {
                        float4* gr = reinterpret_cast<float4*>(mine + lane * 16);
                        float4* cr = reinterpret_cast<float4*>(mine + 256 + lane * 16);
#pragma unroll
                        for (int c = 0; c < 4; c++) {
                            cr[c] = make_float4(__uint_as_float(v[4 * c]), __uint_as_float(v[4 * c + 1]),
                                                __uint_as_float(v[4 * c + 2]), __uint_as_float(v[4 * c + 3]));
                            gr[c] = make_float4(__uint_as_float(v[16 + 4 * c]), __uint_as_float(v[17 + 4 * c]),
                                                __uint_as_float(v[18 + 4 * c]), __uint_as_float(v[19 + 4 * c]));
                        }
                    }
                    __syncwarp();
                    // contract to 8 numbers per cell, stored [cell][number]: a lane takes four numbers of its cell
#pragma unroll
                    for (int i = 0; i < kSumVals / 32; i++) {
                        const int number = (lane >> 4) + 2 * i;
                        dst[(long long)j * p.NSg * kSumVals + (lane & 15) * 8 + number] =
                            combine_sums(mine_a, lane & 15, number, lg, W2s);
                    }
                    __syncwarp();
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTcCols) : "memory");
    }
    if (timed_out && p.status != nullptr) atomicOr(p.status, kStatusWaitTimeout);
}

}  // namespace sttm
