// Launch interface of the split form of the decode step: one thread-block cluster per unit,
// each CTA of the cluster streaming a slice of the unit's token slots.  For launches with far
// fewer units than SMs (one layer of a batch-1 model), where one CTA per unit would leave most
// of the machine idle.
#pragma once

#include "zsm_decode.cuh"

namespace zsm {

constexpr int kSplitMaxCluster = 8;   // portable cluster size limit
constexpr int kSplitRowBlock = 16;    // slices are cut at multiples of 16 token rows

struct SplitParams {
    DecodeParams d;       // sched_desc: the launch's units in plain order; sched_off unused;
                          // l_stride: weight entries one CTA can hold (split_l_stride)
    int32_t n_units;      // clusters in the launch
    int32_t kr_rows;      // merged key rows rank 0 can keep in shared memory (0: none)
    int32_t early;        // 1: the kernel that precedes this launch in its stream does not write
                          // these units' cache, so their counters and first tiles may be read
                          // while that kernel is still running (programmatic dependent launch)
};

// Token rows [lo, hi) of rank c of C.  Rank 0 also carries the merged rows (fp32 masters, so one
// of them weighs 4 / elem_size token rows) and takes that many fewer token rows.
__host__ __device__ inline void split_slice(int n_live, int n_res, int elem_size, int C, int c,
                                            int &lo, int &hi) {
    const int nb = (n_live + kSplitRowBlock - 1) / kSplitRowBlock;
    if (C <= 1) {
        lo = 0;
        hi = n_live;
        return;
    }
    const int eb = (n_res * (4 / elem_size) + kSplitRowBlock - 1) / kSplitRowBlock;
    const int sh = (nb + eb + C - 1) / C;
    int b0 = sh - eb;
    b0 = b0 < 0 ? 0 : (b0 > nb ? nb : b0);
    int blo, bhi;
    if (c == 0) {
        blo = 0;
        bhi = b0;
    } else {
        const int shr = (nb - b0 + C - 2) / (C - 1);
        blo = b0 + (c - 1) * shr;
        blo = blo > nb ? nb : blo;
        bhi = blo + shr;
        bhi = bhi > nb ? nb : bhi;
    }
    lo = blo * kSplitRowBlock;
    hi = bhi * kSplitRowBlock;
    hi = hi > n_live ? n_live : hi;
    lo = lo > hi ? hi : lo;
}

// Weight entries a CTA must be able to hold: its largest possible slice, the merged slots and
// the new token (both on rank 0), rounded up to 4.
__host__ __device__ inline int split_l_stride(int cap_max, int br_max, int elem_size, int C) {
    const int nb = (cap_max + kSplitRowBlock - 1) / kSplitRowBlock;
    const int eb = (br_max * (4 / elem_size) + kSplitRowBlock - 1) / kSplitRowBlock;
    const int sh = C <= 1 ? nb : (nb + eb + C - 1) / C;
    return (sh * kSplitRowBlock + br_max + 1 + 3) & ~3;
}

// Shared-memory map of one CTA of the split form (byte offsets).
struct SplitSmem {
    uint32_t ring, bars, flags, hdr, meta, probs, qf, krs, opart, redf, xs, xv, xo, total;
};

// Bytes of the header a CTA receives after the launch's inputs are known to be ready: q (G rows),
// k_new, v_new in the storage dtype, then the unit's fusion counts.
__host__ __device__ inline uint32_t split_header_bytes(int G, int row_bytes, int br_max_pad) {
    return static_cast<uint32_t>((G + 2) * row_bytes + br_max_pad * 4);
}

__host__ __device__ inline SplitSmem split_smem_layout(int stages, int G, int D, int row_bytes,
                                                       int l_stride, int br_max_pad, int kr_rows,
                                                       int consumer_warps, int cluster) {
    SplitSmem L;
    uint32_t o = 0;
    auto take = [&](uint32_t bytes) {
        uint32_t at = o;
        o += (bytes + 127u) & ~127u;
        return at;
    };
    L.ring = take(static_cast<uint32_t>(stages) * kTileBytes);
    L.bars = take((2u * static_cast<uint32_t>(stages) + 6u) * 8u);
    L.flags = take(64u);
    L.hdr = take(split_header_bytes(G, row_bytes, br_max_pad));
    L.meta = take(static_cast<uint32_t>(l_stride) * 8u);  // the slice's scores, then its positions
    L.probs = take(static_cast<uint32_t>(G) * l_stride * 4u);
    L.qf = take(static_cast<uint32_t>(G) * D * 4u);
    L.krs = take(static_cast<uint32_t>(kr_rows) * D * 4u);
    L.opart = take(static_cast<uint32_t>(consumer_warps) * G * D * 4u);
    L.redf = take(2u * kMaxConsumerWarps * 8u * 4u);
    L.xs = take(kSplitMaxCluster * 2u * 8u * 4u);                       // (max, sum) per rank and head
    L.xv = take(kSplitMaxCluster * 16u);                                // victim candidate per rank
    L.xo = take(static_cast<uint32_t>(cluster) * G * D * 4u);           // partial outputs per rank
    L.total = o;
    return L;
}

// dtype: 0 fp32, 1 fp16, 2 bf16.  Returns a cudaError_t as int; -1: no kernel for the shape.
int launch_decode_split(int dtype, int D, int G, const SplitParams &p, int cluster,
                        int consumer_warps, cudaStream_t stream);
// Raises the kernel's dynamic shared-memory limit; returns a cudaError_t as int (-1: no kernel)
// and how many clusters of this size and footprint the device can hold at once (0: none).
int prepare_decode_split(int dtype, int D, int G, int cluster, int smem_bytes, int threads,
                         int *max_clusters);

}  // namespace zsm
