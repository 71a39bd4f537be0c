// Launch interface of the fused decode-step kernel.
#pragma once

#include "zsm_common.cuh"

namespace zsm {

constexpr int kTileBytes = 16384;     // one ring stage
constexpr int kMaxConsumerWarps = 16;  // wide form (one CTA per SM); + 1 producer + 1 tail warp
constexpr int kPairConsumerWarps = 8;  // two CTAs per SM
constexpr int kExtraWarps = 2;
constexpr int kMailFixed = 128;       // bytes of a mailbox before its key, value and count arrays

struct DecodeParams {
    uint8_t *base;               // cache buffer
    const int32_t *sched_off;    // [grid + 1] first schedule entry of each CTA
    const UnitDesc *sched_desc;  // unit descriptors in CTA order
    UnitCounters *counters;      // [n_units]
    int32_t *status;             // sticky device status
    const void *q;               // [units][G][d]
    const void *k_new;           // [units][d]
    const void *v_new;           // [units][d]
    void *out;                   // [units][G][d]
    int32_t *victim_pos;         // [units] or null
    int32_t *merge_slot;         // [units] or null
    int32_t unit_base;           // global index of the tensors' first unit
    int32_t stages;              // ring depth
    int32_t l_stride;            // floats per query head in the weight array
    int32_t br_max_pad;          // largest B_r, rounded up to 4
    int32_t cosine;              // slot similarity of Eq. (hatr): 0 raw dot product, 1 cosine
    float lambda, alpha, scale;
};

// Shared-memory map of one CTA (byte offsets), computed the same way on host and device.
struct DecodeSmem {
    uint32_t ring, bars, flags, probs, qf, mail, opart, redf, red64, total;
    uint32_t mail_stride;
};

// A mailbox hands one unit's cache update (residual fill/merge, insertion, counters) from the
// consumer warps to the tail warp; two of them, used alternately.
__host__ __device__ inline uint32_t decode_mail_bytes(int row_bytes, int br_max_pad) {
    const uint32_t b = kMailFixed + 2u * row_bytes + static_cast<uint32_t>(br_max_pad > 0 ? br_max_pad : 4) * 4u;
    return (b + 127u) & ~127u;
}

__host__ __device__ inline DecodeSmem decode_smem_layout(int stages, int G, int D, int row_bytes,
                                                         int l_stride, int br_max_pad,
                                                         int consumer_warps) {
    DecodeSmem L;
    uint32_t o = 0;
    auto take = [&](uint32_t bytes) {
        uint32_t at = o;
        o += (bytes + 127u) & ~127u;
        return at;
    };
    L.ring = take(static_cast<uint32_t>(stages) * kTileBytes);
    L.bars = take((2u * static_cast<uint32_t>(stages) + 6u) * 8u);
    L.flags = take(64u);
    // the warps' partial outputs are folded where the weights were (the weights are dead once the
    // output pass is over): one region, sized for the larger of the two
    const uint32_t probs_bytes = static_cast<uint32_t>(G) * l_stride * 4u;
    const uint32_t opart_bytes = static_cast<uint32_t>(consumer_warps) * G * D * 4u;
    L.probs = take(probs_bytes > opart_bytes ? probs_bytes : opart_bytes);
    L.qf = take(static_cast<uint32_t>(G) * D * 4u);
    L.mail_stride = decode_mail_bytes(row_bytes, br_max_pad);
    L.mail = take(2u * L.mail_stride);
    L.opart = L.probs;
    L.redf = take(2u * kMaxConsumerWarps * 8u * 4u);
    L.red64 = take(kMaxConsumerWarps * 16u);
    L.total = o;
    return L;
}

// dtype: 0 fp32, 1 fp16, 2 bf16.  Returns a cudaError_t as int; -1: no kernel for the shape.
int launch_decode_fused(int dtype, int D, int G, const DecodeParams &p, int grid,
                        int consumer_warps, bool wide, cudaStream_t stream);
// Sets the dynamic shared-memory limit of the matching kernel; returns a cudaError_t as int
// (-1: no kernel) and the CTAs per SM the occupancy calculator allows.
int prepare_decode_fused(int dtype, int D, int G, int smem_bytes, int threads,
                         int *max_ctas_per_sm);

// One CTA, one thread, waiting with the library's bounded wait on a barrier nothing arrives at;
// gives up after limit_us and records DEV_ERR_TIMEOUT in *status.  Returns a cudaError_t as int.
int launch_wait_selftest(int32_t *status, uint32_t limit_us, cudaStream_t stream);

}  // namespace zsm
