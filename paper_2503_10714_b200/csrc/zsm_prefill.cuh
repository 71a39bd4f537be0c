// Launch interface of the one-shot prompt compression kernels.
#pragma once

#include "zsm_common.cuh"

namespace zsm {

constexpr int kPrefillChunk = 128;  // prompt positions per CTA in the scoring pass

// Workspace map (byte offsets into the caller's workspace), same on host and device side.
struct PrefillWorkspace {
    size_t scores;     // fp32 [units][T]           (unused when the caller supplies scores)
    size_t logits;     // fp32 [units][G*W][T]      scaled, causally masked q.k
    size_t partial;    // float2 [units][G*W][chunks]  per-chunk (max, sum exp)
    size_t rowstat;    // float2 [units][G*W]       (row max, weight of the row / its sum)
    size_t flags;      // uint8 [units][T]          1 = evicted
    size_t evict_list; // int32 [units][T]          evicted positions, ascending
    size_t kept_list;  // int32 [units][T]          surviving positions, ascending
    size_t counts;     // int32 [units][4]          n_evicted, n_kept
    size_t total;
};

inline PrefillWorkspace prefill_workspace_layout(int units, int T, int GW) {
    PrefillWorkspace w;
    size_t o = 0;
    auto take = [&](size_t bytes) {
        size_t at = o;
        o += (bytes + 255) & ~static_cast<size_t>(255);
        return at;
    };
    const size_t chunks = (static_cast<size_t>(T) + kPrefillChunk - 1) / kPrefillChunk;
    w.scores = take(static_cast<size_t>(units) * T * 4);
    w.logits = take(static_cast<size_t>(units) * GW * T * 4);
    w.partial = take(static_cast<size_t>(units) * GW * chunks * 8);
    w.rowstat = take(static_cast<size_t>(units) * GW * 8);
    w.flags = take(static_cast<size_t>(units) * T);
    w.evict_list = take(static_cast<size_t>(units) * T * 4);
    w.kept_list = take(static_cast<size_t>(units) * T * 4);
    w.counts = take(static_cast<size_t>(units) * 16);
    w.total = o;
    return w;
}

struct PrefillParams {
    uint8_t *base;             // cache buffer
    const UnitDesc *desc;      // descriptors of this layer's units, [units] in (b, h) order
    UnitCounters *counters;    // [all units]
    int32_t *status;
    const void *K, *V;         // [units][T][d]
    const void *Qw;            // [batch][n_q_heads][W][d] or null
    const float *scores_in;    // [units][T] or null
    uint8_t *ws;               // workspace
    PrefillWorkspace wl;
    float *dbg_scores;         // [units][T] or null
    uint8_t *dbg_evicted;      // [units][T] or null
    int32_t *dbg_targets;      // [units][T] or null
    int32_t units, T, W, G, n_kv_heads;
    int32_t n_sm;              // SMs of the device (picks the form of the merge kernel)
    int32_t max_cap;           // largest B_p + B_c among these units
    int32_t cosine;            // slot similarity of Eq. (hatr): 0 raw dot product, 1 cosine
    float lambda, scale;
};

// Largest B_r the merge kernel can hold in shared memory for this head dimension.
int prefill_max_residual(int D);

// Enqueues the whole pass on `stream`.  Returns a cudaError_t as int; -1: no kernel.
int launch_prefill(int dtype, int D, const PrefillParams &p, int max_br, cudaStream_t stream);
int prepare_prefill(int dtype, int D);

}  // namespace zsm
