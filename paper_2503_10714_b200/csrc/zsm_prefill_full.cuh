// Launch interface of the full-history prompt scoring (every prompt query scores every earlier
// key: the W = T case of App. B, Eq. (score) unrolled over the whole prompt).
#pragma once

#include "zsm_common.cuh"

namespace zsm {


struct FullScoreParams {
    const void *K;      // [batch][n_kv_heads][T][d]
    const void *Q;      // [batch][n_q_heads][T][d]
    const float *lse;   // [batch][n_q_heads][T] natural log-sum-exp of each query's causal row
    float *lse_out;     // same shape, written by the first pass (null when `lse` is supplied)
    float *scores;      // [batch][n_kv_heads][T]
    int32_t *status;    // sticky device status word of the cache
    int32_t batch, n_kv_heads, G, T;
    float lambda, scale;
};

// Enqueues one or both passes on `stream`: row statistics (skipped when p.lse is set), then the
// decayed column sums.  dtype: 1 fp16, 2 bf16.  Returns a cudaError_t as int; -1: no kernel.
int launch_full_scores(int dtype, int D, const FullScoreParams &p, cudaStream_t stream);
// The first pass alone: every query row's log-sum-exp into p.lse_out.
int launch_row_statistics(int dtype, int D, const FullScoreParams &p, cudaStream_t stream);
// Causal attention of the prompt in one pass: out [batch][n_q_heads][T][d] in the storage dtype and
// every query row's log-sum-exp into p.lse_out (required; p.lse is not read); V [batch][n_kv_heads][T][d].
int launch_attention_output(int dtype, int D, const FullScoreParams &p, const void *V, void *out,
                            cudaStream_t stream);
// Window scoring of the prompt pass on tcgen05 (16-bit storage, windows of G*W = 32, 64, 96, 128 rows).
struct WindowLogitsParams {
    const void *K;     // [units][T][d]
    const void *Qw;    // [batch][n_q_heads][W][d]: a unit's G*W rows are consecutive
    float *logits;     // fp32 [units][G*W][T], scaled, causally masked (-inf)
    float2 *partial;   // [units][G*W][chunks of 128 keys]: (max, sum exp) of the chunk
    int32_t *status;
    int32_t units, n_kv_heads, T, W, G;
    float scale;
};
bool window_logits_tc_supported(int GW);
// grid_x persistent CTAs per unit.  Returns a cudaError_t as int; -1: no kernel for this case.
int launch_window_logits_tc(int dtype, int D, const WindowLogitsParams &p, int grid_x, cudaStream_t stream);
// Raises the kernels' dynamic shared-memory limit; returns a cudaError_t as int (-1: no kernel).
int prepare_full_scores(int dtype, int D);

}  // namespace zsm
