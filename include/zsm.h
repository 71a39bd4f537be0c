/*
 * zsm.h -- C ABI of the B200 (sm_100a) compressed-KV decode path of ZSMerge.
 *
 * What the library computes (paper sections in brackets):
 *   - a per-head budgeted KV cache of B = B_p + B_c + B_r slots: the latest B_p
 *     tokens, the B_c highest-scoring older tokens and B_r merged slots [Sec. 3.2];
 *   - per decode step, for every (layer, sequence, kv-head): compensated attention
 *     over the slots plus the new token [Eq. (att_score2), Sec. 3.5], the score
 *     update s <- lambda*s + a_hat [Eq. (score), Sec. 3.3], eviction of the lowest
 *     (score, position) token that is no longer among the B_p latest [Alg. 1
 *     l.7-11], its fill-or-merge into the residual slots [Eq. (hatr), (kvr), Sec.
 *     3.4; Alg. 1 l.12-16] and the insertion of the new token [Alg. 1 l.6] -- one
 *     fused kernel launch;
 *   - the one-shot compression of a prompt's K/V into the budgets after prefill
 *     [App. B for the score window; the procedure itself is this library's reading:
 *     latest B_p kept, top-B_c of the rest by score kept, the remainder merged in
 *     ascending position by the same fill-or-merge rule].
 *
 * Conventions
 *   - Every function returns a zsm_status_t; nothing throws, aborts or prints.
 *   - "dev" pointers are CUDA device pointers of the current device, owned by the
 *     caller; "host" pointers are ordinary host memory.  The library never
 *     allocates device memory: the cache lives in a caller-supplied buffer, scratch
 *     for the prompt pass in a caller-supplied workspace.
 *   - Launches are asynchronous on the given stream (a cudaStream_t passed as an
 *     opaque pointer; NULL is the default stream) unless stated otherwise.
 *   - Arguments are validated on the host before any launch.  Checks that can
 *     only be made on the device set a sticky status word read back by
 *     zsm_last_device_status(); device code never traps.  Every wait inside a
 *     kernel is bounded and reports ZSM_ERR_TIMEOUT instead of hanging.
 *   - Tensors are dense, row-major, innermost dimension head_dim, in the cache's
 *     storage dtype unless a type is written out.  16-byte alignment is required
 *     for every dev tensor pointer.
 *   - A unit is one (layer, sequence b, kv-head h); units never interact.
 *     Positions are 0-based.  Query head g of kv-head h is q head h*G + g,
 *     G = n_q_heads / n_kv_heads; grouped heads share one K/V read and their
 *     attention weights are averaged for the score [App. C.4].
 *   - Merged (residual) slots are held in fp32 whatever the storage dtype, so
 *     thousands of incremental means do not stall at half precision.
 *   - Contribution scores [Eq. (score)] are fp32 and ordered as floats of either sign
 *     (the method itself only produces non-negative ones; -0.0 equals +0.0); equal
 *     scores are ordered by position.  NaN is not a score: zsm_cache_import_unit
 *     refuses it (ZSM_ERR_INVALID_ARG) and the prompt pass reports it through the
 *     sticky status word (ZSM_ERR_DEVICE_CHECK).
 *   - A handle is not thread-safe: calls on one handle come from one thread at a time.
 */
#ifndef ZSM_H
#define ZSM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ZSM_OK = 0,
    ZSM_ERR_INVALID_ARG = 1,      /* null / negative / inconsistent argument */
    ZSM_ERR_BUFFER_TOO_SMALL = 2, /* caller's cache buffer or workspace is too small */
    ZSM_ERR_STATE = 3,            /* call not valid in the handle's state */
    ZSM_ERR_CUDA = 4,             /* a CUDA runtime call failed */
    ZSM_ERR_UNSUPPORTED = 5,      /* shape outside what the kernels are built for */
    ZSM_ERR_DEVICE_CHECK = 6,     /* a device-side consistency check failed */
    ZSM_ERR_TIMEOUT = 7,          /* a bounded device-side wait gave up */
    ZSM_ERR_NO_MEMORY = 8         /* host memory for the handle could not be allocated */
} zsm_status_t;

typedef enum { ZSM_F32 = 0, ZSM_F16 = 1, ZSM_BF16 = 2 } zsm_dtype_t;

typedef void *zsm_stream_t; /* cudaStream_t */

typedef struct zsm_cache zsm_cache_t; /* host-side handle; owns no device memory */

typedef struct {
    int32_t n_layers;
    int32_t batch;      /* sequences */
    int32_t n_q_heads;  /* multiple of n_kv_heads; group size 1, 2, 4 or 8 */
    int32_t n_kv_heads;
    int32_t head_dim;   /* 64 or 128 */
    int32_t dtype;      /* zsm_dtype_t: storage of q, k, v, out and token slots */
    /* Per-head budgets, host arrays of n_layers*n_kv_heads int32 (layer-major),
     * read during zsm_cache_create only.  B_p + B_c >= 1, B_r >= 0 [Sec. 3.2]. */
    const int32_t *budget_p;
    const int32_t *budget_c;
    const int32_t *budget_r;
    float lambda;        /* score decay, 0.98 in the paper [Sec. 3.3] */
    float alpha;         /* compensation strength, 1.0 in the paper [Sec. 3.5] */
    float softmax_scale; /* 0 selects 1/sqrt(head_dim) [Eq. (att_score)] */
    /* Launch tuning of the fused decode kernel; 0 selects the library default. */
    int32_t tune_stages;         /* 16 KiB ring stages per CTA */
    int32_t tune_ctas_per_sm;    /* persistent CTAs per SM (default: 2, or 1 for a launch with no
                                  * more units than SMs) */
    int32_t tune_consumer_warps; /* compute warps per CTA: at most 8 with two CTAs per SM, 16 with
                                  * one (two more warps feed them
                                  * and write the cache update back) */
    int32_t tune_split;          /* CTAs that share one unit in a launch with few units (each takes
                                  * a slice of the unit's slots; a thread-block cluster): 0 = the
                                  * library's choice (the largest of 8, 4, 2 that keeps the launch
                                  * within the SM count, when units are at most half the SMs),
                                  * 1 = never split, 2, 4 or 8 = at most that many */
    int32_t similarity;          /* how an evicted token picks its merged slot [Eq. (hatr)]:
                                  * 0 = raw dot product k_r.k_t, as the paper prints it;
                                  * 1 = cosine k_r.k_t / (|k_r||k_t|), the form the paper's source
                                  * carries commented out beside it (a zero vector is similar to
                                  * nothing).  With 1 the prompt pass runs its general merge
                                  * kernel, whatever B_r is. */
} zsm_config_t;

/* Budget split of App. C.2: B_p = floor(tail_ratio*B); B_r = round(dense_ratio*
 * (B-B_p)), at least 1 when dense_ratio > 0; B_c the rest.  Recommended ratios:
 * 0.5 and 0.02.  Host only.  INVALID_ARG for B < 1 or ratios outside [0,1]. */
zsm_status_t zsm_split_budget(int32_t B, float tail_ratio, float dense_ratio, int32_t *Bp,
                              int32_t *Bc, int32_t *Br);

/* Bytes of device memory a cache of this configuration needs. */
zsm_status_t zsm_cache_bytes(const zsm_config_t *cfg, size_t *bytes);

/* Lay the cache out in dev_buf (256-byte aligned, >= zsm_cache_bytes) and
 * return a handle.  Writes the layout tables and empties every unit; blocks
 * until that is done.  The handle keeps dev_buf but never frees it.  Also does
 * the per-device set-up of zsm_prefill_compress_static (see there).
 * UNSUPPORTED: head_dim, group size or a budget the kernels cannot hold in
 * shared memory.  NO_MEMORY: the host handle could not be allocated. */
zsm_status_t zsm_cache_create(const zsm_config_t *cfg, void *dev_buf, size_t bytes,
                              zsm_cache_t **out);

/* Empty every unit (occupancy 0, next position 0); asynchronous. */
zsm_status_t zsm_cache_reset(zsm_cache_t *c, zsm_stream_t stream);

/* Release the host handle.  dev_buf stays with the caller. */
zsm_status_t zsm_cache_free(zsm_cache_t *c);

/* Workspace bytes zsm_prefill_compress needs for a T-token prompt scored with
 * its last W queries (W = 0 when scores are supplied). */
zsm_status_t zsm_prefill_workspace_bytes(const zsm_cache_t *c, int32_t T, int32_t W,
                                         size_t *bytes);

/* One-shot compression of one layer's prompt K/V into that layer's units,
 * replacing their contents; afterwards the next position of each unit is T.
 *   K, V     dev [batch][n_kv_heads][T][head_dim]
 *   Qw       dev [batch][n_q_heads][W][head_dim], the prompt's last W queries
 *            (1 <= W <= T): each attends causally to keys 0..its own position and
 *            the rows are combined by Eq. (score) unrolled (weight lambda^(T-1-tau)
 *            for query position tau), averaged over a group.  NULL to use `scores`.
 *   scores   dev fp32 [batch][n_kv_heads][T], used iff Qw is NULL
 *   workspace dev, >= zsm_prefill_workspace_bytes, 256-byte aligned
 * Layers are independent: calls for different layers may run at the same time on different
 * streams, each with a workspace of its own (the sequential merge chain of one layer keeps
 * only one CTA per unit busy, so several layers in flight use the machine far better).
 * Optional dev outputs for inspection (NULL to skip), each [batch][n_kv_heads][T]:
 *   dbg_scores  fp32 score of every prompt position
 *   dbg_evicted uint8, 1 where the position was evicted (merged or dropped)
 *   dbg_targets int32, for the i-th evicted position in ascending order the
 *               residual slot it went to (-2: took a free slot, -1: dropped, B_r=0)
 */
zsm_status_t zsm_prefill_compress(zsm_cache_t *c, int32_t layer, const void *K, const void *V,
                                  const void *Qw, const float *scores, int32_t T, int32_t W,
                                  void *workspace, size_t workspace_bytes, float *dbg_scores,
                                  uint8_t *dbg_evicted, int32_t *dbg_targets,
                                  zsm_stream_t stream);

/* zsm_prefill_compress for callers that cannot allocate device memory when they call
 * (the paper has no counterpart; this is a convenience of the library).  Typical cases: a
 * serving process whose own memory pool has already reserved the whole GPU, so that a
 * cudaMalloc made now would fail, or a latency-critical loop that cannot afford the device
 * synchronisation an allocation may imply.  Arguments, results and status codes are those of
 * zsm_prefill_compress without `workspace`: the scratch is a fixed array of
 * ZSM_STATIC_SCRATCH_BYTES that is part of the library image -- every GPU on which a cache
 * has been created holds those bytes until the process exits -- and the call makes no
 * cudaMalloc, cudaFree or other allocating call.
 *   - ZSM_ERR_BUFFER_TOO_SMALL when the prompt needs more scratch than that
 *     (zsm_prefill_workspace_bytes(c, T, W) tells how much; roughly
 *     batch*n_kv_heads*T*(13 + 4*G*W) bytes).  Nothing is launched then.
 *   - Set-up: the array's device address is looked up once per device, and that first look-up
 *     is also when the device loads the part of the library that holds the array, i.e. when
 *     the bytes are reserved.  zsm_cache_create does it (a handle is needed for this call
 *     anyway, so the set-up has always happened on the handle's device); from then on this
 *     call neither allocates nor synchronises.  Create the cache outside any stream capture.
 *   - All calls on a device share the one array, which keeps what the last call left in
 *     it.  The pass overwrites every entry before it reads it, so nothing needs clearing;
 *     but two calls whose kernels overlap on the GPU (different streams) race on it.
 *     Calls on one stream are ordered and safe. */
#define ZSM_STATIC_SCRATCH_BYTES (16u << 20)
zsm_status_t zsm_prefill_compress_static(zsm_cache_t *c, int32_t layer, const void *K,
                                         const void *V, const void *Qw, const float *scores,
                                         int32_t T, int32_t W, float *dbg_scores,
                                         uint8_t *dbg_evicted, int32_t *dbg_targets,
                                         zsm_stream_t stream);

/* Full-history prompt scores: the scoring window of App. B taken as the whole prompt, i.e.
 * Eq. (score) unrolled over every prompt query,
 *   scores[b][h][t] = (1/G) sum_g sum_{tau = t}^{T-1} lambda^(T-1-tau) * a^(tau)_{g,t},
 * with a^(tau) the causal softmax row of query tau [Eq. (att_score)] and the mean over the G
 * query heads of kv head h [App. C.4].  A dense T x T x d contraction on the tensor cores, two
 * passes: the log-sum-exp of every query's row, then the decayed column sums.  The result is
 * what zsm_prefill_compress takes as `scores` (with Qw == NULL), for any layer of the cache.
 *   K       dev [batch][n_kv_heads][T][head_dim], Q dev [batch][n_q_heads][T][head_dim],
 *           storage dtype of the cache, 16-byte aligned; fp16 or bf16 only
 *           (ZSM_ERR_UNSUPPORTED for fp32 storage: use the window form with W = T there).
 *   lse     dev fp32 [batch][n_q_heads][T] or NULL: natural-log sum-exp of each query's scaled
 *           causal logits, as a prefill attention kernel returns it; when given, the first
 *           pass is skipped and `workspace` may be NULL.
 *   scores  dev fp32 [batch][n_kv_heads][T], written.
 *   workspace  dev, 256-byte aligned, zsm_prefill_scores_full_workspace_bytes(c, T) bytes
 *           (the row statistics); caller-owned, free to reuse once the stream has passed.
 * Errors: ZSM_ERR_INVALID_ARG (null or misaligned pointers, T < 1), ZSM_ERR_BUFFER_TOO_SMALL,
 * ZSM_ERR_UNSUPPORTED, ZSM_ERR_CUDA.  Asynchronous on `stream`; nothing is allocated. */
zsm_status_t zsm_prefill_scores_full_workspace_bytes(const zsm_cache_t *c, int32_t T,
                                                     size_t *bytes);
zsm_status_t zsm_prefill_scores_full(zsm_cache_t *c, const void *K, const void *Q,
                                     const float *lse, int32_t T, float *scores,
                                     void *workspace, size_t workspace_bytes,
                                     zsm_stream_t stream);

/* Causal prefill attention of one layer's prompt with the compression's inputs as by-products
 * [Eq. (att_score) for every prompt query; App. B: the scores come from the prefill's attention
 * history]: out[b][hq][tau] = sum_{t <= tau} a^(tau)_t v_t, the rows' log-sum-exp, and -- when
 * `scores` is given -- the full-history scores of zsm_prefill_scores_full, ready for
 * zsm_prefill_compress(scores = ...).  A model that runs this as its prefill attention needs no
 * separate scoring pass.  Tensor cores throughout (tcgen05): one pass for the output and the
 * rows' log-sum-exp (two products per key tile: Q K^T; 16-bit weights of a running softmax times
 * V), then, if asked for, the decayed column sums.
 *   K, V    dev [batch][n_kv_heads][T][head_dim];  Q dev [batch][n_q_heads][T][head_dim];
 *           storage dtype of the cache (fp16 or bf16; ZSM_ERR_UNSUPPORTED for fp32), 16-byte aligned
 *   out     dev [batch][n_q_heads][T][head_dim], storage dtype, written
 *   lse     dev fp32 [batch][n_q_heads][T], written (natural log of each row's sum of exponentials)
 *   scores  dev fp32 [batch][n_kv_heads][T], written, or NULL
 * Asynchronous on `stream`; nothing is allocated. */
zsm_status_t zsm_prefill_attention(zsm_cache_t *c, const void *K, const void *V, const void *Q,
                                   int32_t T, void *out, float *lse, float *scores,
                                   zsm_stream_t stream);

/* One decode step [Algorithm 1 with Eq. (att_score2)], one kernel launch.
 *   layer      0..n_layers-1: that layer's units; tensors have no layer dimension.
 *              -1: every layer in one launch; tensors carry a leading
 *              [n_layers] dimension.
 *   q          dev [batch][n_q_heads][head_dim]
 *   k_new,v_new dev [batch][n_kv_heads][head_dim]
 *   out        dev [batch][n_q_heads][head_dim]: attention output over the cache
 *              as it stood plus the new token
 *   victim_pos dev int32 [batch][n_kv_heads] or NULL: evicted position, -1 none
 *   merge_slot dev int32 [batch][n_kv_heads] or NULL: residual slot merged into;
 *              -2 took a free slot; -1 none
 * The cache is updated in place.  Decoding into an empty cache is legal: it
 * fills first, then starts evicting. */
zsm_status_t zsm_decode_step(zsm_cache_t *c, int32_t layer, const void *q, const void *k_new,
                             const void *v_new, void *out, int32_t *victim_pos,
                             int32_t *merge_slot, zsm_stream_t stream);

/* The same step for callers whose tensors live in HOST memory (pinned for
 * speed): copies q, k_new, v_new to `staging`, runs the step, copies out back
 * and waits for the stream.  staging: dev scratch of at least
 * zsm_decode_staging_bytes(). */
zsm_status_t zsm_decode_staging_bytes(const zsm_cache_t *c, int32_t layer, size_t *bytes);
zsm_status_t zsm_decode_step_host(zsm_cache_t *c, int32_t layer, const void *q_host,
                                  const void *k_new_host, const void *v_new_host,
                                  void *out_host, void *staging, size_t staging_bytes,
                                  zsm_stream_t stream);

/* The host-buffer step pipelined over two staging halves, for callers that stream steps: the
 * call only enqueues -- one copy in on an internal copy stream, the step on `stream`, one copy
 * out on a second internal copy stream, tied together by events -- and returns; step i+1's
 * copy in and step i's copy out then run under the other step's kernel.  Steps stay ordered
 * (they update one cache) because all of them run on `stream`.
 *   in_host    pinned host buffer holding q, k_new and v_new at the offsets
 *              zsm_decode_host_layout gives (in_bytes long; one copy moves it)
 *   out_host   pinned host buffer of out_bytes; valid after zsm_decode_step_host_wait(slot)
 *   staging    dev scratch, 256-byte aligned, >= 2 * (in_bytes + out_bytes rounded up to 256)
 *   slot       0 or 1: which staging half (and which set of events) this step uses; alternate
 *              them, and call zsm_decode_step_host_wait(slot) before reusing a slot's host
 *              buffers.  At most one step per slot is in flight.
 * The first call creates two streams and six events (no device memory) that live until
 * zsm_cache_free; make it outside any stream capture.  wait: ZSM_ERR_STATE if the slot was
 * never used. */
zsm_status_t zsm_decode_host_layout(const zsm_cache_t *c, int32_t layer, size_t *q_off,
                                    size_t *k_off, size_t *v_off, size_t *in_bytes,
                                    size_t *out_bytes);
zsm_status_t zsm_decode_step_host_async(zsm_cache_t *c, int32_t layer, const void *in_host,
                                        void *out_host, void *staging, size_t staging_bytes,
                                        int32_t slot, zsm_stream_t stream);
zsm_status_t zsm_decode_step_host_wait(zsm_cache_t *c, int32_t slot);

/* Decode attention over an UNCOMPRESSED cache [Eq. (att_score), Sec. 3.1]: what the paper's
 * FullKV baseline computes per step, for the cache path only -- the same-hardware comparator of
 * zsm_decode_step (Sec. 4.2 compares the two end to end).  No cache handle: the caller owns K and V.
 *   dtype      ZSM_F16 or ZSM_BF16 (UNSUPPORTED for ZSM_F32)
 *   n_units    (layers x sequences x kv heads) handled by the call; group = query heads per kv
 *              head (1, 2, 4, 8); head_dim 64 or 128; T tokens per unit, all attended
 *   K, V       dev [n_units][T][head_dim];  q, out  dev [n_units][group][head_dim]
 *   workspace  dev, 256-byte aligned, >= zsm_fullkv_workspace_bytes: per-chunk partial results
 *              and a status word; contents need not survive between calls
 * Asynchronous on `stream` (two kernels).  zsm_fullkv_status waits for the stream and returns
 * the device status of the most recent call on that workspace (ZSM_ERR_TIMEOUT if a bounded
 * wait inside the kernel gave up). */
zsm_status_t zsm_fullkv_workspace_bytes(int32_t n_units, int32_t group, int32_t head_dim, int32_t T,
                                        size_t *bytes);
zsm_status_t zsm_fullkv_decode(int32_t dtype, int32_t n_units, int32_t group, int32_t head_dim,
                               int32_t T, const void *K, const void *V, const void *q, void *out,
                               float softmax_scale, void *workspace, size_t workspace_bytes,
                               zsm_stream_t stream);
zsm_status_t zsm_fullkv_status(void *workspace, zsm_stream_t stream);

/* Slot capacities of unit (layer, h): token slots B_p + B_c and residual slots. */
zsm_status_t zsm_unit_capacity(const zsm_cache_t *c, int32_t layer, int32_t h,
                               int32_t *n_token_slots, int32_t *n_residual_slots);

/* Copy one unit's state to HOST arrays (any may be NULL); blocks on `stream`.
 *   K, V     fp32 [n_token_slots][head_dim] (storage values widened), live rows first
 *   score    fp32 [n_token_slots];  pos int32 [n_token_slots]
 *   Kr, Vr   fp32 [n_residual_slots][head_dim];  w uint32 [n_residual_slots]
 *   counters int32[3]: live token slots, used residual slots, next position */
zsm_status_t zsm_cache_export_unit(zsm_cache_t *c, int32_t layer, int32_t b, int32_t h,
                                   float *K, float *V, float *score, int32_t *pos, float *Kr,
                                   float *Vr, uint32_t *w, int32_t *counters,
                                   zsm_stream_t stream);

/* Inverse of export (resume / checkpoint restore): all arrays required, K and V
 * are rounded to the storage dtype.  INVALID_ARG if counters exceed capacity or a
 * live slot's score is NaN. */
zsm_status_t zsm_cache_import_unit(zsm_cache_t *c, int32_t layer, int32_t b, int32_t h,
                                   const float *K, const float *V, const float *score,
                                   const int32_t *pos, const float *Kr, const float *Vr,
                                   const uint32_t *w, const int32_t *counters,
                                   zsm_stream_t stream);

/* Waits for `stream`, then returns the sticky device status (ZSM_OK if no
 * device-side check or wait has failed since creation or the last call) and
 * clears it. */
zsm_status_t zsm_last_device_status(zsm_cache_t *c, zsm_stream_t stream);

/* Exercises the device-side failure detector without a fault: launches one CTA whose single
 * thread waits, with the same bounded wait every kernel of the library uses, on a barrier that
 * nothing ever arrives at.  After limit_us microseconds (1..1 000 000) the wait gives up, the
 * kernel records ZSM_ERR_TIMEOUT in the cache's sticky status word and returns normally; the
 * context stays usable.  Asynchronous; read the outcome with zsm_last_device_status. */
zsm_status_t zsm_selftest_wait_timeout(zsm_cache_t *c, uint32_t limit_us, zsm_stream_t stream);

/* Launch shape of the fused decode kernel for this layer argument (diagnostics). */
zsm_status_t zsm_decode_launch_info(const zsm_cache_t *c, int32_t layer, int32_t *grid,
                                    int32_t *block, int32_t *dynamic_smem_bytes);

const char *zsm_status_string(zsm_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* ZSM_H */
