/*
 * ZSMerge CPU oracle -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 restatement of the per-head compressed-KV cache of the
 * ZSMerge paper: Algorithm 1 (online compression) with the three lists K_p,
 * K_c, K_r of Sec. 3.2, the contribution score of Eq. (score) in Sec. 3.3, the
 * residual merge of Eq. (hatr)/(kvr) in Sec. 3.4, the compensated attention of
 * Eq. (att_score2) in Sec. 3.5, and a one-shot prompt compression built from
 * the same pieces (App. B gives only the score-window idea; the procedure is a
 * stated reading, see zso_prefill_compress).
 *
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may
 * call this library.  It shares no code with the CUDA path and is never a
 * fallback for it.
 *
 * One zso_unit is one (layer, sequence, kv-head): units never interact.
 * Positions are 0-based.  All vectors are host fp64; inputs that came from a
 * narrower storage type are passed already widened (exactly representable).
 * Scores are rounded to fp32 after every update and compared as fp32.
 *
 * Pins (tests/test_oracle_*.py): full-attention equivalence while nothing is
 * evicted; duplicate-key closed form for merge + compensation; Theorem 1;
 * merge conservation laws; occupancy bounds; brute-force score recomputation;
 * an independently written single-pool formulation; restriction-to-retained
 * equivalence for B_r = 0; naive causal-attention scores for the prompt pass;
 * brute-force sort for the prompt selection; constructed exact ties of the
 * residual arg-max (identical slots, equal products) in both the decode step
 * and the prompt chain; the two ratios of the budget split.
 * Parity unpinned (no published worked example or code to compare with): the
 * order in which the prompt's evicted tokens are merged, the default score
 * window, and the rounding of the budget split helper.
 */
#ifndef ZSM_ORACLE_H
#define ZSM_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct zso_unit zso_unit;

typedef struct {
    int32_t d;      /* head dimension */
    int32_t G;      /* query heads sharing this kv head (1 = MHA) */
    int32_t Bp;     /* proximity budget  (Sec. 3.2) */
    int32_t Bc;     /* context budget    (Sec. 3.2) */
    int32_t Br;     /* residual budget   (Sec. 3.2) */
    double lambda;  /* score decay, Eq. (score) */
    double alpha;   /* compensation strength, Eq. (att_score2) */
    double scale;   /* logit scale, 1/sqrt(d) in Eq. (att_score) */
    int32_t cosine; /* 0: Eq. (hatr) as printed, raw dot product; 1: the cosine form the
                     * paper's source carries commented out beside it,
                     * k_r . k_t / (|k_r| |k_t|) */
} zso_params;

/* Optional guidance for the two integer decisions of a step.  A hinted choice
 * is taken only when it is within `tol` (relative) of the oracle's own best;
 * otherwise the oracle keeps its own choice and reports a mismatch. */
typedef struct {
    int32_t victim_pos;  /* position the other side evicted, or -1: no hint */
    int32_t merge_slot;  /* residual slot the other side merged into, or -1 */
    double tol;
} zso_hint;

typedef struct {
    int32_t victim_pos;        /* evicted position, -1 if none this step */
    int32_t victim_own_pos;    /* oracle's own argmin (== victim_pos unless a hint was taken) */
    int32_t victim_runner_pos; /* runner-up of the argmin, -1 if none */
    double victim_gap;         /* (s_runner - s_best)/s_best, +inf if no runner-up */
    int32_t merge_slot;        /* slot merged into; -2: appended to a free slot; -1: none */
    int32_t merge_own_slot;
    int32_t merge_runner_slot;
    double merge_gap;          /* (dot_best - dot_runner)/max abs-dot, +inf if none */
    int32_t victim_near_tie;   /* 1: hint differed from own choice and was accepted */
    int32_t merge_near_tie;
    int32_t victim_mismatch;   /* 1: hint differed and was NOT acceptable */
    int32_t merge_mismatch;
    int32_t victim_exact_tie;  /* 1: hint differed but fp32 scores were equal (tie-rule breach) */
    int32_t merge_exact_tie;
} zso_step_report;

typedef struct {
    int32_t n_evicted;     /* tokens that left the prompt's candidate set */
    int32_t n_near_tie_sel;   /* hinted evictions accepted although not the oracle's own */
    int32_t n_mismatch_sel;   /* hinted evictions rejected */
    int32_t n_near_tie_merge;
    int32_t n_mismatch_merge;
    double min_merge_gap;
    double sel_gap;        /* (smallest kept score - largest evicted score)/largest evicted */
    int32_t n_exact_tie_merge; /* hinted merge targets that differed from the oracle's own although
                                * the two fp32 dot products were equal (tie-rule breaches) */
} zso_prefill_report;

zso_unit *zso_unit_new(const zso_params *p);
void zso_unit_free(zso_unit *u);

/* One pass of Algorithm 1 for a new token.  q: [G][d]; k_new, v_new: [d];
 * out: [G][d].  hint and rep may be NULL.  Returns 0, or -1 on a bad call. */
int zso_decode_step(zso_unit *u, const double *q, const double *k_new, const double *v_new,
                    double *out, const zso_hint *hint, zso_step_report *rep);

/* One-shot compression of a T-token prompt (replaces the unit's state).
 * K, V: [T][d].  Qw: [G][W][d], the prompt's last W queries, or NULL, in which
 * case scores_in [T] supplies the scores.  hint_evicted: [T] bytes, 1 where the
 * other side evicted that position, or NULL.  hint_targets: [n_evicted] slot
 * chosen by the other side for each evicted token in ascending position (fills
 * included), or NULL.  Outputs (each may be NULL): scores_out [T] fp32,
 * evicted_out [T] bytes, targets_out [T] (first n_evicted used). */
int zso_prefill_compress(zso_unit *u, const double *K, const double *V, const double *Qw,
                         const float *scores_in, int32_t T, int32_t W,
                         const uint8_t *hint_evicted, const int32_t *hint_targets, double tol,
                         float *scores_out, uint8_t *evicted_out, int32_t *targets_out,
                         zso_prefill_report *rep);

/* State inspection. */
void zso_counts(const zso_unit *u, int32_t *np, int32_t *nc, int32_t *nr, int64_t *T);
/* Tokens of K_p then K_c: pos [np+nc], score [np+nc], K and V [np+nc][d]. */
void zso_export_tokens(const zso_unit *u, int32_t *pos, float *score, double *K, double *V);
/* Residual slots: Kr, Vr [nr][d], w [nr]. */
void zso_export_residual(const zso_unit *u, double *Kr, double *Vr, uint32_t *w);
/* Attention weights of the last decode step: returns the entry count n;
 * a: [G][n]; id: [n] with id >= 0 a token position (the new token included)
 * and id = -(r+1) residual slot r.  Pass NULL pointers to query n only. */
int32_t zso_last_attention(const zso_unit *u, double *a, int64_t *id);

/* The same step over n independent units, OpenMP-parallel (timed CPU baseline).
 * q: [n][G][d], k_new/v_new: [n][d], out: [n][G][d].  Returns threads used. */
int zso_decode_step_batch(zso_unit **units, int32_t n, const double *q, const double *k_new,
                          const double *v_new, double *out);

/* Budget split helper of App. C.2 (tail ratio, dense ratio). */
int zso_split_budget(int32_t B, double tail_ratio, double dense_ratio, int32_t *Bp, int32_t *Bc,
                     int32_t *Br);

#ifdef __cplusplus
}
#endif
#endif
