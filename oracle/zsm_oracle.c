/*
 * ZSMerge CPU oracle -- TEST INFRASTRUCTURE (see zsm_oracle.h).
 *
 * Written from the paper's text: three explicit lists per unit, fp64 arithmetic,
 * no blocking, no fusion, no reordering beyond what Algorithm 1 states.
 */
#include "zsm_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* A token held in K_p or K_c: its key/value rows, its contribution score
 * (fp32, Eq. (score)) and its position in the sequence. */
typedef struct {
    double *kv; /* k = kv[0..d), v = kv[d..2d) */
    float s;
    int32_t pos;
} zso_tok;

struct zso_unit {
    zso_params p;
    zso_tok *P; /* proximity list, oldest first (FIFO) */
    int32_t np;
    zso_tok *C; /* context list, no particular order */
    int32_t nc;
    double *Kr, *Vr; /* residual slots [Br][d] */
    uint32_t *w;     /* fusion counts */
    int32_t nr;
    int64_t T; /* tokens seen so far = position of the next token */
    /* attention weights of the last step, for the tests */
    double *last_a;
    int64_t *last_id;
    int32_t last_n;
    int32_t last_cap;
};

static double dotd(const double *a, const double *b, int d) {
    double acc = 0.0;
    for (int i = 0; i < d; ++i) acc += a[i] * b[i];
    return acc;
}

zso_unit *zso_unit_new(const zso_params *p) {
    if (!p || p->d <= 0 || p->G <= 0 || p->Bp < 0 || p->Bc < 0 || p->Br < 0) return NULL;
    if (p->Bp + p->Bc < 1) return NULL;
    zso_unit *u = (zso_unit *)calloc(1, sizeof(zso_unit));
    if (!u) return NULL;
    u->p = *p;
    u->P = (zso_tok *)calloc((size_t)p->Bp + 2, sizeof(zso_tok));
    u->C = (zso_tok *)calloc((size_t)p->Bc + 2, sizeof(zso_tok));
    u->Kr = (double *)calloc((size_t)(p->Br > 0 ? p->Br : 1) * p->d, sizeof(double));
    u->Vr = (double *)calloc((size_t)(p->Br > 0 ? p->Br : 1) * p->d, sizeof(double));
    u->w = (uint32_t *)calloc((size_t)(p->Br > 0 ? p->Br : 1), sizeof(uint32_t));
    return u;
}

static void clear_lists(zso_unit *u) {
    for (int i = 0; i < u->np; ++i) free(u->P[i].kv);
    for (int i = 0; i < u->nc; ++i) free(u->C[i].kv);
    u->np = u->nc = u->nr = 0;
    u->T = 0;
    u->last_n = 0;
}

void zso_unit_free(zso_unit *u) {
    if (!u) return;
    clear_lists(u);
    free(u->P);
    free(u->C);
    free(u->Kr);
    free(u->Vr);
    free(u->w);
    free(u->last_a);
    free(u->last_id);
    free(u);
}

static zso_tok make_tok(const double *k, const double *v, int d, float s, int32_t pos) {
    zso_tok t;
    t.kv = (double *)malloc(sizeof(double) * 2 * (size_t)d);
    memcpy(t.kv, k, sizeof(double) * (size_t)d);
    memcpy(t.kv + d, v, sizeof(double) * (size_t)d);
    t.s = s;
    t.pos = pos;
    return t;
}

/* Sec. 3.4: fold an evicted token into the residual component.
 * Free slot left -> the token takes it with fusion count 1 (Alg. 1 l.13-14).
 * Otherwise Eq. (hatr): slot with the largest raw dot product k_r . k_t
 * (or, with p.cosine, its cosine form; compared in fp32, equal values -> lowest slot), then Eq. (kvr): incremental
 * mean of keys and values, and the fusion count goes up by one.
 * Returns the slot merged into, -2 for a fill, -1 when B_r = 0. */
static int32_t residual_absorb(zso_unit *u, const double *k, const double *v, int32_t hint_slot,
                               double tol, int32_t *own_slot, int32_t *runner_slot, double *gap,
                               int32_t *near_tie, int32_t *mismatch, int32_t *exact_tie) {
    const int d = u->p.d;
    *own_slot = -1;
    *runner_slot = -1;
    *gap = INFINITY;
    *near_tie = *mismatch = *exact_tie = 0;
    if (u->p.Br == 0) return -1; /* Sec. 3.2: B_r = 0 is pure eviction */
    if (u->nr < u->p.Br) {
        memcpy(u->Kr + (size_t)u->nr * d, k, sizeof(double) * (size_t)d);
        memcpy(u->Vr + (size_t)u->nr * d, v, sizeof(double) * (size_t)d);
        u->w[u->nr] = 1;
        u->nr += 1;
        *own_slot = -2;
        return -2;
    }
    int32_t best = -1, runner = -1;
    float best_dot = 0.f, runner_dot = 0.f;
    double best_abs = 0.0, runner_abs = 0.0;
    float hint_dot = 0.f;
    double hint_abs = 0.0;
    for (int r = 0; r < u->nr; ++r) {
        const double *kr = u->Kr + (size_t)r * d;
        double acc = 0.0, aabs = 0.0, nr2 = 0.0, nt2 = 0.0;
        for (int i = 0; i < d; ++i) {
            acc += kr[i] * k[i];
            aabs += fabs(kr[i] * k[i]);
            nr2 += kr[i] * kr[i];
            nt2 += k[i] * k[i];
        }
        if (u->p.cosine) {
            /* cosine form of Eq. (hatr); a zero vector is similar to nothing */
            const double nn = sqrt(nr2) * sqrt(nt2);
            acc = nn > 0.0 ? acc / nn : 0.0;
            aabs = nn > 0.0 ? aabs / nn : 0.0;
        }
        float f = (float)acc;
        if (r == hint_slot) {
            hint_dot = f;
            hint_abs = aabs;
        }
        if (best < 0 || f > best_dot) {
            runner = best;
            runner_dot = best_dot;
            runner_abs = best_abs;
            best = r;
            best_dot = f;
            best_abs = aabs;
        } else if (runner < 0 || f > runner_dot) {
            runner = r;
            runner_dot = f;
            runner_abs = aabs;
        }
    }
    *own_slot = best;
    *runner_slot = runner;
    if (runner >= 0) {
        double den = fmax(fmax(best_abs, runner_abs), 1e-300);
        *gap = ((double)best_dot - (double)runner_dot) / den;
    }
    int32_t take = best;
    if (hint_slot >= 0 && hint_slot != best) {
        if (hint_slot >= u->nr) {
            *mismatch = 1;
        } else {
            double den = fmax(fmax(best_abs, hint_abs), 1e-300);
            double g = ((double)best_dot - (double)hint_dot) / den;
            if (hint_dot == best_dot) {
                *exact_tie = 1;
                *near_tie = 1;
                take = hint_slot;
            } else if (g <= tol) {
                *near_tie = 1;
                take = hint_slot;
            } else {
                *mismatch = 1;
            }
        }
    }
    double *kr = u->Kr + (size_t)take * d;
    double *vr = u->Vr + (size_t)take * d;
    const double wr = (double)u->w[take];
    for (int i = 0; i < d; ++i) {
        kr[i] = (wr * kr[i] + k[i]) / (wr + 1.0);
        vr[i] = (wr * vr[i] + v[i]) / (wr + 1.0);
    }
    u->w[take] += 1;
    return take;
}

int zso_decode_step(zso_unit *u, const double *q, const double *k_new, const double *v_new,
                    double *out, const zso_hint *hint, zso_step_report *rep) {
    if (!u || !q || !k_new || !v_new || !out) return -1;
    const int d = u->p.d, G = u->p.G;
    const int32_t n_tok = u->np + u->nc;
    const int32_t n = n_tok + u->nr + 1; /* cache as it stands plus the new token */

    if (u->last_cap < n) {
        free(u->last_a);
        free(u->last_id);
        u->last_cap = n + 64;
        u->last_a = (double *)malloc(sizeof(double) * (size_t)G * u->last_cap);
        u->last_id = (int64_t *)malloc(sizeof(int64_t) * (size_t)u->last_cap);
    }
    u->last_n = n;

    /* entry list: K_p, K_c, K_r, then the new token */
    const double **ek = (const double **)malloc(sizeof(double *) * (size_t)n);
    const double **ev = (const double **)malloc(sizeof(double *) * (size_t)n);
    double *comp = (double *)malloc(sizeof(double) * (size_t)n); /* alpha * log w */
    double *mean_a = (double *)calloc((size_t)n, sizeof(double));
    double *logit = (double *)malloc(sizeof(double) * (size_t)n);
    int32_t e = 0;
    for (int i = 0; i < u->np; ++i, ++e) {
        ek[e] = u->P[i].kv;
        ev[e] = u->P[i].kv + d;
        comp[e] = 0.0; /* w = 1 for uncompressed tokens */
        u->last_id[e] = u->P[i].pos;
    }
    for (int i = 0; i < u->nc; ++i, ++e) {
        ek[e] = u->C[i].kv;
        ev[e] = u->C[i].kv + d;
        comp[e] = 0.0;
        u->last_id[e] = u->C[i].pos;
    }
    for (int r = 0; r < u->nr; ++r, ++e) {
        ek[e] = u->Kr + (size_t)r * d;
        ev[e] = u->Vr + (size_t)r * d;
        comp[e] = u->p.alpha * log((double)u->w[r]); /* Eq. (att_score2) */
        u->last_id[e] = -(int64_t)(r + 1);
    }
    ek[e] = k_new;
    ev[e] = v_new;
    comp[e] = 0.0;
    u->last_id[e] = u->T;

    /* Eq. (att_score2): compensated softmax per query head, then the output */
    for (int g = 0; g < G; ++g) {
        const double *qg = q + (size_t)g * d;
        double m = -INFINITY;
        for (int j = 0; j < n; ++j) {
            logit[j] = dotd(qg, ek[j], d) * u->p.scale + comp[j];
            if (logit[j] > m) m = logit[j];
        }
        double Z = 0.0;
        for (int j = 0; j < n; ++j) {
            logit[j] = exp(logit[j] - m);
            Z += logit[j];
        }
        double *og = out + (size_t)g * d;
        for (int i = 0; i < d; ++i) og[i] = 0.0;
        for (int j = 0; j < n; ++j) {
            double a = logit[j] / Z;
            u->last_a[(size_t)g * n + j] = a;
            mean_a[j] += a / (double)G; /* grouped queries: mean over the group */
            for (int i = 0; i < d; ++i) og[i] += a * ev[j][i];
        }
    }

    /* Eq. (score): s <- lambda s + a, kept in fp32 */
    e = 0;
    for (int i = 0; i < u->np; ++i, ++e)
        u->P[i].s = (float)(u->p.lambda * (double)u->P[i].s + mean_a[e]);
    for (int i = 0; i < u->nc; ++i, ++e)
        u->C[i].s = (float)(u->p.lambda * (double)u->C[i].s + mean_a[e]);
    const float s_new = (float)mean_a[n - 1];

    zso_step_report R;
    memset(&R, 0, sizeof(R));
    R.victim_pos = R.victim_own_pos = R.victim_runner_pos = -1;
    R.merge_slot = R.merge_own_slot = R.merge_runner_slot = -1;
    R.victim_gap = INFINITY;
    R.merge_gap = INFINITY;

    /* Alg. 1 l.6: the new token joins the proximity list */
    u->P[u->np++] = make_tok(k_new, v_new, d, s_new, (int32_t)u->T);
    u->T += 1;

    int evicted = 0;
    /* Alg. 1 l.7-9: proximity overflow -> its oldest token moves to the context list */
    if (u->np > u->p.Bp) {
        zso_tok old = u->P[0];
        memmove(u->P, u->P + 1, sizeof(zso_tok) * (size_t)(u->np - 1));
        u->np -= 1;
        u->C[u->nc++] = old;
        /* Alg. 1 l.10-11: context overflow -> evict the lowest score (ties: lowest position) */
        if (u->nc > u->p.Bc) {
            int best = -1, runner = -1;
            for (int i = 0; i < u->nc; ++i) {
                const zso_tok *t = &u->C[i];
                if (best < 0 || t->s < u->C[best].s ||
                    (t->s == u->C[best].s && t->pos < u->C[best].pos)) {
                    runner = best;
                    best = i;
                } else if (runner < 0 || t->s < u->C[runner].s ||
                           (t->s == u->C[runner].s && t->pos < u->C[runner].pos)) {
                    runner = i;
                }
            }
            R.victim_own_pos = u->C[best].pos;
            if (runner >= 0) {
                R.victim_runner_pos = u->C[runner].pos;
                double sb = (double)u->C[best].s, sr = (double)u->C[runner].s;
                R.victim_gap = (sb > 0.0) ? (sr - sb) / sb : (sr > 0.0 ? INFINITY : 0.0);
            }
            int take = best;
            if (hint && hint->victim_pos >= 0 && hint->victim_pos != u->C[best].pos) {
                int hi = -1;
                for (int i = 0; i < u->nc; ++i)
                    if (u->C[i].pos == hint->victim_pos) hi = i;
                if (hi < 0) {
                    R.victim_mismatch = 1;
                } else {
                    double sb = (double)u->C[best].s, sh = (double)u->C[hi].s;
                    if (u->C[hi].s == u->C[best].s) {
                        R.victim_exact_tie = 1;
                        R.victim_near_tie = 1;
                        take = hi;
                    } else if (sh - sb <= hint->tol * sb) {
                        R.victim_near_tie = 1;
                        take = hi;
                    } else {
                        R.victim_mismatch = 1;
                    }
                }
            }
            zso_tok vic = u->C[take];
            u->C[take] = u->C[u->nc - 1];
            u->nc -= 1;
            R.victim_pos = vic.pos;
            evicted = 1;
            /* Alg. 1 l.12-16 */
            R.merge_slot = residual_absorb(
                u, vic.kv, vic.kv + d, hint ? hint->merge_slot : -1, hint ? hint->tol : 0.0,
                &R.merge_own_slot, &R.merge_runner_slot, &R.merge_gap, &R.merge_near_tie,
                &R.merge_mismatch, &R.merge_exact_tie);
            free(vic.kv);
        }
    }
    if (!evicted && hint && hint->victim_pos >= 0) R.victim_mismatch = 1;
    if (rep) *rep = R;

    free(ek);
    free(ev);
    free(comp);
    free(mean_a);
    free(logit);
    return 0;
}

typedef struct {
    float s;
    int32_t pos;
} zso_key;

static int key_cmp(const void *a, const void *b) {
    const zso_key *x = (const zso_key *)a, *y = (const zso_key *)b;
    if (x->s < y->s) return -1;
    if (x->s > y->s) return 1;
    return (x->pos > y->pos) - (x->pos < y->pos);
}

int zso_prefill_compress(zso_unit *u, const double *K, const double *V, const double *Qw,
                         const float *scores_in, int32_t T, int32_t W,
                         const uint8_t *hint_evicted, const int32_t *hint_targets, double tol,
                         float *scores_out, uint8_t *evicted_out, int32_t *targets_out,
                         zso_prefill_report *rep) {
    if (!u || !K || !V || T < 1) return -1;
    if (!Qw && !scores_in) return -1;
    if (Qw && (W < 1 || W > T)) return -1;
    const int d = u->p.d, G = u->p.G;
    clear_lists(u);

    zso_prefill_report R;
    memset(&R, 0, sizeof(R));
    R.min_merge_gap = INFINITY;
    R.sel_gap = INFINITY;

    /* P1. Scores from the prompt's last W queries: each query tau attends
     * causally to keys 0..tau (Eq. (att_score)); the unrolled recurrence of
     * Eq. (score) weights the row of query tau by lambda^(T-1-tau); grouped
     * queries are averaged.  Rounded to fp32 once, at the end. */
    float *s = (float *)malloc(sizeof(float) * (size_t)T);
    if (Qw) {
        double *acc = (double *)calloc((size_t)T, sizeof(double));
        double *row = (double *)malloc(sizeof(double) * (size_t)T);
        for (int g = 0; g < G; ++g) {
            for (int wq = 0; wq < W; ++wq) {
                const int32_t tau = T - W + wq;
                const double *qv = Qw + ((size_t)g * W + wq) * d;
                double m = -INFINITY;
                for (int t = 0; t <= tau; ++t) {
                    row[t] = dotd(qv, K + (size_t)t * d, d) * u->p.scale;
                    if (row[t] > m) m = row[t];
                }
                double Z = 0.0;
                for (int t = 0; t <= tau; ++t) {
                    row[t] = exp(row[t] - m);
                    Z += row[t];
                }
                const double coef = pow(u->p.lambda, (double)(T - 1 - tau));
                for (int t = 0; t <= tau; ++t) acc[t] += coef * (row[t] / Z);
            }
        }
        for (int t = 0; t < T; ++t) s[t] = (float)(acc[t] / (double)G);
        free(acc);
        free(row);
    } else {
        memcpy(s, scores_in, sizeof(float) * (size_t)T);
    }
    if (scores_out) memcpy(scores_out, s, sizeof(float) * (size_t)T);

    /* P2. The latest B_p positions are the proximity component (Sec. 3.2). */
    const int32_t n_prox = T < u->p.Bp ? T : u->p.Bp;
    const int32_t n_cand = T - n_prox;

    /* P3. Context component: the B_c candidates of highest score; the rest are
     * evicted, lowest (score, position) first -- the order of Alg. 1 l.11. */
    uint8_t *ev = (uint8_t *)calloc((size_t)T, 1);
    int32_t n_ev = n_cand > u->p.Bc ? n_cand - u->p.Bc : 0;
    if (n_ev > 0) {
        zso_key *keys = (zso_key *)malloc(sizeof(zso_key) * (size_t)n_cand);
        for (int t = 0; t < n_cand; ++t) {
            keys[t].s = s[t];
            keys[t].pos = t;
        }
        qsort(keys, (size_t)n_cand, sizeof(zso_key), key_cmp);
        for (int i = 0; i < n_ev; ++i) ev[keys[i].pos] = 1;
        const double s_emax = (double)keys[n_ev - 1].s; /* largest evicted score */
        const double s_kmin = (double)keys[n_ev].s;     /* smallest kept score */
        R.sel_gap = s_emax > 0.0 ? (s_kmin - s_emax) / s_emax : (s_kmin > 0.0 ? INFINITY : 0.0);
        if (hint_evicted) {
            /* take the other side's eviction set where it differs only by near ties */
            int32_t n_h = 0, ok = 1, differ = 0;
            for (int t = 0; t < n_cand; ++t) n_h += hint_evicted[t] ? 1 : 0;
            for (int t = n_cand; t < T; ++t)
                if (hint_evicted[t]) ok = 0;
            if (n_h != n_ev) ok = 0;
            for (int t = 0; ok && t < n_cand; ++t) {
                if (hint_evicted[t] && !ev[t]) { /* oracle keeps it, hint evicts it */
                    differ += 1;
                    if ((double)s[t] - s_emax > tol * s_emax) ok = 0;
                } else if (!hint_evicted[t] && ev[t]) { /* oracle evicts it, hint keeps it */
                    if (s_kmin - (double)s[t] > tol * s_kmin) ok = 0;
                }
            }
            if (ok) {
                R.n_near_tie_sel = differ;
                for (int t = 0; t < n_cand; ++t) ev[t] = hint_evicted[t] ? 1 : 0;
            } else {
                for (int t = 0; t < T; ++t)
                    if ((hint_evicted[t] ? 1 : 0) != ev[t]) R.n_mismatch_sel += 1;
            }
        }
        free(keys);
    } else if (hint_evicted) {
        for (int t = 0; t < T; ++t)
            if (hint_evicted[t]) R.n_mismatch_sel += 1;
    }
    R.n_evicted = n_ev;
    if (evicted_out) memcpy(evicted_out, ev, (size_t)T);

    /* P4. Evicted tokens enter the residual component in ascending position,
     * by the fill-or-merge rule of Alg. 1 l.12-16. */
    int32_t ie = 0;
    for (int t = 0; t < n_cand; ++t) {
        if (!ev[t]) continue;
        int32_t own, runner, nt, mm, et;
        double gap;
        int32_t slot = residual_absorb(u, K + (size_t)t * d, V + (size_t)t * d,
                                       hint_targets ? hint_targets[ie] : -1, tol, &own, &runner,
                                       &gap, &nt, &mm, &et);
        if (targets_out) targets_out[ie] = slot;
        R.n_near_tie_merge += nt;
        R.n_mismatch_merge += mm;
        R.n_exact_tie_merge += et;
        if (gap < R.min_merge_gap) R.min_merge_gap = gap;
        ie += 1;
    }

    /* P5. Survivors keep their rows, scores and positions. */
    for (int t = 0; t < n_cand; ++t) {
        if (ev[t]) continue;
        u->C[u->nc++] = make_tok(K + (size_t)t * d, V + (size_t)t * d, d, s[t], t);
    }
    for (int t = n_cand; t < T; ++t)
        u->P[u->np++] = make_tok(K + (size_t)t * d, V + (size_t)t * d, d, s[t], t);
    u->T = T;

    if (rep) *rep = R;
    free(ev);
    free(s);
    return 0;
}

void zso_counts(const zso_unit *u, int32_t *np, int32_t *nc, int32_t *nr, int64_t *T) {
    if (np) *np = u->np;
    if (nc) *nc = u->nc;
    if (nr) *nr = u->nr;
    if (T) *T = u->T;
}

void zso_export_tokens(const zso_unit *u, int32_t *pos, float *score, double *K, double *V) {
    const int d = u->p.d;
    int32_t e = 0;
    for (int pass = 0; pass < 2; ++pass) {
        const zso_tok *L = pass == 0 ? u->P : u->C;
        const int32_t n = pass == 0 ? u->np : u->nc;
        for (int i = 0; i < n; ++i, ++e) {
            if (pos) pos[e] = L[i].pos;
            if (score) score[e] = L[i].s;
            if (K) memcpy(K + (size_t)e * d, L[i].kv, sizeof(double) * (size_t)d);
            if (V) memcpy(V + (size_t)e * d, L[i].kv + d, sizeof(double) * (size_t)d);
        }
    }
}

void zso_export_residual(const zso_unit *u, double *Kr, double *Vr, uint32_t *w) {
    const size_t n = (size_t)u->nr * u->p.d;
    if (Kr) memcpy(Kr, u->Kr, sizeof(double) * n);
    if (Vr) memcpy(Vr, u->Vr, sizeof(double) * n);
    if (w) memcpy(w, u->w, sizeof(uint32_t) * (size_t)u->nr);
}

int32_t zso_last_attention(const zso_unit *u, double *a, int64_t *id) {
    if (a) memcpy(a, u->last_a, sizeof(double) * (size_t)u->p.G * u->last_n);
    if (id) memcpy(id, u->last_id, sizeof(int64_t) * (size_t)u->last_n);
    return u->last_n;
}

int zso_decode_step_batch(zso_unit **units, int32_t n, const double *q, const double *k_new,
                          const double *v_new, double *out) {
    int threads = 1;
#ifdef _OPENMP
    threads = omp_get_max_threads();
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t i = 0; i < n; ++i) {
        const int d = units[i]->p.d, G = units[i]->p.G;
        zso_decode_step(units[i], q + (size_t)i * G * d, k_new + (size_t)i * d,
                        v_new + (size_t)i * d, out + (size_t)i * G * d, NULL, NULL);
    }
    return threads;
}

int zso_split_budget(int32_t B, double tail_ratio, double dense_ratio, int32_t *Bp, int32_t *Bc,
                     int32_t *Br) {
    if (B < 1 || tail_ratio < 0.0 || tail_ratio > 1.0 || dense_ratio < 0.0 || dense_ratio > 1.0)
        return -1;
    /* App. C.2: B_p = tail ratio * B first, then B_r = dense ratio * (B - B_p),
     * the rest is B_c.  Rounding is a reading: floor, then round-half-up with a
     * floor of one slot whenever the dense ratio is positive. */
    int32_t bp = (int32_t)floor(tail_ratio * (double)B);
    int32_t rest = B - bp;
    int32_t br = 0;
    if (dense_ratio > 0.0 && rest > 0) {
        br = (int32_t)floor(dense_ratio * (double)rest + 0.5);
        if (br < 1) br = 1;
        if (br > rest) br = rest;
    }
    int32_t bc = rest - br;
    if (bp + bc < 1) { /* keep at least one token slot */
        if (br > 0) {
            br -= 1;
            bc += 1;
        }
    }
    *Bp = bp;
    *Bc = bc;
    *Br = br;
    return 0;
}
