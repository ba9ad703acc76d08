/*
 * Moment-KV reference oracle: plain, slow, fp64, one sequence of one attention
 * layer per state object.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the test-suite, the smoke
 * check and the benchmark's CPU-baseline leg may build, load or call it.  It
 * shares no code, header, table or helper with the CUDA library, and neither
 * side includes or imports the other.
 *
 * What it follows (Moment-KV paper):
 *   - Sec. 4.1 "KV Cache Preliminaries": cache pool = prefill pool U decode
 *     pool (Eq. 1) and softmax(q K^T / sqrt(d)) V over the whole pool (Eq. 2).
 *   - Sec. 4.2, Algorithm 1 "Decoding with Moment-KV", steps in the printed
 *     order: append (K_t,V_t) and a zero importance; attention over the whole
 *     pool including the fresh token; mean over heads; slice the decode part;
 *     I_i <- alpha*I_i + abar_i for every decode token; if the decode pool is
 *     over budget remove the overflow-many lowest-importance tokens.
 *   - Sec. 4.2 "Momentum-Based Attention Aggregation" (Eq. 4, Eq. 5),
 *     "Handling Newly Generated Tokens" (Eq. 6: eviction after the update),
 *     "Capacity Enforcement and Eviction" (Eq. 7-9).
 *
 * Readings where the paper is silent (all listed in the design document):
 *   - GQA: query head h reads KV head h / G (G = q_heads / kv_heads).
 *   - Head mean: GROUP mode averages the G query heads of one KV head and every
 *     KV head keeps its own importance vector; LAYER mode averages all H query
 *     heads (the formula exactly as printed in Eq. 4) and all KV heads share
 *     one importance vector.  With one KV head the two coincide.
 *   - d in 1/sqrt(d) is the head dimension.
 *   - Ties in the arg-min: the older token (lower index == smaller position
 *     id) goes first.
 *   - The attention output of a step uses the pool as it is BEFORE that
 *     step's eviction (attention is computed before the capacity check).
 *
 * No blocking, fusion or reordering: every logit, every exponential, every
 * probability is formed exactly as the definitions state.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define MKO_GROUP_MEAN 0
#define MKO_LAYER_MEAN 1

typedef struct {
    double *K, *V;     /* [cap][d] decode pool of one KV head, insertion order */
    double *I;         /* [cap] importance                                     */
    int64_t *pos;      /* [cap] decode-step id at which the token was appended */
    double *abar;      /* [cap] head-averaged attention of the last step       */
    int n, cap;
    /* record of the last eviction */
    int64_t *ev_pos;
    double *ev_score;
    int ev_n, ev_cap;
} mko_head;

typedef struct mko_state {
    int Hq, Hkv, d, G, budget, Lp, mode;
    double beta;
    double *Kp, *Vp;   /* [Hkv][Lp][d] frozen prefill pool */
    mko_head *h;       /* [Hkv] */
    int64_t t;         /* decode steps completed */
    int pending;       /* 1 between attend_update and evict */
    double *logit;     /* scratch [Lp + n] */
    double *prob;      /* scratch [Hq][max n] decode-token probabilities */
    int prob_cap;
} mko_state;

static void head_reserve(mko_head *hd, int d, int want) {
    if (want <= hd->cap) return;
    int cap = hd->cap ? hd->cap : 16;
    while (cap < want) cap *= 2;
    hd->K = (double *)realloc(hd->K, sizeof(double) * (size_t)cap * d);
    hd->V = (double *)realloc(hd->V, sizeof(double) * (size_t)cap * d);
    hd->I = (double *)realloc(hd->I, sizeof(double) * (size_t)cap);
    hd->abar = (double *)realloc(hd->abar, sizeof(double) * (size_t)cap);
    hd->pos = (int64_t *)realloc(hd->pos, sizeof(int64_t) * (size_t)cap);
    hd->cap = cap;
}

mko_state *mko_create(int q_heads, int kv_heads, int head_dim, int budget, double beta,
                      int prefill_len, int mode) {
    if (q_heads <= 0 || kv_heads <= 0 || head_dim <= 0 || budget < 1 || prefill_len < 0) return NULL;
    if (q_heads % kv_heads) return NULL;
    if (mode != MKO_GROUP_MEAN && mode != MKO_LAYER_MEAN) return NULL;
    mko_state *s = (mko_state *)calloc(1, sizeof(mko_state));
    s->Hq = q_heads; s->Hkv = kv_heads; s->d = head_dim; s->G = q_heads / kv_heads;
    s->budget = budget; s->beta = beta; s->Lp = prefill_len; s->mode = mode;
    size_t np = (size_t)kv_heads * (size_t)prefill_len * (size_t)head_dim;
    s->Kp = (double *)calloc(np ? np : 1, sizeof(double));
    s->Vp = (double *)calloc(np ? np : 1, sizeof(double));
    s->h = (mko_head *)calloc((size_t)kv_heads, sizeof(mko_head));
    return s;
}

void mko_destroy(mko_state *s) {
    if (!s) return;
    for (int g = 0; g < s->Hkv; ++g) {
        free(s->h[g].K); free(s->h[g].V); free(s->h[g].I); free(s->h[g].pos);
        free(s->h[g].abar); free(s->h[g].ev_pos); free(s->h[g].ev_score);
    }
    free(s->h); free(s->Kp); free(s->Vp); free(s->logit); free(s->prob); free(s);
}

/* Sec. 4.1 prefill phase: the prompt's K_P, V_P are written once; frozen afterwards. */
void mko_prefill(mko_state *s, const double *K, const double *V) {
    size_t np = (size_t)s->Hkv * (size_t)s->Lp * (size_t)s->d;
    memcpy(s->Kp, K, np * sizeof(double));
    memcpy(s->Vp, V, np * sizeof(double));
    for (int g = 0; g < s->Hkv; ++g) { s->h[g].n = 0; s->h[g].ev_n = 0; }
    s->t = 0; s->pending = 0;
}

void mko_set_budget(mko_state *s, int budget) { if (budget >= 1) s->budget = budget; }

/*
 * State loader (no arithmetic): puts KV head g's decode pool into a given state -- n tokens
 * with keys, values, importances and position ids, in the given order -- and sets the number of
 * completed steps.  A harness uses it to start the step-by-step comparison from a state that was
 * reached elsewhere (a long warm-up that the oracle is too slow to follow).
 */
int mko_load_decode_state(mko_state *s, int g, int n, const double *K, const double *V,
                          const double *I, const int64_t *pos, int64_t steps_done) {
    if (g < 0 || g >= s->Hkv || n < 0 || s->pending) return -1;
    mko_head *hd = &s->h[g];
    head_reserve(hd, s->d, n + 1);
    memcpy(hd->K, K, sizeof(double) * (size_t)n * s->d);
    memcpy(hd->V, V, sizeof(double) * (size_t)n * s->d);
    for (int i = 0; i < n; ++i) { hd->I[i] = I[i]; hd->pos[i] = pos[i]; hd->abar[i] = 0.0; }
    hd->n = n;
    hd->ev_n = 0;
    s->t = steps_done;
    return 0;
}

/*
 * Algorithm 1, from the append up to and including the importance update.
 * q [Hq][d], k_new, v_new [Hkv][d], out [Hq][d].
 */
int mko_attend_update(mko_state *s, const double *q, const double *k_new, const double *v_new,
                      double *out) {
    if (s->pending) return -1;
    const int d = s->d, Lp = s->Lp, G = s->G;
    /* Algorithm 1: Phi_d <- Phi_d U {(K_t, V_t)};  I <- I U {0}. */
    int nmax = 0;
    for (int g = 0; g < s->Hkv; ++g) {
        mko_head *hd = &s->h[g];
        head_reserve(hd, d, hd->n + 1);
        memcpy(hd->K + (size_t)hd->n * d, k_new + (size_t)g * d, sizeof(double) * d);
        memcpy(hd->V + (size_t)hd->n * d, v_new + (size_t)g * d, sizeof(double) * d);
        hd->I[hd->n] = 0.0;
        hd->pos[hd->n] = s->t;
        hd->n += 1;
        if (hd->n > nmax) nmax = hd->n;
    }
    if (nmax > s->prob_cap) {
        s->prob_cap = nmax * 2;
        s->prob = (double *)realloc(s->prob, sizeof(double) * (size_t)s->Hq * s->prob_cap);
        s->logit = (double *)realloc(s->logit, sizeof(double) * (size_t)(Lp + s->prob_cap));
    }
    const double inv_sqrt_d = 1.0 / sqrt((double)d);
    /* Eq. 2 / Algorithm 1: A_t = softmax(q K^T / sqrt(d)) over prefill then decode tokens. */
    for (int hq = 0; hq < s->Hq; ++hq) {
        const int g = hq / G;
        const mko_head *hd = &s->h[g];
        const int n = hd->n, N = Lp + n;
        const double *qh = q + (size_t)hq * d;
        double *lg = s->logit;
        double mx = -INFINITY;
        for (int j = 0; j < N; ++j) {
            const double *kj = (j < Lp) ? s->Kp + ((size_t)g * Lp + j) * d
                                        : hd->K + (size_t)(j - Lp) * d;
            double acc = 0.0;
            for (int c = 0; c < d; ++c) acc += qh[c] * kj[c];
            lg[j] = acc * inv_sqrt_d;
            if (lg[j] > mx) mx = lg[j];
        }
        double Z = 0.0;
        for (int j = 0; j < N; ++j) { lg[j] = exp(lg[j] - mx); Z += lg[j]; }
        double *oh = out + (size_t)hq * d;
        for (int c = 0; c < d; ++c) oh[c] = 0.0;
        for (int j = 0; j < N; ++j) {
            const double p = lg[j] / Z;
            const double *vj = (j < Lp) ? s->Vp + ((size_t)g * Lp + j) * d
                                        : hd->V + (size_t)(j - Lp) * d;
            for (int c = 0; c < d; ++c) oh[c] += p * vj[c];
            /* Algorithm 1: a_dec = A_t[|Phi_p|:] -- keep the decode part only. */
            if (j >= Lp) s->prob[(size_t)hq * s->prob_cap + (j - Lp)] = p;
        }
    }
    /* Eq. 4: mean over heads; Eq. 5: I_i(t) = alpha * I_i(t-1) + abar_i(t). */
    if (s->mode == MKO_GROUP_MEAN) {
        for (int g = 0; g < s->Hkv; ++g) {
            mko_head *hd = &s->h[g];
            for (int i = 0; i < hd->n; ++i) {
                double sum = 0.0;
                for (int r = 0; r < G; ++r) sum += s->prob[(size_t)(g * G + r) * s->prob_cap + i];
                hd->abar[i] = sum / (double)G;
                hd->I[i] = s->beta * hd->I[i] + hd->abar[i];
            }
        }
    } else {
        /* all KV heads hold the same token set; one shared vector, kept as equal copies */
        const int n = s->h[0].n;
        for (int i = 0; i < n; ++i) {
            double sum = 0.0;
            for (int hq = 0; hq < s->Hq; ++hq) sum += s->prob[(size_t)hq * s->prob_cap + i];
            const double ab = sum / (double)s->Hq;
            for (int g = 0; g < s->Hkv; ++g) {
                s->h[g].abar[i] = ab;
                s->h[g].I[i] = s->beta * s->h[g].I[i] + ab;
            }
        }
    }
    s->pending = 1;
    return 0;
}

/*
 * Eq. 8: the k lowest importances, written as the sort it defines.  Order is
 * (score ascending, position id ascending); out_idx receives the k chosen
 * indices in that order.  Also usable on its own with scores produced elsewhere.
 */
typedef struct { double s; int64_t p; int i; } mko_key;
static int key_cmp(const void *a, const void *b) {
    const mko_key *x = (const mko_key *)a, *y = (const mko_key *)b;
    if (x->s < y->s) return -1;
    if (x->s > y->s) return 1;
    if (x->p < y->p) return -1;
    if (x->p > y->p) return 1;
    return (x->i > y->i) - (x->i < y->i);
}
int mko_select(const double *score, const int64_t *pos, int n, int k, int *out_idx) {
    if (k < 0 || k > n) return -1;
    mko_key *keys = (mko_key *)malloc(sizeof(mko_key) * (size_t)(n ? n : 1));
    for (int i = 0; i < n; ++i) { keys[i].s = score[i]; keys[i].p = pos ? pos[i] : i; keys[i].i = i; }
    qsort(keys, (size_t)n, sizeof(mko_key), key_cmp);
    for (int j = 0; j < k; ++j) out_idx[j] = keys[j].i;
    free(keys);
    return 0;
}

/* Eq. 5 on its own: I <- beta * I + abar, elementwise. */
void mko_update(double *I, const double *abar, int n, double beta) {
    for (int i = 0; i < n; ++i) I[i] = beta * I[i] + abar[i];
}

/* What Eq. 7-8 would evict from KV head g right now (no state change). */
int mko_choose(const mko_state *s, int g, int64_t *out_pos, int cap) {
    const mko_head *hd = &s->h[g];
    int k = hd->n - s->budget;            /* Eq. 7 */
    if (k <= 0) return 0;
    if (k > cap) return -1;
    int *idx = (int *)malloc(sizeof(int) * (size_t)k);
    mko_select(hd->I, hd->pos, hd->n, k, idx);
    for (int j = 0; j < k; ++j) out_pos[j] = hd->pos[idx[j]];
    free(idx);
    return k;
}

static void head_remove(mko_head *hd, int d, const char *drop) {
    int w = 0; hd->ev_n = 0;
    for (int i = 0; i < hd->n; ++i) {
        if (drop[i]) {
            if (hd->ev_n >= hd->ev_cap) {
                hd->ev_cap = hd->ev_cap ? hd->ev_cap * 2 : 8;
                hd->ev_pos = (int64_t *)realloc(hd->ev_pos, sizeof(int64_t) * (size_t)hd->ev_cap);
                hd->ev_score = (double *)realloc(hd->ev_score, sizeof(double) * (size_t)hd->ev_cap);
            }
            hd->ev_pos[hd->ev_n] = hd->pos[i];
            hd->ev_score[hd->ev_n] = hd->I[i];
            hd->ev_n += 1;
            continue;
        }
        if (w != i) {
            memcpy(hd->K + (size_t)w * d, hd->K + (size_t)i * d, sizeof(double) * d);
            memcpy(hd->V + (size_t)w * d, hd->V + (size_t)i * d, sizeof(double) * d);
            hd->I[w] = hd->I[i]; hd->pos[w] = hd->pos[i]; hd->abar[w] = hd->abar[i];
        }
        ++w;
    }
    hd->n = w;
}

/*
 * Algorithm 1, capacity check and removal (Eq. 7-9).  force_pos, when not NULL,
 * lists for each KV head the position ids to evict instead of the arg-min
 * ([Hkv][force_stride], force_cnt[g] entries used); a harness uses it to keep a
 * free-running comparison in lockstep after a tolerated near-tie.
 */
int mko_evict(mko_state *s, const int64_t *force_pos, const int *force_cnt, int force_stride) {
    if (!s->pending) return -1;
    for (int g = 0; g < s->Hkv; ++g) {
        mko_head *hd = &s->h[g];
        const int k = hd->n - s->budget;  /* overflow */
        hd->ev_n = 0;
        if (k <= 0) continue;
        char *drop = (char *)calloc((size_t)hd->n, 1);
        if (force_pos) {
            if (force_cnt[g] != k) { free(drop); return -2; }
            for (int j = 0; j < k; ++j) {
                int found = 0;
                for (int i = 0; i < hd->n; ++i)
                    if (hd->pos[i] == force_pos[(size_t)g * force_stride + j]) { drop[i] = 1; found = 1; break; }
                if (!found) { free(drop); return -3; }
            }
        } else {
            int *idx = (int *)malloc(sizeof(int) * (size_t)k);
            mko_select(hd->I, hd->pos, hd->n, k, idx);
            for (int j = 0; j < k; ++j) drop[idx[j]] = 1;
            free(idx);
        }
        head_remove(hd, s->d, drop);      /* Phi_d <- Phi_d \ E_t ; I <- I \ E_t */
        free(drop);
    }
    s->t += 1;
    s->pending = 0;
    return 0;
}

int mko_step(mko_state *s, const double *q, const double *k_new, const double *v_new, double *out) {
    int rc = mko_attend_update(s, q, k_new, v_new, out);
    if (rc) return rc;
    return mko_evict(s, NULL, NULL, 0);
}

/* ---- inspection ---- */
int mko_decode_count(const mko_state *s, int g) { return s->h[g].n; }
int64_t mko_steps_done(const mko_state *s) { return s->t; }
int mko_get_decode_state(const mko_state *s, int g, int64_t *pos, double *score, double *abar, int cap) {
    const mko_head *hd = &s->h[g];
    if (hd->n > cap) return -1;
    for (int i = 0; i < hd->n; ++i) {
        if (pos) pos[i] = hd->pos[i];
        if (score) score[i] = hd->I[i];
        if (abar) abar[i] = hd->abar[i];
    }
    return hd->n;
}
int mko_get_last_evicted(const mko_state *s, int g, int64_t *pos, double *score, int cap) {
    const mko_head *hd = &s->h[g];
    if (hd->ev_n > cap) return -1;
    for (int i = 0; i < hd->ev_n; ++i) { if (pos) pos[i] = hd->ev_pos[i]; if (score) score[i] = hd->ev_score[i]; }
    return hd->ev_n;
}
int mko_read_decode_kv(const mko_state *s, int g, double *K, double *V, int cap) {
    const mko_head *hd = &s->h[g];
    if (hd->n > cap) return -1;
    memcpy(K, hd->K, sizeof(double) * (size_t)hd->n * s->d);
    memcpy(V, hd->V, sizeof(double) * (size_t)hd->n * s->d);
    return hd->n;
}
const double *mko_prefill_k(const mko_state *s) { return s->Kp; }
const double *mko_prefill_v(const mko_state *s) { return s->Vp; }
