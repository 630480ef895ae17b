/*
 * lar_oracle.c — plain CPU oracle for LineAR decode attention and line-end eviction.
 *
 * TEST INFRASTRUCTURE.  This file is the slow, obviously-correct statement of what the CUDA
 * library must compute.  Only tests, the smoke check and the benchmark's cpu-baseline leg may
 * build or call it; the product path never does.  It shares no code with the CUDA path.
 *
 * Everything is written out from the paper's definitions, in double precision, with no
 * blocking, fusion or reordering:
 *   - decode attention ........ Sec. 3.1, Eq. 2-3 (softmax(q K^T / sqrt(d)) V over the live cache)
 *   - cache append ............ Sec. 3.1, Eq. 4
 *   - line view, budget B ..... Sec. 3.3 "Visual KV Cache Management in a 2D View", "Cache Budget"
 *   - progressive pipeline .... Sec. 3.3, Eq. 5-7 (partition init / mid / rec, evict n from mid,
 *                               |cache| = B - n after a compression, n-token buffer for the next line)
 *   - guide queue ............. Sec. 3.3, Eq. 8
 *   - saliency score .......... Sec. 3.3, Eq. 9
 *   - BottomK eviction ........ Sec. 3.3, Eq. 10
 *
 * Readings taken where the paper is silent (each is a parameter or a stated convention):
 *   - B counts visual tokens only; the C conditional tokens are kept in addition (the efficiency
 *     table lists B = 96 for N = 576 at ratio 1/6, i.e. exactly rho * N).
 *   - first compression happens at the end of line B/n (cache exactly full).
 *   - N_init and r are parameters (their values are not in the paper's main text).
 *   - the softmax of Eq. 9 normalises over the mid keys only, as the equation is written
 *     (score_norm = 1 selects the other reading: the probabilities the queries had at decode time;
 *     score_norm = 2 the accumulated-attention scoring of the paper's ablation "w. AttAcc" and of the
 *     H2O-style baselines it describes: every cached token's attention probability of Eq. 2-3, summed
 *     over all decode steps since the token was appended and over the G heads).
 *   - with grouped-query attention the score of a cached token is the mean over the G query heads
 *     that share its KV head (folded into the 1/n of Eq. 9 as 1/(nG)).
 *   - ties in BottomK: among equal scores the token with the higher original position is evicted
 *     first (the older one is kept).
 *   - kept tokens stay in ascending original position (stable compaction).
 *
 * Parity status: decode attention, saliency, BottomK and the pipeline's size/retention behaviour
 * are pinned by tests (library softmax/matmul, closed forms, brute force, invariants).  The kept
 * sets on real model attention, and the values of N_init / r / the GQA and normalisation readings
 * against the authors' implementation, are "parity unpinned": the paper prints no worked example.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int cond_len;      /* C      */
    int line_width;    /* n      */
    int n_lines;       /* h, N = h * n */
    int budget_lines;  /* B / n; >= n_lines means the cache is never compressed */
    int anchor_len;    /* N_init */
    int recent_lines;  /* r      */
    int group;         /* G query heads per KV head */
    int head_dim;      /* d      */
    double scale;      /* logit scale; 0 selects 1/sqrt(d) */
    int score_norm;    /* 0: Eq. 9 as written (softmax over the mid keys only);
                          1: variant -- softmax over every entry the query attended to when it was decoded;
                          2: accumulated attention over all history (the "w. AttAcc" ablation): the score of an
                             entry is the sum of the probabilities Eq. 2-3 gave it at every step since it was
                             appended, over the G heads, divided by n G (so that a sum that restarted at every
                             line end would equal variant 1) */
} lar_oracle_cfg;

typedef struct {
    lar_oracle_cfg c;
    int cap;          /* C + N entries (never more are live) */
    int len;          /* live entries */
    int n_vis;        /* visual tokens appended so far (the step index i) */
    int n_guide;      /* queries in the guide queue */
    int *pos;         /* [cap] original position: prefix j -> j, visual token i (1-based) -> C + i - 1 */
    double *K, *V;    /* [cap][d] */
    double *guide;    /* [n][G][d] */
    double *acc;      /* [cap] attention mass each live entry has received so far (score_norm = 2) */
} lar_oracle_unit;

static double cfg_scale(const lar_oracle_cfg *c) {
    return c->scale != 0.0 ? c->scale : 1.0 / sqrt((double)c->head_dim);
}

/* ---------------------------------------------------------------------------------------------
 * Eq. 2: out = softmax(q K^T * scale) V for one query row.  probs (len) may be NULL.
 * ------------------------------------------------------------------------------------------- */
void lar_oracle_attention(const double *q, const double *K, const double *V, int len, int d,
                          double scale, double *out, double *probs) {
    double *p = (double *)malloc(sizeof(double) * (size_t)(len > 0 ? len : 1));
    double mx = -INFINITY;
    for (int j = 0; j < len; ++j) {
        double s = 0.0;
        for (int t = 0; t < d; ++t) s += q[t] * K[(size_t)j * d + t];
        p[j] = s * scale;
        if (p[j] > mx) mx = p[j];
    }
    double den = 0.0;
    for (int j = 0; j < len; ++j) { p[j] = exp(p[j] - mx); den += p[j]; }
    for (int j = 0; j < len; ++j) p[j] /= den;
    for (int t = 0; t < d; ++t) out[t] = 0.0;
    for (int j = 0; j < len; ++j)
        for (int t = 0; t < d; ++t) out[t] += p[j] * V[(size_t)j * d + t];
    if (probs) memcpy(probs, p, sizeof(double) * (size_t)len);
    free(p);
}

/* ---------------------------------------------------------------------------------------------
 * Eq. 9: S = (1/nq) * 1^T Softmax(Qg Kmid^T * scale); Qg is [nq][d], Kmid is [M][d], S is [M].
 * Each query row is normalised over the M mid keys, then the rows are averaged.
 * ------------------------------------------------------------------------------------------- */
void lar_oracle_saliency(const double *Qg, int nq, const double *Kmid, int M, int d, double scale,
                         double *S) {
    double *a = (double *)malloc(sizeof(double) * (size_t)(M > 0 ? M : 1));
    for (int m = 0; m < M; ++m) S[m] = 0.0;
    for (int j = 0; j < nq; ++j) {
        double mx = -INFINITY;
        for (int m = 0; m < M; ++m) {
            double s = 0.0;
            for (int t = 0; t < d; ++t) s += Qg[(size_t)j * d + t] * Kmid[(size_t)m * d + t];
            a[m] = s * scale;
            if (a[m] > mx) mx = a[m];
        }
        double den = 0.0;
        for (int m = 0; m < M; ++m) { a[m] = exp(a[m] - mx); den += a[m]; }
        for (int m = 0; m < M; ++m) S[m] += a[m] / den;
    }
    for (int m = 0; m < M; ++m) S[m] /= (double)nq;
    free(a);
}

/* ---------------------------------------------------------------------------------------------
 * Variant of Eq. 9 (the alternative reading of its softmax): each guide query is normalised over
 * every entry it attended to when it was decoded -- all live entries whose original position does
 * not exceed the query's own -- and the mid columns of those probabilities are averaged.  These are
 * the attention probabilities of Eq. 2-3 accumulated over the steps of the line.
 *   Qg [n][G][d] guide rows, query t of the line has original position first_qpos + t;
 *   K [len][d] live keys with original positions pos[len]; mid_slot[M] slots of the mid entries.
 * ------------------------------------------------------------------------------------------- */
void lar_oracle_saliency_cache(const double *Qg, int n, int G, const double *K, const int *pos, int len,
                               int d, double scale, int first_qpos, const int *mid_slot, int M,
                               double *S) {
    double *a = (double *)malloc(sizeof(double) * (size_t)(len > 0 ? len : 1));
    for (int m = 0; m < M; ++m) S[m] = 0.0;
    for (int t = 0; t < n; ++t) {
        for (int g = 0; g < G; ++g) {
            const double *qrow = Qg + ((size_t)t * G + g) * d;
            double mx = -INFINITY;
            for (int s = 0; s < len; ++s) {
                if (pos[s] > first_qpos + t) { a[s] = -INFINITY; continue; }   /* appended after this query */
                double x = 0.0;
                for (int e = 0; e < d; ++e) x += qrow[e] * K[(size_t)s * d + e];
                a[s] = x * scale;
                if (a[s] > mx) mx = a[s];
            }
            double den = 0.0;
            for (int s = 0; s < len; ++s) { a[s] = exp(a[s] - mx); den += a[s]; }
            for (int m = 0; m < M; ++m) S[m] += a[mid_slot[m]] / den;
        }
    }
    for (int m = 0; m < M; ++m) S[m] /= (double)(n * G);
    free(a);
}

/* ---------------------------------------------------------------------------------------------
 * Eq. 10: indices (into the mid list) of the k least salient entries.
 * Total order "evicted earlier": lower score first; among equal scores the higher position first.
 * evict_idx receives the k indices in the order they are chosen (least salient first).
 * ------------------------------------------------------------------------------------------- */
void lar_oracle_bottomk(const double *S, const int *pos, int M, int k, int *evict_idx) {
    char *gone = (char *)calloc((size_t)(M > 0 ? M : 1), 1);
    for (int e = 0; e < k; ++e) {
        int best = -1;
        for (int m = 0; m < M; ++m) {
            if (gone[m]) continue;
            if (best < 0 || S[m] < S[best] || (S[m] == S[best] && pos[m] > pos[best])) best = m;
        }
        gone[best] = 1;
        evict_idx[e] = best;
    }
    free(gone);
}

/* ---------------------------------------------------------------------------------------------
 * One independent unit = (layer, sequence, KV head): its cache, positions and guide queue.
 * ------------------------------------------------------------------------------------------- */
lar_oracle_unit *lar_oracle_unit_create(const lar_oracle_cfg *cfg) {
    if (!cfg || cfg->head_dim < 1 || cfg->line_width < 1 || cfg->n_lines < 1 || cfg->group < 1 ||
        cfg->cond_len < 0 || cfg->anchor_len < 0 || cfg->recent_lines < 0 || cfg->budget_lines < 1)
        return NULL;
    if (cfg->budget_lines < cfg->n_lines) {
        /* a compressing configuration needs at least n mid candidates at every line end */
        int B = cfg->budget_lines * cfg->line_width;
        if (B - cfg->anchor_len - cfg->recent_lines * cfg->line_width < cfg->line_width) return NULL;
    }
    lar_oracle_unit *u = (lar_oracle_unit *)calloc(1, sizeof(*u));
    u->c = *cfg;
    u->cap = cfg->cond_len + cfg->line_width * cfg->n_lines;
    size_t d = (size_t)cfg->head_dim;
    u->pos = (int *)calloc((size_t)u->cap, sizeof(int));
    u->K = (double *)calloc((size_t)u->cap * d, sizeof(double));
    u->V = (double *)calloc((size_t)u->cap * d, sizeof(double));
    u->guide = (double *)calloc((size_t)cfg->line_width * (size_t)cfg->group * d, sizeof(double));
    u->acc = (double *)calloc((size_t)u->cap, sizeof(double));
    return u;
}

void lar_oracle_unit_destroy(lar_oracle_unit *u) {
    if (!u) return;
    free(u->pos); free(u->K); free(u->V); free(u->guide); free(u->acc); free(u);
}

int lar_oracle_unit_len(const lar_oracle_unit *u) { return u->len; }
int lar_oracle_unit_n_visual(const lar_oracle_unit *u) { return u->n_vis; }
void lar_oracle_unit_positions(const lar_oracle_unit *u, int *pos_out) {
    memcpy(pos_out, u->pos, sizeof(int) * (size_t)u->len);
}

/* Attention mass every live entry has received since it was appended (cache order), summed over the G heads. */
void lar_oracle_unit_accumulated(const lar_oracle_unit *u, double *acc_out) {
    memcpy(acc_out, u->acc, sizeof(double) * (size_t)u->len);
}

/* Prefill (Sec. 3.1): the C conditional K/V rows become entries 0..C-1.  kc, vc: [C][d] floats. */
int lar_oracle_unit_prefill(lar_oracle_unit *u, const float *kc, const float *vc) {
    if (u->len != 0) return -1;
    int d = u->c.head_dim;
    for (int j = 0; j < u->c.cond_len; ++j) {
        u->pos[j] = j;
        for (int t = 0; t < d; ++t) {
            u->K[(size_t)j * d + t] = (double)kc[(size_t)j * d + t];
            u->V[(size_t)j * d + t] = (double)vc[(size_t)j * d + t];
        }
    }
    u->len = u->c.cond_len;
    return 0;
}

/* One decode step for visual token i = n_vis + 1:
 *   Eq. 4  append (k_i, v_i);
 *   Eq. 2  each of the G query heads attends to every live entry, the new one included;
 *   Eq. 8  the G queries join the guide queue of the current line.
 * q: [G][d], k, v: [d] floats; out: [G][d] doubles; probs: [G][len_after] doubles or NULL. */
int lar_oracle_unit_step(lar_oracle_unit *u, const float *q, const float *k, const float *v,
                         double *out, double *probs) {
    const lar_oracle_cfg *c = &u->c;
    int d = c->head_dim, G = c->group, n = c->line_width;
    if (u->len >= u->cap) return -1;
    if (u->n_guide >= n) return -2;        /* the line is complete: a line-end call is due */
    if (c->budget_lines < c->n_lines && u->len - c->cond_len >= c->budget_lines * n) return -3;
    int s = u->len;
    u->pos[s] = c->cond_len + u->n_vis;
    for (int t = 0; t < d; ++t) { u->K[(size_t)s * d + t] = (double)k[t]; u->V[(size_t)s * d + t] = (double)v[t]; }
    u->len += 1;
    u->n_vis += 1;
    u->acc[s] = 0.0;                       /* a new entry has received no attention yet */
    double *qd = (double *)malloc(sizeof(double) * (size_t)d);
    double *pr = (double *)malloc(sizeof(double) * (size_t)u->len);
    for (int g = 0; g < G; ++g) {
        for (int t = 0; t < d; ++t) qd[t] = (double)q[(size_t)g * d + t];
        lar_oracle_attention(qd, u->K, u->V, u->len, d, cfg_scale(c), out + (size_t)g * d, pr);
        if (probs) memcpy(probs + (size_t)g * u->len, pr, sizeof(double) * (size_t)u->len);
        for (int j = 0; j < u->len; ++j) u->acc[j] += pr[j];   /* accumulated attention of every live entry */
        memcpy(u->guide + ((size_t)u->n_guide * G + g) * d, qd, sizeof(double) * (size_t)d);
    }
    free(pr);
    free(qd);
    u->n_guide += 1;
    return 0;
}

/* Partition of the live visual entries at the end of line l (Sec. 3.3, before Eq. 5):
 * init = visual index <= N_init, rec = visual index > (l - r) n, mid = the rest.
 * Writes the slot numbers of the mid entries (cache order) and returns their count. */
static int mid_slots(const lar_oracle_unit *u, int *slots) {
    const lar_oracle_cfg *c = &u->c;
    int l = u->n_vis / c->line_width, M = 0;
    for (int s = 0; s < u->len; ++s) {
        int p = u->pos[s];
        if (p < c->cond_len) continue;                       /* conditional prefix */
        int vi = p - c->cond_len + 1;                        /* 1-based visual index */
        if (vi <= c->anchor_len) continue;                   /* init */
        if (vi > (l - c->recent_lines) * c->line_width) continue; /* rec */
        slots[M++] = s;
    }
    return M;
}

/* Does the end of the current line compress?  1 yes, 0 no (cache below budget or never compressed),
 * -1 not at a line boundary / guide queue incomplete. */
int lar_oracle_unit_line_end_due(const lar_oracle_unit *u) {
    const lar_oracle_cfg *c = &u->c;
    if (u->n_vis == 0 || u->n_vis % c->line_width != 0 || u->n_guide != c->line_width) return -1;
    if (c->budget_lines >= c->n_lines) return 0;
    return (u->len - c->cond_len) >= c->budget_lines * c->line_width ? 1 : 0;
}

/* Scores of the mid region at a compressing line end (Eq. 8-9); does not modify the unit.
 * scores: [M] doubles, mid_pos: [M] original positions.  Returns M, or <0 if no compression is due. */
int lar_oracle_unit_mid_scores(const lar_oracle_unit *u, double *scores, int *mid_pos) {
    if (lar_oracle_unit_line_end_due(u) != 1) return -1;
    const lar_oracle_cfg *c = &u->c;
    int d = c->head_dim;
    int *slots = (int *)malloc(sizeof(int) * (size_t)u->len);
    int M = mid_slots(u, slots);
    double *Kmid = (double *)malloc(sizeof(double) * (size_t)(M > 0 ? M : 1) * (size_t)d);
    for (int m = 0; m < M; ++m) {
        memcpy(Kmid + (size_t)m * d, u->K + (size_t)slots[m] * d, sizeof(double) * (size_t)d);
        mid_pos[m] = u->pos[slots[m]];
    }
    /* all n * G guide rows contribute equally: mean over the n queries and the G heads */
    if (c->score_norm == 0)
        lar_oracle_saliency(u->guide, c->line_width * c->group, Kmid, M, d, cfg_scale(c), scores);
    else if (c->score_norm == 2)   /* the attention mass the entry has received since it was appended */
        for (int m = 0; m < M; ++m) scores[m] = u->acc[slots[m]] / (double)(c->line_width * c->group);
    else   /* query t of the line is visual token n_vis - n + t + 1, at position C + n_vis - n + t */
        lar_oracle_saliency_cache(u->guide, c->line_width, c->group, u->K, u->pos, u->len, d, cfg_scale(c),
                                  c->cond_len + u->n_vis - c->line_width, slots, M, scores);
    free(Kmid); free(slots);
    return M;
}

/* Remove the entries with the given original positions (Eq. 5-6), keep the order of the rest,
 * clear the guide queue.  All positions must lie in the mid region.  Returns 0, or <0 on error. */
int lar_oracle_unit_evict(lar_oracle_unit *u, const int *evict_pos, int n_evict) {
    const lar_oracle_cfg *c = &u->c;
    int d = c->head_dim;
    int *slots = (int *)malloc(sizeof(int) * (size_t)u->len);
    int M = mid_slots(u, slots);
    char *drop = (char *)calloc((size_t)u->len, 1);
    int rc = 0;
    for (int e = 0; e < n_evict && rc == 0; ++e) {
        int found = 0;
        for (int m = 0; m < M; ++m)
            if (u->pos[slots[m]] == evict_pos[e] && !drop[slots[m]]) { drop[slots[m]] = 1; found = 1; break; }
        if (!found) rc = -1;
    }
    if (rc == 0) {
        int w = 0;
        for (int s = 0; s < u->len; ++s) {
            if (drop[s]) continue;
            if (w != s) {
                u->pos[w] = u->pos[s];
                u->acc[w] = u->acc[s];   /* an entry keeps the attention it has accumulated */
                memcpy(u->K + (size_t)w * d, u->K + (size_t)s * d, sizeof(double) * (size_t)d);
                memcpy(u->V + (size_t)w * d, u->V + (size_t)s * d, sizeof(double) * (size_t)d);
            }
            ++w;
        }
        u->len = w;
        u->n_guide = 0;
    }
    free(drop); free(slots);
    return rc;
}

/* The whole line-end step (Sec. 3.3): gate, score, BottomK(n), compact.
 * Returns 1 if the cache was compressed, 0 if the line end was a no-op, <0 on a call-order error.
 * scores / mid_pos ([M]), evicted_pos ([n]) and boundary ([2]: lowest kept score, highest evicted
 * score) are optional outputs. */
int lar_oracle_unit_line_end(lar_oracle_unit *u, double *scores, int *mid_pos, int *evicted_pos,
                             double *boundary) {
    int due = lar_oracle_unit_line_end_due(u);
    if (due < 0) return -1;
    if (due == 0) { u->n_guide = 0; return 0; }
    const lar_oracle_cfg *c = &u->c;
    int n = c->line_width;
    double *S = (double *)malloc(sizeof(double) * (size_t)u->len);
    int *mp = (int *)malloc(sizeof(int) * (size_t)u->len);
    int *ev = (int *)malloc(sizeof(int) * (size_t)n);
    int *evp = (int *)malloc(sizeof(int) * (size_t)n);
    int M = lar_oracle_unit_mid_scores(u, S, mp);
    lar_oracle_bottomk(S, mp, M, n, ev);
    for (int e = 0; e < n; ++e) evp[e] = mp[ev[e]];
    if (boundary) {
        /* ev[n-1] is the most salient evicted entry; the least salient kept one is the next in order */
        double lowest_kept = INFINITY;
        char *is_ev = (char *)calloc((size_t)(M > 0 ? M : 1), 1);
        for (int e = 0; e < n; ++e) is_ev[ev[e]] = 1;
        for (int m = 0; m < M; ++m) if (!is_ev[m] && S[m] < lowest_kept) lowest_kept = S[m];
        free(is_ev);
        boundary[0] = lowest_kept;
        boundary[1] = S[ev[n - 1]];
    }
    if (scores) memcpy(scores, S, sizeof(double) * (size_t)M);
    if (mid_pos) memcpy(mid_pos, mp, sizeof(int) * (size_t)M);
    if (evicted_pos) memcpy(evicted_pos, evp, sizeof(int) * (size_t)n);
    int rc = lar_oracle_unit_evict(u, evp, n);
    free(S); free(mp); free(ev); free(evp);
    return rc == 0 ? 1 : -2;
}

/* ---------------------------------------------------------------------------------------------
 * Whole generations of many independent units (prefill, then for each visual token: step, and a
 * line-end call after each complete line except the last).  Units run in parallel with OpenMP.
 *   q  [U][N][G][d]   k, v [U][N][d]   kc, vc [U][C][d]          (floats)
 *   out [U][n_steps][G][d] doubles, or NULL
 *   kept_pos [U][n_line_ends][keep_stride] ints (live positions after each line end, -1 padded), or NULL
 * Returns the number of threads used, or <0 on error.
 * ------------------------------------------------------------------------------------------- */
int lar_oracle_run_units(const lar_oracle_cfg *cfg, int n_units, const float *q, const float *k,
                         const float *v, const float *kc, const float *vc, int n_steps, double *out,
                         int *kept_pos, int keep_stride, int n_threads) {
    int N = cfg->line_width * cfg->n_lines, G = cfg->group, d = cfg->head_dim, n = cfg->line_width;
    int n_line_ends = n_steps / n;
    if (n_steps > N) return -1;
    int err = 0, used = 1;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
    used = omp_get_max_threads();
#endif
    (void)n_threads;
#pragma omp parallel for schedule(dynamic, 1)
    for (int un = 0; un < n_units; ++un) {
        lar_oracle_unit *u = lar_oracle_unit_create(cfg);
        if (!u) { err = 1; continue; }
        double *o = (double *)malloc(sizeof(double) * (size_t)G * d);
        lar_oracle_unit_prefill(u, kc + (size_t)un * cfg->cond_len * d, vc + (size_t)un * cfg->cond_len * d);
        for (int i = 0; i < n_steps; ++i) {
            int rc = lar_oracle_unit_step(u, q + ((size_t)un * N + i) * G * d, k + ((size_t)un * N + i) * d,
                                          v + ((size_t)un * N + i) * d, o, NULL);
            if (rc) { err = 1; break; }
            if (out) memcpy(out + ((size_t)un * n_steps + i) * G * d, o, sizeof(double) * (size_t)G * d);
            if ((i + 1) % n == 0 && (i + 1) < N) {
                if (lar_oracle_unit_line_end(u, NULL, NULL, NULL, NULL) < 0) { err = 1; break; }
                if (kept_pos) {
                    int *dst = kept_pos + ((size_t)un * n_line_ends + (size_t)((i + 1) / n - 1)) * keep_stride;
                    for (int s = 0; s < keep_stride; ++s) dst[s] = s < u->len ? u->pos[s] : -1;
                }
            }
        }
        free(o);
        lar_oracle_unit_destroy(u);
    }
    return err ? -2 : used;
}
