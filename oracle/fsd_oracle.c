/*
 * fsd_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, double-precision CPU statement of the verification step of
 * Fuzzy Speculative Decoding (FSD) and of strict speculative sampling (SD),
 * written from the paper's definitions.  It exists only so that tests, the
 * smoke check and the benchmark's CPU-baseline leg have something independent
 * to compare the CUDA library with.  It shares no code with the CUDA path and
 * nothing in the product may call it.
 *
 * What each function follows:
 *   softmax of a logit row ............ Section 4 ("next token distributions at
 *                                       candidate position i")
 *   KL(P_T || P_D), JS, TV ............ Appendix C.1, C.2, C.3, term by term
 *   SD acceptance probability/rule .... Section 3, Eq. 1 and Eq. 2
 *   SD resampling distribution ........ Section 3, Eq. 3 (read as the positive
 *                                       part of P_T - P_D, renormalised)
 *   FSD acceptance rule ............... Section 4, Eq. 4 (Div < T; "<=" selectable)
 *   FSD rejection sampling ............ Section 4 (sample from P_T at the rejected
 *                                       position)
 *   rFSD .............................. Section 4.3, Eq. 6
 *   greedy choice on rejection ........ Section 6.3
 *   tree drafts ....................... Section 6.4 gives no algorithm; the reading
 *                                       used is stated at fsd_oracle_tree below
 *
 * Parity status: every function here is pinned by tests against hand-computed
 * values, closed forms, invariants and brute-force enumeration.  The paper's
 * measured acceptance rates and accuracies depend on model weights and
 * datasets: for those, parity unpinned.
 *
 * Summation: every sum over the vocabulary runs in index order with Neumaier
 * compensation.  Logarithms are natural (divergences in nats).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_F32 = 0, ORC_BF16 = 1 };
enum { ORC_DIV_JS = 0, ORC_DIV_KL = 1, ORC_DIV_TV = 2 };
enum { ORC_MODE_FSD = 0, ORC_MODE_SD = 1, ORC_MODE_RFSD = 2 };
enum { ORC_CMP_LT = 0, ORC_CMP_LE = 1 };
enum { ORC_SAMPLE_INVCDF = 0, ORC_SAMPLE_GREEDY = 1 };
enum { ORC_ST_NONFINITE = 1, ORC_ST_BADTREE = 4 };

/* ---- compensated running sum ------------------------------------------- */
typedef struct { double s, c; } ksum;
static void ks_add(ksum *k, double x) {
    double t = k->s + x;
    if (fabs(k->s) >= fabs(x)) k->c += (k->s - t) + x;
    else                       k->c += (x - t) + k->s;
    k->s = t;
}
static double ks_val(const ksum *k) { return k->s + k->c; }

/* ---- exact widening of a stored logit ------------------------------------ */
static double widen(const void *base, size_t idx, int dtype) {
    if (dtype == ORC_BF16) {
        uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return (double)((const float *)base)[idx];
}
static const void *row_ptr(const void *base, size_t row, int V, int dtype) {
    size_t es = dtype == ORC_BF16 ? 2 : 4;
    return (const char *)base + row * (size_t)V * es;
}

/* ---- softmax (Section 4): p_k = exp(a_k - A) / sum_j exp(a_j - A) ---------
 * -inf logits are allowed (probability 0).  Returns 0, or ORC_ST_NONFINITE when
 * the row holds a NaN, a +inf or no finite entry; p is then filled with NaN. */
int fsd_oracle_softmax(const void *logits, int V, int dtype, double *p) {
    double A = -INFINITY;
    int bad = 0;
    for (int k = 0; k < V; ++k) {
        double a = widen(logits, (size_t)k, dtype);
        if (isnan(a) || a == INFINITY) bad = 1;
        if (a > A) A = a;
    }
    if (A == -INFINITY) bad = 1;
    if (bad) {
        for (int k = 0; k < V; ++k) p[k] = NAN;
        return ORC_ST_NONFINITE;
    }
    ksum Z = {0.0, 0.0};
    for (int k = 0; k < V; ++k) {
        double a = widen(logits, (size_t)k, dtype);
        p[k] = (a == -INFINITY) ? 0.0 : exp(a - A);
        ks_add(&Z, p[k]);
    }
    double z = ks_val(&Z);
    for (int k = 0; k < V; ++k) p[k] /= z;
    return 0;
}

/* ---- divergences on probability vectors (Appendix C) ---------------------- */
static double kl_terms(const double *p, const double *q, int V) {
    /* sum_k p_k ln(p_k / q_k), with 0 ln(0/.) = 0 and +inf when p_k > 0 = q_k */
    ksum s = {0.0, 0.0};
    for (int k = 0; k < V; ++k) {
        if (p[k] > 0.0) {
            if (q[k] <= 0.0) return INFINITY;
            ks_add(&s, p[k] * log(p[k] / q[k]));
        }
    }
    return ks_val(&s);
}

double fsd_oracle_divergence_probs(const double *p, const double *q, int V, int kind) {
    double d;
    if (kind == ORC_DIV_KL) {
        d = kl_terms(p, q, V);                               /* App. C.1 : KL(P_T || P_D) */
    } else if (kind == ORC_DIV_JS) {                         /* App. C.2 */
        double *m = (double *)malloc((size_t)V * sizeof(double));
        for (int k = 0; k < V; ++k) m[k] = 0.5 * (p[k] + q[k]);
        d = 0.5 * kl_terms(p, m, V) + 0.5 * kl_terms(q, m, V);
        free(m);
    } else {                                                 /* App. C.3 */
        ksum s = {0.0, 0.0};
        for (int k = 0; k < V; ++k) ks_add(&s, fabs(p[k] - q[k]));
        d = 0.5 * ks_val(&s);
    }
    if (d < 0.0) d = 0.0;                                    /* rounding can leave -1e-17 */
    return d;
}

/* divergence between softmax(target row) and softmax(draft row); NaN if either is non-finite */
double fsd_oracle_divergence_logits(const void *a, const void *b, int V, int dtype, int kind, int *status) {
    double *p = (double *)malloc((size_t)V * sizeof(double));
    double *q = (double *)malloc((size_t)V * sizeof(double));
    int st = fsd_oracle_softmax(a, V, dtype, p) | fsd_oracle_softmax(b, V, dtype, q);
    double d = st ? NAN : fsd_oracle_divergence_probs(p, q, V, kind);
    if (status) *status = st;
    free(p);
    free(q);
    return d;
}

/* ---- SD acceptance probability (Section 3, Eq. 1) -------------------------- */
double fsd_oracle_sd_accept_prob(double p_x, double q_x) {
    if (q_x <= 0.0) return p_x > 0.0 ? 1.0 : 0.0;
    double r = p_x / q_x;
    return r < 1.0 ? r : 1.0;
}

/* ---- token choice from non-negative weights w[0..V) ------------------------
 * Inverse CDF in vocabulary order: W = sum w, t = u*W, token = smallest k with
 * sum_{j<=k} w_j > t; if rounding leaves none (u close to 1), the largest k
 * with w_k > 0.  Also reports the distance of t from the nearer edge of the
 * chosen token's CDF interval, relative to W, and the tokens chosen for
 * t -/+ band*W (the set of tokens a summation-order difference of relative size
 * `band` could legitimately select).  Returns -1 when W is not positive. */
static int pick_at(const double *w, int V, double t) {
    ksum c = {0.0, 0.0};
    int last_pos = -1;
    for (int k = 0; k < V; ++k) {
        if (w[k] > 0.0) last_pos = k;
        ks_add(&c, w[k]);
        if (w[k] > 0.0 && ks_val(&c) > t) return k;
    }
    return last_pos;
}

int fsd_oracle_sample(const double *w, int V, double u, double band,
                      int *tok_lo, int *tok_hi, double *margin) {
    ksum tot = {0.0, 0.0};
    for (int k = 0; k < V; ++k) ks_add(&tot, w[k]);
    double W = ks_val(&tot);
    if (!(W > 0.0)) {
        if (tok_lo) *tok_lo = -1;
        if (tok_hi) *tok_hi = -1;
        if (margin) *margin = NAN;
        return -1;
    }
    double t = u * W;
    int tok = pick_at(w, V, t);
    if (margin) {
        ksum c = {0.0, 0.0};
        double below = 0.0;
        for (int k = 0; k < tok; ++k) ks_add(&c, w[k]);
        below = ks_val(&c);
        ks_add(&c, w[tok]);
        double lo = t - below, hi = ks_val(&c) - t;
        *margin = (lo < hi ? lo : hi) / W;
    }
    if (tok_lo) { double tl = t - band * W; *tok_lo = pick_at(w, V, tl < 0.0 ? 0.0 : tl); }
    if (tok_hi) *tok_hi = pick_at(w, V, t + band * W);
    return tok;
}

/* greedy choice (Section 6.3): index of the largest weight, ties to the lowest index */
int fsd_oracle_argmax(const double *w, int V) {
    int best = -1;
    double bv = 0.0;
    for (int k = 0; k < V; ++k)
        if (w[k] > bv) { bv = w[k]; best = k; }
    return best;
}

/* ---- replacement / bonus token ---------------------------------------------
 * residual == 0: weights are P_T of the row (FSD rejection, Section 4; and the
 * bonus row when every candidate was accepted).
 * residual == 1: weights are max(0, P_T - P_D) (Section 3, Eq. 3); if that has no
 * mass, or the draft row is non-finite, P_T is used.
 * Returns the token, or -1 when the target row is non-finite. */
static int draw_token(const void *a_row, const void *b_row, int V, int dtype, int residual,
                      int sample_kind, double u, double band,
                      int *tok_lo, int *tok_hi, double *margin, int *status) {
    double *p = (double *)malloc((size_t)V * sizeof(double));
    double *w = p;
    double *q = NULL;
    int tok;
    int st = fsd_oracle_softmax(a_row, V, dtype, p);
    if (st) {
        *status |= st;
        if (tok_lo) *tok_lo = -1;
        if (tok_hi) *tok_hi = -1;
        if (margin) *margin = NAN;
        free(p);
        return -1;
    }
    if (residual) {
        q = (double *)malloc((size_t)V * sizeof(double));
        int sq = fsd_oracle_softmax(b_row, V, dtype, q);
        *status |= sq;
        if (!sq) {
            ksum tot = {0.0, 0.0};
            for (int k = 0; k < V; ++k) {
                double r = p[k] - q[k];
                q[k] = r > 0.0 ? r : 0.0;
                ks_add(&tot, q[k]);
            }
            if (ks_val(&tot) > 0.0) w = q;
        }
    }
    if (sample_kind == ORC_SAMPLE_GREEDY) {
        tok = fsd_oracle_argmax(w, V);
        if (tok_lo) *tok_lo = tok;
        if (tok_hi) *tok_hi = tok;
        if (margin) *margin = 1.0;
    } else {
        tok = fsd_oracle_sample(w, V, u, band, tok_lo, tok_hi, margin);
    }
    free(p);
    free(q);
    return tok;
}

static int passes(double D, double T, int cmp) {
    if (isnan(D)) return 0;
    return cmp == ORC_CMP_LE ? (D <= T) : (D < T);
}

/* per-(row, position) quantities: divergence, SD acceptance probability, accept bit */
static void judge_pair(const void *a_row, const void *b_row, int V, int dtype, int div, int mode, int cmp,
                       double T, const int32_t *token, const float *u_acc,
                       double *D_out, double *pacc_out, int8_t *bit_out, int *status) {
    double *p = (double *)malloc((size_t)V * sizeof(double));
    double *q = (double *)malloc((size_t)V * sizeof(double));
    int st = fsd_oracle_softmax(a_row, V, dtype, p) | fsd_oracle_softmax(b_row, V, dtype, q);
    double D = st ? NAN : fsd_oracle_divergence_probs(p, q, V, div);
    double pacc = NAN;
    int ratio_ok = 0;
    if (!st && token && *token >= 0 && *token < V) {
        pacc = fsd_oracle_sd_accept_prob(p[*token], q[*token]);          /* Eq. 1 */
        if (u_acc) ratio_ok = (pacc > (double)*u_acc);                   /* Eq. 2 */
    }
    int bit;
    if (mode == ORC_MODE_FSD)      bit = passes(D, T, cmp);             /* Eq. 4 */
    else if (mode == ORC_MODE_SD)  bit = !st && ratio_ok;               /* Eq. 2 */
    else                           bit = passes(D, T, cmp) || (!st && ratio_ok); /* Eq. 6 */
    *D_out = D;
    if (pacc_out) *pacc_out = pacc;
    *bit_out = (int8_t)bit;
    *status = st;
    free(p);
    free(q);
}

/* ---- chain verification -------------------------------------------------------
 * target [B, gamma+1, V], draft [B, gamma, V] (row-major, dtype F32 or BF16),
 * draft_tokens [B, gamma] and u_accept [B, gamma] (needed unless mode == FSD),
 * u_sample [B].  forced (nullable) [B, gamma]: -1 leaves the accept bit alone, 0/1
 * overrides it (used to replay a decision that fell inside the threshold band).
 * Outputs (each nullable except accept_len/next_token): accept_len [B] = index of
 * the first rejected position or gamma; next_token [B]; divergence [B, gamma];
 * p_accept [B, gamma]; accept_bits [B, gamma]; tok_lo/tok_hi/margin [B];
 * row_status [B].  The row after the last candidate (row gamma) supplies the bonus
 * token when every candidate is accepted. */
int fsd_oracle_chain(const void *target, const void *draft, const int32_t *draft_tokens,
                     const float *u_accept, const float *u_sample,
                     int B, int gamma, int V, int dtype, int div, int mode, int cmp, int sample_kind,
                     double T, double band, const int8_t *forced,
                     int32_t *accept_len, int32_t *next_token, double *divergence, double *p_accept,
                     int8_t *accept_bits, int32_t *tok_lo, int32_t *tok_hi, double *margin,
                     int32_t *row_status, int nthreads) {
    if (B < 1 || gamma < 1 || V < 1) return -1;
    if (mode != ORC_MODE_FSD && (!draft_tokens || !u_accept)) return -2;
    size_t items = (size_t)B * (size_t)gamma;
    double *D = (double *)malloc(items * sizeof(double));
    int8_t *bits = (int8_t *)malloc(items);
    int *ist = (int *)malloc(items * sizeof(int));
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#else
    (void)nthreads;
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (long it = 0; it < (long)items; ++it) {
        int b = (int)(it / gamma), i = (int)(it % gamma);
        judge_pair(row_ptr(target, (size_t)b * (gamma + 1) + i, V, dtype),
                   row_ptr(draft, (size_t)b * gamma + i, V, dtype), V, dtype, div, mode, cmp, T,
                   draft_tokens ? draft_tokens + it : NULL, u_accept ? u_accept + it : NULL,
                   &D[it], p_accept ? &p_accept[it] : NULL, &bits[it], &ist[it]);
        if (forced && forced[it] >= 0) bits[it] = forced[it];
    }
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        int st = 0;
        int n = gamma;                                         /* first rejection, Section 3 */
        for (int i = 0; i < gamma; ++i) st |= ist[(size_t)b * gamma + i];
        for (int i = 0; i < gamma; ++i)
            if (!bits[(size_t)b * gamma + i]) { n = i; break; }
        int residual = (mode != ORC_MODE_FSD) && (n < gamma);
        int lo, hi;
        double mg;
        int tok = draw_token(row_ptr(target, (size_t)b * (gamma + 1) + n, V, dtype),
                             residual ? row_ptr(draft, (size_t)b * gamma + n, V, dtype) : NULL,
                             V, dtype, residual, sample_kind, (double)u_sample[b], band, &lo, &hi, &mg, &st);
        accept_len[b] = n;
        next_token[b] = tok;
        if (tok_lo) tok_lo[b] = lo;
        if (tok_hi) tok_hi[b] = hi;
        if (margin) margin[b] = mg;
        if (row_status) row_status[b] = st;
    }
    if (divergence) memcpy(divergence, D, items * sizeof(double));
    if (accept_bits) memcpy(accept_bits, bits, items);
    free(D);
    free(bits);
    free(ist);
    return 0;
}

/* ---- tree verification ----------------------------------------------------------
 * The paper applies FSD to EAGLE-2 draft trees (Section 6.4) without stating the
 * rule.  Reading used here: node j was proposed from its parent's context, so it
 * passes iff Div(P_T[row parent(j)+1], P_D[row j]) cmp T; a node lies on an accepted
 * path iff it and all its ancestors pass; the result is the deepest such node (ties:
 * lowest node index; nodes deeper than max_depth are not eligible), the path from
 * the root to it, and a next token drawn from the target row after that node (row 0
 * when nothing was accepted).  parent[j] = -1 marks a child of the root and
 * parent[j] < j must hold; a row violating it gets ORC_ST_BADTREE, accept_len 0,
 * next_token -1 and a path of -1.  Only FSD mode is defined for trees. */
int fsd_oracle_tree(const void *target, const void *draft, const int32_t *parent, const float *u_sample,
                    int B, int N, int V, int max_depth, int dtype, int div, int cmp, int sample_kind,
                    double T, double band, const int8_t *forced,
                    int32_t *accept_len, int32_t *path, int32_t *next_token, double *divergence,
                    int8_t *accept_bits, int32_t *end_node, int32_t *tok_lo, int32_t *tok_hi,
                    double *margin, int32_t *row_status, int nthreads) {
    if (B < 1 || N < 1 || V < 1 || max_depth < 1) return -1;
    size_t items = (size_t)B * (size_t)N;
    double *D = (double *)malloc(items * sizeof(double));
    int8_t *bits = (int8_t *)malloc(items);
    int *ist = (int *)malloc(items * sizeof(int));
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#else
    (void)nthreads;
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (long it = 0; it < (long)items; ++it) {
        int b = (int)(it / N), j = (int)(it % N);
        int par = parent[it];
        if (par < -1 || par >= j) { D[it] = NAN; bits[it] = 0; ist[it] = ORC_ST_BADTREE; continue; }
        judge_pair(row_ptr(target, (size_t)b * (N + 1) + (size_t)(par + 1), V, dtype),
                   row_ptr(draft, (size_t)b * N + j, V, dtype), V, dtype, div, ORC_MODE_FSD, cmp, T,
                   NULL, NULL, &D[it], NULL, &bits[it], &ist[it]);
        if (forced && forced[it] >= 0) bits[it] = forced[it];
    }
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        const int32_t *par = parent + (size_t)b * N;
        int st = 0;
        for (int j = 0; j < N; ++j) st |= ist[(size_t)b * N + j];
        int32_t *pth = path ? path + (size_t)b * max_depth : NULL;
        if (pth) for (int d = 0; d < max_depth; ++d) pth[d] = -1;
        if (st & ORC_ST_BADTREE) {
            accept_len[b] = 0;
            next_token[b] = -1;
            if (end_node) end_node[b] = -1;
            if (tok_lo) tok_lo[b] = -1;
            if (tok_hi) tok_hi[b] = -1;
            if (margin) margin[b] = NAN;
            if (row_status) row_status[b] = st;
            continue;
        }
        int *depth = (int *)malloc((size_t)N * sizeof(int));
        int8_t *ok = (int8_t *)malloc((size_t)N);
        int best = -1, best_depth = 0;
        for (int j = 0; j < N; ++j) {
            int p = par[j];
            depth[j] = p < 0 ? 1 : depth[p] + 1;
            ok[j] = (int8_t)(bits[(size_t)b * N + j] && (p < 0 || ok[p]));
            if (ok[j] && depth[j] <= max_depth && depth[j] > best_depth) { best = j; best_depth = depth[j]; }
        }
        if (pth) for (int j = best, d = best_depth - 1; j >= 0; j = par[j], --d) pth[d] = j;
        int lo, hi;
        double mg;
        int tok = draw_token(row_ptr(target, (size_t)b * (N + 1) + (size_t)(best + 1), V, dtype), NULL,
                             V, dtype, 0, sample_kind, (double)u_sample[b], band, &lo, &hi, &mg, &st);
        accept_len[b] = best_depth;
        next_token[b] = tok;
        if (end_node) end_node[b] = best;
        if (tok_lo) tok_lo[b] = lo;
        if (tok_hi) tok_hi[b] = hi;
        if (margin) margin[b] = mg;
        if (row_status) row_status[b] = st;
        free(depth);
        free(ok);
    }
    if (divergence) memcpy(divergence, D, items * sizeof(double));
    if (accept_bits) memcpy(accept_bits, bits, items);
    free(D);
    free(bits);
    free(ist);
    return 0;
}

int fsd_oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
