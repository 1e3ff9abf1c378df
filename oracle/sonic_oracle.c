/*
 * CPU oracle for the fused sampling / speculative-verification path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what
 * the path computes, written from the paper's definitions.  It shares no code
 * with the CUDA library and must never be linked into, imported by or called
 * from the product path; only the tests, the smoke check and the benchmark's
 * CPU-baseline leg may use it.
 *
 * What it follows (paper sections / equations / algorithms):
 *   - logit processing: grammar mask, repetition / frequency / presence
 *     penalties, logit bias, temperature (Appendix "Logit Processing
 *     Operations"; order as in Algorithm "Stage 1", prologue);
 *   - truncation: top-k, then top-p by cumulative softmax over the top-k
 *     survivors, then min-p in its log-domain form x >= M + ln(theta)
 *     (Appendix "Probability Truncation", Eq. min_p_trick; order as in
 *     Algorithm "Stage 2", epilogue);
 *   - token selection: a draw from the truncated, renormalised categorical
 *     distribution (the distribution the Gumbel-max formulation of Appendix
 *     "Sampling" draws from); greedy = argmax;
 *   - speculative verification: accept iff u*q(d) <= p(d), else resample from
 *     normalise(max(0, p - q)) (Section "Speculative Verification" of the
 *     background and of the appendix);
 *   - ties go to the lowest index (the paper's packing complements the index
 *     for exactly this purpose, Section 3.4 "Numerical Lexicographic Encoding");
 *   - per-request bit indicators (Section 3.5, indicator table).
 *
 * Arithmetic: the prologue is fp32, one IEEE round-to-nearest operation per
 * operator and no fused multiply-add, because its result decides integers
 * (argmax, top-k membership) and both sides must take that decision in one
 * precision.  Everything after the ordering (softmax weights, cumulative
 * sums, CDF) is fp64.  Random numbers are Philox4x32-10 with
 * key = (seed_lo, seed_hi), counter = (pos_lo, pos_hi, request, 0).
 *
 * Readings adopted where the paper is silent are listed in the design notes of
 * the repository; each is marked "reading:" below.
 *
 * Parity pins: every exported function is pinned by tests that do not call it
 * to produce their expectations (published Philox vectors, hand-worked
 * examples, brute force on tiny vocabularies, closed forms, the exact
 * enumeration identity of rejection sampling, chi-squared on many draws).
 */
#define _GNU_SOURCE
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_GRAMMAR     0x001u
#define ORACLE_REPETITION  0x002u
#define ORACLE_FREQUENCY   0x004u
#define ORACLE_PRESENCE    0x008u
#define ORACLE_BIAS        0x010u
#define ORACLE_TEMPERATURE 0x020u
#define ORACLE_GREEDY      0x040u
#define ORACLE_TOP_K       0x080u
#define ORACLE_TOP_P       0x100u
#define ORACLE_MIN_P       0x200u

#define ORACLE_FLAG_NO_TOKEN 0x1u
#define ORACLE_FLAG_BADPARAM 0x2u

/* ------------------------------------------------------------------ Philox */
/* Philox4x32 with 10 rounds (Salmon et al., "Parallel random numbers: as easy
 * as 1, 2, 3"): multipliers 0xD2511F53 / 0xCD9E8D57, Weyl key increments
 * 0x9E3779B9 / 0xBB67AE85. */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Uniform in (0,1) from 32 random bits: the top 24 bits, centred in their
 * cell, so the value is an exact fp32 (and fp64) number. */
double oracle_u01(uint32_t r)
{
    return ((double)(r >> 8) + 0.5) * (1.0 / 16777216.0);
}

/* Draws for (seed, position, request): u_accept from word 0, u_draw from word 1. */
void oracle_uniforms(uint64_t seed, uint64_t pos, uint32_t request, double *u_accept, double *u_draw)
{
    uint32_t ctr[4] = {(uint32_t)pos, (uint32_t)(pos >> 32), request, 0u};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t r[4];
    oracle_philox4x32_10(ctr, key, r);
    *u_accept = oracle_u01(r[0]);
    *u_draw = oracle_u01(r[1]);
}

/* ---------------------------------------------------------------- prologue */
/* Logit processing for one row, in the order mask -> repetition -> frequency
 * -> presence -> bias -> temperature.  Returns nonzero if a list id is out of
 * range. */
int oracle_prologue(const float *x, int V, uint32_t z, const uint32_t *mask,
                    float alpha, float beta, float gamma,
                    const int32_t *hist_ids, const int32_t *hist_counts, int hist_len,
                    const int32_t *bias_ids, const float *bias_vals, int bias_len,
                    float tau, float *y)
{
    int bad = 0;
    for (int i = 0; i < V; ++i) y[i] = x[i];
    if (z & ORACLE_GRAMMAR) {
        for (int i = 0; i < V; ++i)
            if (((mask[i >> 5] >> (i & 31)) & 1u) == 0u) y[i] = -INFINITY;
    }
    if (z & (ORACLE_REPETITION | ORACLE_FREQUENCY | ORACLE_PRESENCE)) {
        for (int e = 0; e < hist_len; ++e) {
            int id = hist_ids[e];
            int c = hist_counts[e];
            if (id < 0 || id >= V) { bad = 1; continue; }
            if (c <= 0) continue;
            float v = y[id];
            if (z & ORACLE_REPETITION) {
                if (v > 0.0f) v = v / alpha; else v = v * alpha;
            }
            if (z & ORACLE_FREQUENCY) {
                float t = beta * (float)c;
                v = v - t;
            }
            if (z & ORACLE_PRESENCE) v = v - gamma;
            y[id] = v;
        }
    }
    if (z & ORACLE_BIAS) {
        for (int e = 0; e < bias_len; ++e) {
            int id = bias_ids[e];
            if (id < 0 || id >= V) { bad = 1; continue; }
            y[id] = y[id] + bias_vals[e];
        }
    }
    if (z & ORACLE_TEMPERATURE) {
        for (int i = 0; i < V; ++i) y[i] = y[i] / tau;
    }
    /* reading: -0 and +0 compare equal, so make them one value before ordering */
    for (int i = 0; i < V; ++i) y[i] = y[i] + 0.0f;
    return bad;
}

/* ----------------------------------------------------------------- ordering */
typedef struct { float y; int32_t idx; } item_t;

static int cmp_desc_value_asc_index(const void *pa, const void *pb)
{
    const item_t *a = (const item_t *)pa, *b = (const item_t *)pb;
    if (a->y > b->y) return -1;
    if (a->y < b->y) return 1;
    return (a->idx > b->idx) - (a->idx < b->idx);
}

/* indices ordered by (value descending, index ascending) */
static void order_row(const float *y, int V, item_t *items)
{
    for (int i = 0; i < V; ++i) { items[i].y = y[i]; items[i].idx = i; }
    qsort(items, (size_t)V, sizeof(item_t), cmp_desc_value_asc_index);
}

/* Sorted top-k of raw rows (values descending, ties to the lowest index). */
void oracle_topk(const float *logits, int B, int V, int64_t row_stride, int k,
                 float *out_vals, int32_t *out_idx)
{
    item_t *items = (item_t *)malloc(sizeof(item_t) * (size_t)V);
    float *y = (float *)malloc(sizeof(float) * (size_t)V);
    for (int b = 0; b < B; ++b) {
        const float *x = logits + (int64_t)b * row_stride;
        for (int i = 0; i < V; ++i) y[i] = x[i] + 0.0f;
        order_row(y, V, items);
        for (int j = 0; j < k; ++j) {
            out_vals[(int64_t)b * k + j] = items[j].y;
            out_idx[(int64_t)b * k + j] = items[j].idx;
        }
    }
    free(y);
    free(items);
}

/* ---------------------------------------------------------------- truncation */
typedef struct {
    int n_finite;        /* finite processed logits */
    int n;               /* survivors: the first n entries of the ordering */
    double M;            /* largest processed logit */
    double W;            /* sum of w over the survivors */
    double margin;       /* smallest relative distance of a float decision to its threshold */
} trunc_t;

/* Truncation of an ordered row.  w[j] = exp(y_j - M) for the first n_k entries.
 * TopK -> TopP (mass >= p over the top-k survivors) -> MinP (x >= M + ln theta). */
static trunc_t truncate_row(const item_t *items, int V, uint32_t z, int k, float p, float theta, double *w)
{
    trunc_t t;
    memset(&t, 0, sizeof(t));
    t.margin = INFINITY;
    int nf = 0;
    while (nf < V && isfinite(items[nf].y)) ++nf;   /* -inf sorts last */
    t.n_finite = nf;
    if (nf == 0) return t;
    int n = nf;
    if ((z & ORACLE_TOP_K) && k > 0 && k < n) n = k;
    double M = (double)items[0].y;
    t.M = M;
    double acc = 0.0;
    double *C = (double *)malloc(sizeof(double) * (size_t)n);
    for (int j = 0; j < n; ++j) {
        w[j] = exp((double)items[j].y - M);
        acc += w[j];
        C[j] = acc;
    }
    double Z = C[n - 1];
    int n_keep = n;
    /* TopP (Appendix "Probability Truncation"): the smallest ranking prefix whose mass reaches p * Z.  At p = 1 that is
     * the whole set (every weight is positive); taken literally the comparison C_j >= 1 * Z would be decided by the
     * rounding of the running sum, so p = 1 is read as "no truncation". */
    if ((z & ORACLE_TOP_P) && p < 1.0f) {
        double target = (double)p * Z;
        int np_ = n;
        for (int j = 0; j < n; ++j) {
            if (C[j] >= target) { np_ = j + 1; break; }
        }
        double m = fabs(C[np_ - 1] - target);
        if (np_ >= 2) { double m2 = fabs(C[np_ - 2] - target); if (m2 < m) m = m2; }
        if (m / Z < t.margin) t.margin = m / Z;
        if (np_ < n_keep) n_keep = np_;
    }
    if (z & ORACLE_MIN_P) {
        double thr = M + log((double)theta);
        int nm = 0;
        while (nm < n && (double)items[nm].y >= thr) ++nm;
        double m = INFINITY;
        if (nm >= 1) m = fabs((double)items[nm - 1].y - thr);
        if (nm < n) { double m2 = fabs((double)items[nm].y - thr); if (m2 < m) m = m2; }
        if (m < t.margin) t.margin = m;
        if (nm < n_keep) n_keep = nm;
    }
    t.n = n_keep;
    t.W = C[n_keep - 1];
    free(C);
    return t;
}

/* Inverse CDF in vocabulary-index order over survivors (idx[j], r[j]), j<n,
 * already sorted by index.  Returns the position of the first j with
 * F_j > u*R; margin = relative distance of u*R to the nearer bracketing F. */
static int draw_index_order(const double *r, int n, double u, double *total_out, double *margin_out)
{
    double R = 0.0;
    for (int j = 0; j < n; ++j) R += r[j];
    double target = u * R;
    double F = 0.0, Fprev = 0.0;
    int pick = n - 1;
    int found = 0;
    for (int j = 0; j < n; ++j) {
        Fprev = F;
        F += r[j];
        if (F > target) { pick = j; found = 1; break; }
    }
    if (!found) Fprev = F - r[n - 1];
    double m = fabs(F - target);
    double m2 = fabs(Fprev - target);
    if (m2 < m) m = m2;
    *total_out = R;
    *margin_out = (R > 0.0) ? m / R : 0.0;
    return pick;
}

/* -------------------------------------------------------------- parameters */
typedef struct {
    int32_t B, V;
    int32_t K;                    /* verify only */
    const float *logits;          /* [rows, row_stride] fp32 (bf16 inputs are widened exactly by the caller) */
    int64_t row_stride;
    const uint32_t *mode;
    const uint32_t *bitmask;      /* [rows, bitmask_stride] */
    int64_t bitmask_stride;
    const float *temperature;
    const int32_t *top_k;
    const float *top_p;
    const float *min_p;
    const float *rep_penalty;
    const float *freq_penalty;
    const float *pres_penalty;
    const int32_t *hist_ids;
    const int32_t *hist_counts;
    const int32_t *hist_len;
    int32_t hist_stride;
    const int32_t *bias_ids;
    const float *bias_vals;
    const int32_t *bias_len;
    int32_t bias_stride;
    const uint64_t *seed;
    const uint64_t *offset;
    const int32_t *draft_tokens;  /* [B, K] */
    const float *draft_probs;     /* [B, K, V] */
} oracle_args;

static int bad_params(const oracle_args *a, int b)
{
    uint32_t z = a->mode[b];
    if (z & ORACLE_TEMPERATURE) { float t = a->temperature[b]; if (!(t > 0.0f) || !isfinite(t)) return 1; }
    /* penalty coefficients (Appendix "Repetition Penalties": alpha >= 1, beta >= 0, gamma >= 0): a divisor that is
     * not positive and finite, or a coefficient that is not finite, is outside the domain like any other parameter */
    if (z & ORACLE_REPETITION) { float al = a->rep_penalty[b]; if (!(al > 0.0f) || !isfinite(al)) return 1; }
    if ((z & ORACLE_FREQUENCY) && !isfinite(a->freq_penalty[b])) return 1;
    if ((z & ORACLE_PRESENCE) && !isfinite(a->pres_penalty[b])) return 1;
    if (z & ORACLE_GREEDY) return 0;
    if ((z & ORACLE_TOP_K) && a->top_k[b] < 0) return 1;
    if (z & ORACLE_TOP_P) { float p = a->top_p[b]; if (!(p > 0.0f && p <= 1.0f)) return 1; }
    if (z & ORACLE_MIN_P) { float q = a->min_p[b]; if (!(q > 0.0f && q <= 1.0f)) return 1; }
    return 0;
}

/* processed logits of logit-row `row` under request b's parameters */
static int process_row(const oracle_args *a, int b, int64_t row, float *y)
{
    uint32_t z = a->mode[b];
    const float *x = a->logits + row * a->row_stride;
    const uint32_t *mask = (z & ORACLE_GRAMMAR) ? a->bitmask + row * a->bitmask_stride : NULL;
    int hl = 0, bl = 0;
    const int32_t *hi = NULL, *hc = NULL, *bi = NULL;
    const float *bv = NULL;
    if (z & (ORACLE_REPETITION | ORACLE_FREQUENCY | ORACLE_PRESENCE)) {
        hl = a->hist_len[b];
        hi = a->hist_ids + (int64_t)b * a->hist_stride;
        hc = a->hist_counts + (int64_t)b * a->hist_stride;
    }
    if (z & ORACLE_BIAS) {
        bl = a->bias_len[b];
        bi = a->bias_ids + (int64_t)b * a->bias_stride;
        bv = a->bias_vals + (int64_t)b * a->bias_stride;
    }
    return oracle_prologue(x, a->V, z, mask,
                           (z & ORACLE_REPETITION) ? a->rep_penalty[b] : 1.0f,
                           (z & ORACLE_FREQUENCY) ? a->freq_penalty[b] : 0.0f,
                           (z & ORACLE_PRESENCE) ? a->pres_penalty[b] : 0.0f,
                           hi, hc, hl, bi, bv, bl,
                           (z & ORACLE_TEMPERATURE) ? a->temperature[b] : 1.0f, y);
}

/* Exposes the processed logits of one row (used by the prologue pins). */
int oracle_processed_row(const oracle_args *a, int b, float *y)
{
    return process_row(a, b, (int64_t)b, y);
}

/* Exposes the final support of one singular-mode row: survivors in ranking
 * order with their renormalised probabilities.  Returns n (0 if no token). */
int oracle_support(const oracle_args *a, int b, int32_t *idx_out, double *prob_out, double *margin_out)
{
    int V = a->V;
    float *y = (float *)malloc(sizeof(float) * (size_t)V);
    item_t *items = (item_t *)malloc(sizeof(item_t) * (size_t)V);
    double *w = (double *)malloc(sizeof(double) * (size_t)V);
    process_row(a, b, (int64_t)b, y);
    order_row(y, V, items);
    uint32_t z = a->mode[b];
    trunc_t t = truncate_row(items, V, z, a->top_k ? a->top_k[b] : 0, a->top_p ? a->top_p[b] : 1.0f,
                             a->min_p ? a->min_p[b] : 0.0f, w);
    for (int j = 0; j < t.n; ++j) { idx_out[j] = items[j].idx; prob_out[j] = w[j] / t.W; }
    if (margin_out) *margin_out = t.margin;
    free(w); free(items); free(y);
    return t.n;
}

/* survivors (the first n entries of the ordering) rearranged in index order */
typedef struct { int32_t idx; int32_t pos; } idxpos_t;

static int cmp_idxpos(const void *pa, const void *pb)
{
    const idxpos_t *a = (const idxpos_t *)pa, *b = (const idxpos_t *)pb;
    return (a->idx > b->idx) - (a->idx < b->idx);
}

static void survivors_by_index(const item_t *items, int n, idxpos_t *ip)
{
    for (int j = 0; j < n; ++j) { ip[j].idx = items[j].idx; ip[j].pos = j; }
    qsort(ip, (size_t)n, sizeof(idxpos_t), cmp_idxpos);
}

/* ------------------------------------------------------------ singular mode */
/* One token per row.  out_margin[b] is the smallest relative distance between
 * a floating-point decision of the row (top-p cut, min-p cut, CDF draw) and
 * its threshold; rows below 1e-6 admit two outcomes. */
void oracle_sample(const oracle_args *a, int32_t *out_token, float *out_prob, uint32_t *out_flags,
                   int32_t *out_support, double *out_margin)
{
    int V = a->V;
    float *y = (float *)malloc(sizeof(float) * (size_t)V);
    item_t *items = (item_t *)malloc(sizeof(item_t) * (size_t)V);
    idxpos_t *ip = (idxpos_t *)malloc(sizeof(idxpos_t) * (size_t)V);
    double *w = (double *)malloc(sizeof(double) * (size_t)V);
    double *r = (double *)malloc(sizeof(double) * (size_t)V);
    for (int b = 0; b < a->B; ++b) {
        uint32_t z = a->mode[b];
        out_token[b] = -1; out_prob[b] = 0.0f; out_flags[b] = 0; out_support[b] = 0; out_margin[b] = INFINITY;
        int bad = bad_params(a, b);
        bad |= process_row(a, b, (int64_t)b, y);
        if (bad) { out_flags[b] = ORACLE_FLAG_BADPARAM; continue; }
        order_row(y, V, items);
        if (!isfinite(items[0].y)) { out_flags[b] = ORACLE_FLAG_NO_TOKEN; continue; }
        if (z & ORACLE_GREEDY) {       /* reading: greedy is a point mass on the argmax */
            out_token[b] = items[0].idx; out_prob[b] = 1.0f; out_support[b] = 1;
            continue;
        }
        trunc_t t = truncate_row(items, V, z, a->top_k ? a->top_k[b] : 0, a->top_p ? a->top_p[b] : 1.0f,
                                 a->min_p ? a->min_p[b] : 0.0f, w);
        survivors_by_index(items, t.n, ip);
        for (int j = 0; j < t.n; ++j) r[j] = w[ip[j].pos];
        double ua, ud, R, m;
        oracle_uniforms(a->seed[b], a->offset[b], (uint32_t)b, &ua, &ud);
        int pick = draw_index_order(r, t.n, ud, &R, &m);
        out_token[b] = ip[pick].idx;
        out_prob[b] = (float)(r[pick] / t.W);
        out_support[b] = t.n;
        out_margin[b] = (m < t.margin) ? m : t.margin;
    }
    free(r); free(w); free(ip); free(items); free(y);
}

/* ----------------------------------------------------------- multistep mode */
/* Sequential verification of K draft tokens per request against the target
 * rows [b, 0..K].  Stochastic requests: accept d_l iff p(d_l) > 0 and
 * u_l * q(d_l) <= p(d_l); at the first rejection resample from
 * normalise(max(0, p - q)) over p's support (from p itself if that sum is not
 * positive); if every draft is accepted, draw the bonus token from the last
 * row.  Greedy requests: accept while the draft equals the argmax; the
 * correction / bonus token is the argmax.  Position l uses Philox counter
 * offset + l.
 * Outputs: out_tokens [B, K+1] (accepted drafts, then the correction or bonus
 * token, then -1), out_accept_len [B], out_p_draft [B, K] = p_l(d_l) for every
 * position (whether or not it was reached), out_margin [B] over the positions
 * that decide the outputs. */
void oracle_verify(const oracle_args *a, int32_t *out_tokens, int32_t *out_accept_len, float *out_p_draft,
                   uint32_t *out_flags, double *out_margin)
{
    int V = a->V, K = a->K;
    float *y = (float *)malloc(sizeof(float) * (size_t)V);
    item_t *items = (item_t *)malloc(sizeof(item_t) * (size_t)V);
    idxpos_t *ip = (idxpos_t *)malloc(sizeof(idxpos_t) * (size_t)V);
    double *w = (double *)malloc(sizeof(double) * (size_t)V);
    double *r = (double *)malloc(sizeof(double) * (size_t)V);
    for (int b = 0; b < a->B; ++b) {
        uint32_t z = a->mode[b];
        int32_t *toks = out_tokens + (int64_t)b * (K + 1);
        for (int l = 0; l <= K; ++l) toks[l] = -1;
        for (int l = 0; l < K; ++l) out_p_draft[(int64_t)b * K + l] = 0.0f;
        out_accept_len[b] = 0; out_flags[b] = 0; out_margin[b] = INFINITY;
        if (bad_params(a, b)) { out_flags[b] = ORACLE_FLAG_BADPARAM; continue; }
        int decided = 0;      /* set once the correction token has been emitted */
        int acc = 0;
        uint32_t flags = 0;
        for (int l = 0; l <= K; ++l) {
            int64_t row = (int64_t)b * (K + 1) + l;
            if (process_row(a, b, row, y)) { flags |= ORACLE_FLAG_BADPARAM; }
            order_row(y, V, items);
            int d = (l < K) ? a->draft_tokens[(int64_t)b * K + l] : -1;
            if (!isfinite(items[0].y)) {
                if (!decided) { flags |= ORACLE_FLAG_NO_TOKEN; decided = 1; }   /* token stays -1 */
                continue;
            }
            if (z & ORACLE_GREEDY) {
                int g = items[0].idx;
                if (l < K) out_p_draft[(int64_t)b * K + l] = (d == g) ? 1.0f : 0.0f;
                if (decided) continue;
                if (l < K && d == g) { toks[l] = d; acc = l + 1; }
                else { toks[l] = g; decided = 1; }
                continue;
            }
            trunc_t t = truncate_row(items, V, z, a->top_k ? a->top_k[b] : 0, a->top_p ? a->top_p[b] : 1.0f,
                                     a->min_p ? a->min_p[b] : 0.0f, w);
            survivors_by_index(items, t.n, ip);
            double ua, ud;
            oracle_uniforms(a->seed[b], a->offset[b] + (uint64_t)l, (uint32_t)b, &ua, &ud);
            double margin = t.margin;
            double P = 0.0;
            if (l < K) {
                for (int j = 0; j < t.n; ++j)
                    if (ip[j].idx == d) { P = w[ip[j].pos] / t.W; break; }
                out_p_draft[(int64_t)b * K + l] = (float)P;
            }
            if (decided) continue;
            if (l < K) {
                double Q = (double)a->draft_probs[((int64_t)b * K + l) * V + d];
                double lhs = ua * Q;
                int accept = (P > 0.0) && (lhs <= P);
                double den = (P > lhs) ? P : lhs;
                if (den > 0.0) { double m = fabs(lhs - P) / den; if (m < margin) margin = m; }
                if (accept) {
                    toks[l] = d; acc = l + 1;
                    if (margin < out_margin[b]) out_margin[b] = margin;
                    continue;
                }
                /* residual over the support of p, in index order */
                const float *q = a->draft_probs + ((int64_t)b * K + l) * V;
                double R = 0.0;
                for (int j = 0; j < t.n; ++j) {
                    double pj = w[ip[j].pos] / t.W;
                    double rj = pj - (double)q[ip[j].idx];
                    r[j] = (rj > 0.0) ? rj : 0.0;
                    R += r[j];
                }
                if (!(R > 0.0))
                    for (int j = 0; j < t.n; ++j) r[j] = w[ip[j].pos] / t.W;
            } else {
                for (int j = 0; j < t.n; ++j) r[j] = w[ip[j].pos];
            }
            double Rt, m;
            int pick = draw_index_order(r, t.n, ud, &Rt, &m);
            if (m < margin) margin = m;
            toks[l] = ip[pick].idx;
            decided = 1;
            if (margin < out_margin[b]) out_margin[b] = margin;
        }
        out_accept_len[b] = acc;
        out_flags[b] = flags;
        if (flags & ORACLE_FLAG_BADPARAM) {
            for (int l = 0; l <= K; ++l) toks[l] = -1;
            out_accept_len[b] = 0;
        }
    }
    free(r); free(w); free(ip); free(items); free(y);
}
