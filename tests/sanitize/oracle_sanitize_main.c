/* Driver for an AddressSanitizer / UndefinedBehaviorSanitizer build of the CPU oracle (test infrastructure):
 * exercises every exported function on small seeded inputs, including the edge rows (no finite logit, bad
 * parameters, out-of-range list ids, ragged sizes).  Built and run by tests/test_oracle_sanitizers.py; a
 * sanitizer report makes it exit non-zero. */
#include "../../oracle/sonic_oracle.c"
#include <stdio.h>

static uint32_t lcg(uint32_t *s) { *s = *s * 1664525u + 1013904223u; return *s; }
static float frand(uint32_t *s) { return (float)(lcg(s) >> 8) / 16777216.0f * 8.0f - 4.0f; }

int main(void)
{
    uint32_t s = 12345u;
    const int B = 6, K = 2, V = 77, H = 5, L = 3;
    const int rows = B * (K + 1);
    float *logits = malloc(sizeof(float) * rows * V);
    for (int i = 0; i < rows * V; ++i) logits[i] = frand(&s);
    for (int i = 0; i < V; ++i) logits[3 * V + i] = -INFINITY;               /* a row without a finite logit */
    uint32_t mode[6] = {ORACLE_GREEDY, ORACLE_TEMPERATURE | ORACLE_TOP_K | ORACLE_TOP_P, ORACLE_TOP_P | ORACLE_MIN_P,
                        ORACLE_GRAMMAR | ORACLE_REPETITION | ORACLE_FREQUENCY | ORACLE_PRESENCE | ORACLE_BIAS,
                        ORACLE_TEMPERATURE, ORACLE_TOP_K};
    const int W = (V + 31) / 32;
    uint32_t *mask = malloc(sizeof(uint32_t) * rows * W);
    for (int i = 0; i < rows * W; ++i) mask[i] = lcg(&s) | 1u;
    float temperature[6] = {1.0f, 0.7f, 1.0f, 1.0f, -1.0f /* bad */, 1.0f};
    int32_t top_k[6] = {0, 5, 0, 0, 0, 1000 /* above V */};
    float top_p[6] = {1.0f, 0.9f, 0.5f, 1.0f, 1.0f, 1.0f};
    float min_p[6] = {0.0f, 0.0f, 0.1f, 0.0f, 0.0f, 0.0f};
    float rep[6] = {1, 1, 1, 1.3f, 1, 1}, freq[6] = {0, 0, 0, 0.2f, 0, 0}, pres[6] = {0, 0, 0, 0.1f, 0, 0};
    int32_t hist_ids[6 * 5], hist_counts[6 * 5], hist_len[6] = {0, 0, 0, 5, 0, 0};
    for (int i = 0; i < B * H; ++i) { hist_ids[i] = (int32_t)(lcg(&s) % V); hist_counts[i] = (int32_t)(lcg(&s) % 3); }
    hist_ids[3 * H + 4] = V + 9;                                              /* out of range: BADPARAM */
    int32_t bias_ids[6 * 3], bias_len[6] = {0, 0, 0, 3, 0, 0};
    float bias_vals[6 * 3];
    for (int i = 0; i < B * L; ++i) { bias_ids[i] = (int32_t)(lcg(&s) % V); bias_vals[i] = frand(&s); }
    uint64_t seed[6] = {0, 1, 2, 3, 4, 5}, offset[6] = {0, 10, 20, 30, 40, 0xFFFFFFFFFFFFFFF0ull};
    int32_t drafts[6 * 2];
    float *q = malloc(sizeof(float) * B * K * V);
    for (int i = 0; i < B * K; ++i) drafts[i] = (int32_t)(lcg(&s) % V);
    for (int i = 0; i < B * K * V; ++i) q[i] = 1.0f / V;

    oracle_args a;
    memset(&a, 0, sizeof(a));
    a.B = B; a.V = V; a.K = 0; a.logits = logits; a.row_stride = V; a.mode = mode; a.bitmask = mask; a.bitmask_stride = W;
    a.temperature = temperature; a.top_k = top_k; a.top_p = top_p; a.min_p = min_p;
    a.rep_penalty = rep; a.freq_penalty = freq; a.pres_penalty = pres;
    a.hist_ids = hist_ids; a.hist_counts = hist_counts; a.hist_len = hist_len; a.hist_stride = H;
    a.bias_ids = bias_ids; a.bias_vals = bias_vals; a.bias_len = bias_len; a.bias_stride = L;
    a.seed = seed; a.offset = offset;
    int32_t tok[6], sup[6]; float prob[6]; uint32_t flags[6]; double margin[6];
    oracle_sample(&a, tok, prob, flags, sup, margin);
    int32_t idx[77]; double pr[77]; double m;
    int n = oracle_support(&a, 1, idx, pr, &m);
    float y[77];
    oracle_processed_row(&a, 3, y);
    a.K = K; a.draft_tokens = drafts; a.draft_probs = q;
    int32_t toks[6 * 3], acc[6]; float pd[6 * 2];
    oracle_verify(&a, toks, acc, pd, flags, margin);
    float vals[6 * 7]; int32_t ti[6 * 7];
    oracle_topk(logits, B, V, V, 7, vals, ti);
    oracle_topk(logits, 1, 1, 1, 1, vals, ti);
    uint32_t ctr[4] = {1, 2, 3, 4}, key[2] = {5, 6}, out[4];
    oracle_philox4x32_10(ctr, key, out);
    double ua, ud;
    oracle_uniforms(~0ull, ~0ull, 0xFFFFFFFFu, &ua, &ud);
    printf("ok %d %d %d %u %f\n", tok[0], n, acc[1], out[0], ua + ud + oracle_u01(0));
    free(q); free(mask); free(logits);
    return 0;
}
