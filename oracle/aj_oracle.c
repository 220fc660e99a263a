/*
 * CPU oracle for the AutoJudge verify-and-judge step.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the plain definition of what one speculation cycle's verification
 * computes, written as slow fp64 loops.  It exists to check the CUDA library and to
 * be timed as a reported CPU baseline.  It shares no code, header, table or helper
 * with the CUDA path and must never be called from it; only the tests, the smoke
 * check and the benchmark's cpu-baseline / reference arms may load it.
 *
 * What is computed, per sequence b (sequences are independent), with K draft tokens
 * and K+1 rows of hidden states (row 0 encodes the last accepted token, row i+1
 * encodes draft token i):
 *
 *   1. logit[j][v] = sum_k h_target[b][j][k] * W[k][v]             (LM head: the target
 *      model's "forward ... outputs next token logits", Section 3.1)
 *   2. y[j] = argmax_v logit[j][v]                                 (greedy target token;
 *      Section 2 footnote on greedy verification, Algorithm 1 ".argmax(-1)")
 *   3. position i mismatches when draft_tok[i] != y[i]             (the set I(x), Section 3.1)
 *   4. at a mismatch the classifier is consulted: z = b + w . [h_draft[i+1] ; h_target[i+1]],
 *      p = sigmoid(z) = P(important); the mismatch is forgiven iff p < tau
 *      (Section 3.2 design choices 1-3, "Classifier model & training"; Section 3.3 Inference)
 *   5. accept_len = number of leading positions that match or are forgiven; the first
 *      unforgiven mismatch and everything after it are rejected (Section 2), and
 *      next_tok = y[accept_len] (the target's own token there; y[K] if all K pass).
 *
 * Readings where the paper is silent: lowest index wins argmax ties; p < tau is strict;
 * tau <= 0 never forgives and tau >= 1 always forgives; feature order is [draft ; target];
 * the comparison p < tau is taken on p rounded to fp32 (the precision the kernel decides in).
 *
 * Variant without the extra row (Section 3.2, design choice 1, the second way to handle the
 * last window token): only K rows of hidden states are given, so the states that encode the last
 * draft token do not exist; a mismatch at the last position is then rejected without consulting
 * the classifier, and when all K positions pass there is no row to predict a further token from
 * (next_tok = -1).
 *
 * Sampling (Appendix A, "Generalization to sampling"): the target's token is drawn by the Gumbel-max
 * trick, token = argmax_v (logit[v] + T * g[v]) with g standard Gumbel noise that is a deterministic
 * function of a random state, so that the draw is reproducible; with temperature T this samples from
 * softmax(logit / T).  The noise for row j (row index within the call), vocabulary entry v, cycle
 * counter `step` and 64-bit `seed` is defined here as: x = word (j mod 4) of Philox4x32-10 with key
 * (seed low, seed high) and counter (v, j div 4, step low, step high); u = ((x >> 9) + 0.5) * 2^-23;
 * g = -ln(-ln(u)).  Everything downstream (mismatch test, classifier, prefix walk) uses the drawn
 * token in place of the greedy one.  T = 0 is greedy verification.
 *
 * Top-K rule (Section 4.1, the lossy baseline the paper compares with): instead of consulting the
 * classifier, a mismatching draft token is accepted iff it is among the top_k most likely tokens of
 * the target, i.e. iff its rank (number of vocabulary entries with a larger logit; among equal
 * logits the lower index ranks first) is below top_k.  A draft token outside the vocabulary is
 * never accepted.  See ajo_verify_topk.
 *
 * All inputs are converted exactly to double; every sum is accumulated in double.
 *
 * parity pins: see tests/test_oracle_pins.py (library matmul special case, one-hot
 * closed forms, tau extremes, monotonicity, brute force over pass patterns, closed-form
 * expectation of accept_len).  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { AJO_BF16 = 0, AJO_F32 = 1 };
enum { AJO_W_VD = 0, AJO_W_DV = 1 };

/* exact widening of one stored element to double */
static double elem_to_double(const void *base, size_t idx, int dtype)
{
    if (dtype == AJO_BF16) {
        uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return (double)((const float *)base)[idx];
}

int ajo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", 2011) */
void ajo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; r++) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1, n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* the uniform variate in (0,1) behind the noise of (row j, entry v): exactly representable in fp32 */
double ajo_noise_uniform(uint64_t seed, uint64_t step, int j, int v)
{
    uint32_t ctr[4] = {(uint32_t)v, (uint32_t)(j >> 2), (uint32_t)step, (uint32_t)(step >> 32)};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)}, out[4];
    ajo_philox4x32_10(ctr, key, out);
    return ((double)(out[j & 3] >> 9) + 0.5) * (1.0 / 8388608.0);
}

/* standard Gumbel noise of (row j, entry v) */
double ajo_gumbel(uint64_t seed, uint64_t step, int j, int v)
{
    return -log(-log(ajo_noise_uniform(seed, step, j, v)));
}

/*
 * Step 1 for R rows: logits[r][v] = sum_k h[r][k] * W[k][v], r < R, v < V.
 * h: R x d row-major; W: [V,d] row-major (w_layout 0) or [d,V] row-major (w_layout 1).
 * logits: R x V doubles, caller-allocated.
 */
int ajo_logits(const void *h, const void *W, int dtype, int w_layout,
               int R, int d, int V, double *logits)
{
    if (!h || !W || !logits || R < 0 || d < 1 || V < 1) return 1;
    double *hd = (double *)malloc((size_t)(R > 0 ? R : 1) * d * sizeof(double));
    if (!hd) return 2;
    for (size_t i = 0; i < (size_t)R * d; i++) hd[i] = elem_to_double(h, i, dtype);

    int failed = 0;
#pragma omp parallel
    {
        double *wcol = (double *)malloc((size_t)d * sizeof(double));
        if (!wcol) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp barrier
        if (!failed) {
#pragma omp for schedule(static)
            for (int v = 0; v < V; v++) {
                for (int k = 0; k < d; k++) {
                    size_t idx = (w_layout == AJO_W_VD) ? (size_t)v * d + k : (size_t)k * V + v;
                    wcol[k] = elem_to_double(W, idx, dtype);
                }
                for (int r = 0; r < R; r++) {
                    const double *hr = hd + (size_t)r * d;
                    double s = 0.0;
                    /* summation order is free: every term is exact in double and the
                       rounding error of any order is far below the comparison tolerances */
#pragma omp simd reduction(+ : s)
                    for (int k = 0; k < d; k++) s += hr[k] * wcol[k];
                    logits[(size_t)r * V + v] = s;
                }
            }
        }
        free(wcol);
    }
    free(hd);
    return failed ? 2 : 0;
}

/*
 * Step 2 for one row: smallest index attaining the maximum, the maximum, and the
 * distance to the largest value found at any other index (0 when the maximum is tied).
 */
void ajo_argmax(const double *row, int V, int32_t *y, double *top1, double *gap)
{
    int best = 0;
    for (int v = 1; v < V; v++)
        if (row[v] > row[best]) best = v;
    double second = -INFINITY;
    for (int v = 0; v < V; v++)
        if (v != best && row[v] > second) second = row[v];
    *y = best;
    *top1 = row[best];
    *gap = (V > 1) ? row[best] - second : INFINITY;
}

/*
 * Step 4 for one position: P(important) from the logistic-regression judge on the
 * concatenation [h_draft_row ; h_target_row]; judge_w has d_draft + d entries in that order.
 */
double ajo_judge_p(const void *h_draft_row, const void *h_target_row, int dtype,
                   const float *judge_w, float judge_b, int d_draft, int d)
{
    double z = (double)judge_b;
    for (int f = 0; f < d_draft; f++)
        z += (double)judge_w[f] * elem_to_double(h_draft_row, (size_t)f, dtype);
    for (int f = 0; f < d; f++)
        z += (double)judge_w[d_draft + f] * elem_to_double(h_target_row, (size_t)f, dtype);
    return 1.0 / (1.0 + exp(-z));
}

/* does the judge forgive a mismatch whose importance probability is p? */
static int forgiven(double p, float tau)
{
    if (tau <= 0.0f) return 0;
    if (tau >= 1.0f) return 1;
    return (float)p < tau;
}

/*
 * The whole step for B sequences.  R = K + 1 rows per sequence, or R = K when extra_row == 0.
 *   h_target [B][R][d], h_draft [B][R][d_draft] (NULL iff d_draft == 0), W per w_layout,
 *   draft_tok [B][K], judge_w [d_draft + d].
 * Outputs (all caller-allocated, all required):
 *   accept_len [B], next_tok [B], target_tok [B][R], top1 [B][R], gap [B][R],
 *   judge_p [B][K]  (p at every mismatching position whose features exist, NaN elsewhere).
 */
int ajo_verify_sampled(const void *h_target, const void *h_draft, const void *W,
                       const int32_t *draft_tok, const float *judge_w, float judge_b, float tau,
                       int dtype, int w_layout, int B, int K, int d, int d_draft, int V, int extra_row,
                       double temperature, uint64_t seed, uint64_t step, int row0,
                       int32_t *accept_len, int32_t *next_tok, int32_t *target_tok,
                       double *top1, double *gap, double *judge_p);

int ajo_verify(const void *h_target, const void *h_draft, const void *W,
               const int32_t *draft_tok, const float *judge_w, float judge_b, float tau,
               int dtype, int w_layout, int B, int K, int d, int d_draft, int V, int extra_row,
               int32_t *accept_len, int32_t *next_tok, int32_t *target_tok,
               double *top1, double *gap, double *judge_p)
{
    return ajo_verify_sampled(h_target, h_draft, W, draft_tok, judge_w, judge_b, tau, dtype, w_layout, B, K, d, d_draft,
                              V, extra_row, 0.0, 0, 0, 0, accept_len, next_tok, target_tok, top1, gap, judge_p);
}

/*
 * The whole step with the target's tokens drawn by the Gumbel-max trick at the given temperature
 * (0 = greedy); top1 and gap then refer to the noisy scores logit + temperature * g.  The noise of row j
 * of sequence b is that of row index row0 + b * (rows per sequence) + j: row0 = 0 for a whole batch, or
 * the index of the first row when the sequences given are a slice of a larger batch.
 */
int ajo_verify_sampled(const void *h_target, const void *h_draft, const void *W,
                       const int32_t *draft_tok, const float *judge_w, float judge_b, float tau,
                       int dtype, int w_layout, int B, int K, int d, int d_draft, int V, int extra_row,
                       double temperature, uint64_t seed, uint64_t step, int row0,
                       int32_t *accept_len, int32_t *next_tok, int32_t *target_tok,
                       double *top1, double *gap, double *judge_p)
{
    if (!h_target || !W || !draft_tok || !judge_w || B < 1 || K < 1 || d < 1 || V < 1 ||
        d_draft < 0 || (d_draft > 0 && !h_draft))
        return 1;
    size_t esz = (dtype == AJO_BF16) ? 2 : 4;
    int R = extra_row ? K + 1 : K;
    double *logits = (double *)malloc((size_t)R * V * sizeof(double));
    if (!logits) return 2;

    for (int b = 0; b < B; b++) {
        const char *ht = (const char *)h_target + (size_t)b * R * d * esz;
        const char *hdr = h_draft ? (const char *)h_draft + (size_t)b * R * d_draft * esz : NULL;
        int rc = ajo_logits(ht, W, dtype, w_layout, R, d, V, logits);
        if (rc) { free(logits); return rc; }
        if (temperature > 0.0) {
#pragma omp parallel for schedule(static)
            for (int v = 0; v < V; v++)
                for (int j = 0; j < R; j++)
                    logits[(size_t)j * V + v] += temperature * ajo_gumbel(seed, step, row0 + b * R + j, v);
        }

        int32_t *y = target_tok + (size_t)b * R;
        for (int j = 0; j < R; j++)
            ajo_argmax(logits + (size_t)j * V, V, &y[j], &top1[(size_t)b * R + j], &gap[(size_t)b * R + j]);

        /* p at every mismatch (the device evaluates all mismatches, so all are comparable) */
        for (int i = 0; i < K; i++) {
            double p = NAN;
            if (draft_tok[(size_t)b * K + i] != y[i] && i + 1 < R) /* row i+1 encodes draft token i */
                p = ajo_judge_p(hdr ? hdr + (size_t)(i + 1) * d_draft * esz : NULL,
                                ht + (size_t)(i + 1) * d * esz, dtype, judge_w, judge_b, d_draft, d);
            judge_p[(size_t)b * K + i] = p;
        }

        /* walk the window in order; stop at the first mismatch the judge does not forgive */
        int n = 0;
        while (n < K) {
            if (draft_tok[(size_t)b * K + n] != y[n]) {
                if (n + 1 >= R) break; /* no features for the last token: rejected without the classifier */
                if (!forgiven(judge_p[(size_t)b * K + n], tau)) break;
            }
            n++;
        }
        accept_len[b] = n;
        next_tok[b] = n < R ? y[n] : -1;
    }
    free(logits);
    return 0;
}

/*
 * Tree drafts (Section 3.3, "Generality": the method applies to tree-based speculative decoding;
 * Appendix on EAGLE-2).  The draft is a tree of N nodes in topological order: parent[n] is -1 for a
 * child of the root (the last accepted token, row 0) or the index (< n) of another node; row n + 1
 * of the hidden states encodes node n.  The target's prediction after a node is the token of that
 * node's row, so node n matches iff tok[n] == y[parent[n] + 1].  The acceptance rule of the paper,
 * applied along every root-to-leaf path as it is applied to a window: a node is accepted iff its
 * parent is accepted (the root always is) and it matches or its mismatch is forgiven (p < tau).  The
 * result is the deepest accepted node (among equally deep ones the lowest index; -1 = the root),
 * its depth as the accepted length, and the target's token after it.  A node whose parent index is
 * outside [-1, n) is never accepted and never judged.
 *
 * This function is the rule alone, on given tokens and probabilities (p[n] is read only where node n
 * mismatches).
 */
void ajo_tree_accept(int N, const int32_t *tok, const int32_t *parent, const int32_t *y, const double *p,
                     float tau, int32_t *accept_len, int32_t *best_node, int32_t *next_tok)
{
    int best = -1, best_depth = 0;
    int *ok = (int *)malloc((size_t)N * sizeof(int)), *depth = (int *)malloc((size_t)N * sizeof(int));
    for (int n = 0; n < N; n++) {
        const int q = parent[n];
        ok[n] = 0;
        depth[n] = 0;
        if (q < -1 || q >= n) continue;
        const int parent_ok = (q == -1) ? 1 : ok[q];
        const int passes = (tok[n] == y[q + 1]) ? 1 : forgiven(p[n], tau);
        depth[n] = (q == -1 ? 0 : depth[q]) + 1;
        ok[n] = parent_ok && passes;
        if (ok[n] && depth[n] > best_depth) {
            best = n;
            best_depth = depth[n];
        }
    }
    free(ok);
    free(depth);
    *accept_len = best_depth;
    *best_node = best;
    *next_tok = y[best + 1];
}

/*
 * The whole step for tree drafts: B sequences of N nodes (N + 1 rows each, layouts as ajo_verify),
 * target tokens greedy or drawn (temperature as in ajo_verify_sampled), the classifier evaluated at
 * every mismatching node with a valid parent, then ajo_tree_accept.
 */
int ajo_verify_tree(const void *h_target, const void *h_draft, const void *W, const int32_t *draft_tok,
                    const int32_t *parent, const float *judge_w, float judge_b, float tau, int dtype, int w_layout,
                    int B, int N, int d, int d_draft, int V, double temperature, uint64_t seed, uint64_t step, int row0,
                    int32_t *accept_len, int32_t *next_tok, int32_t *best_node, int32_t *target_tok,
                    double *top1, double *gap, double *judge_p)
{
    if (!h_target || !W || !draft_tok || !parent || !judge_w || B < 1 || N < 1 || d < 1 || V < 1 ||
        d_draft < 0 || (d_draft > 0 && !h_draft))
        return 1;
    size_t esz = (dtype == AJO_BF16) ? 2 : 4;
    int R = N + 1;
    double *logits = (double *)malloc((size_t)R * V * sizeof(double));
    if (!logits) return 2;
    for (int b = 0; b < B; b++) {
        const char *ht = (const char *)h_target + (size_t)b * R * d * esz;
        const char *hdr = h_draft ? (const char *)h_draft + (size_t)b * R * d_draft * esz : NULL;
        int rc = ajo_logits(ht, W, dtype, w_layout, R, d, V, logits);
        if (rc) { free(logits); return rc; }
        if (temperature > 0.0) {
#pragma omp parallel for schedule(static)
            for (int v = 0; v < V; v++)
                for (int j = 0; j < R; j++)
                    logits[(size_t)j * V + v] += temperature * ajo_gumbel(seed, step, row0 + b * R + j, v);
        }
        int32_t *y = target_tok + (size_t)b * R;
        for (int j = 0; j < R; j++)
            ajo_argmax(logits + (size_t)j * V, V, &y[j], &top1[(size_t)b * R + j], &gap[(size_t)b * R + j]);
        const int32_t *tok = draft_tok + (size_t)b * N, *par = parent + (size_t)b * N;
        double *p = judge_p + (size_t)b * N;
        for (int n = 0; n < N; n++) {
            p[n] = NAN;
            if (par[n] < -1 || par[n] >= n) continue;
            if (tok[n] != y[par[n] + 1]) /* row n + 1 encodes node n */
                p[n] = ajo_judge_p(hdr ? hdr + (size_t)(n + 1) * d_draft * esz : NULL,
                                   ht + (size_t)(n + 1) * d * esz, dtype, judge_w, judge_b, d_draft, d);
        }
        ajo_tree_accept(N, tok, par, y, p, tau, &accept_len[b], &best_node[b], &next_tok[b]);
    }
    free(logits);
    return 0;
}

/*
 * Rank of entry `tok` in one row of logits: how many entries come before it when the row is sorted
 * by decreasing logit, ties by increasing index.  *near receives the number of OTHER entries whose
 * logit lies within `band` of logit[tok] (a device that rounds differently may order those otherwise).
 */
int ajo_rank(const double *row, int V, int tok, double band, int32_t *near)
{
    int rank = 0, n = 0;
    const double t = row[tok];
    for (int v = 0; v < V; v++) {
        if (v == tok) continue;
        if (row[v] > t || (row[v] == t && v < tok)) rank++;
        if (fabs(row[v] - t) <= band) n++;
    }
    if (near) *near = n;
    return rank;
}

/*
 * The whole step under the top-K rule for B sequences, K + 1 rows each (layouts as ajo_verify).
 * Outputs: accept_len [B], next_tok [B], target_tok [B][K+1], top1 [B][K+1], gap [B][K+1],
 *   rank [B][K]  rank of the draft token at every mismatching position (-1 where it matched, V where
 *                the draft token is outside the vocabulary),
 *   near [B][K]  entries within `band` of the draft token's logit there (0 where it matched).
 */
int ajo_verify_topk(const void *h_target, const void *W, const int32_t *draft_tok, int top_k, double band,
                    int dtype, int w_layout, int B, int K, int d, int V,
                    int32_t *accept_len, int32_t *next_tok, int32_t *target_tok,
                    double *top1, double *gap, int32_t *rank, int32_t *near)
{
    if (!h_target || !W || !draft_tok || B < 1 || K < 1 || d < 1 || V < 1 || top_k < 1) return 1;
    size_t esz = (dtype == AJO_BF16) ? 2 : 4;
    int R = K + 1;
    double *logits = (double *)malloc((size_t)R * V * sizeof(double));
    if (!logits) return 2;
    for (int b = 0; b < B; b++) {
        const char *ht = (const char *)h_target + (size_t)b * R * d * esz;
        int rc = ajo_logits(ht, W, dtype, w_layout, R, d, V, logits);
        if (rc) { free(logits); return rc; }
        int32_t *y = target_tok + (size_t)b * R;
        for (int j = 0; j < R; j++)
            ajo_argmax(logits + (size_t)j * V, V, &y[j], &top1[(size_t)b * R + j], &gap[(size_t)b * R + j]);
        for (int i = 0; i < K; i++) {
            int tok = draft_tok[(size_t)b * K + i];
            int32_t r = -1, n = 0;
            if (tok != y[i]) {
                if (tok < 0 || tok >= V) r = V;
                else r = ajo_rank(logits + (size_t)i * V, V, tok, band, &n);
            }
            rank[(size_t)b * K + i] = r;
            near[(size_t)b * K + i] = n;
        }
        int n = 0;
        while (n < K) {
            int32_t r = rank[(size_t)b * K + n];
            int t = draft_tok[(size_t)b * K + n];
            if (r >= 0 && (t < 0 || t >= V || !(r < top_k))) break; /* a mismatch outside the target's top_k */
            n++;
        }
        accept_len[b] = n;
        next_tok[b] = y[n];
    }
    free(logits);
    return 0;
}
