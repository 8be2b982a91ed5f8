/*
 * CPU oracle for LOOK-M's prefill-time KV-cache compression (test infrastructure only).
 *
 * A plain, slow, fp64 restatement of the method, one function per step, written from the paper's
 * definitions.  It exists to check the CUDA library and shares no code with it; nothing but the
 * tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Inputs are float arrays whose values are exactly representable in bf16 (the generator rounds
 * them); every value is widened to double before use and all arithmetic is double.
 *
 * Each function works on ONE KV head (and, for the scores, the query heads that share it).
 * Tensors are addressed as base pointer + token stride (in elements), feature index contiguous.
 *
 * Pinned by tests/test_oracle_*.py: closed forms (uniform attention -> harmonic numbers, the
 * two-token sigmoid form, single-kept-token merges, the decode step's uniform mean and a
 * three-row hand case), invariants (row sums, kept count, window, text survival, sum
 * preservation, shift invariance) and brute force on tiny inputs.  No function is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------------
 * Step 1. Cumulative attention score (Eq. 4): A_s[j] = sum over prompt rows i of A_p[i, j],
 * with A_p the causal row-softmax of Q K^T * scale.  Under grouped-query attention the sums of
 * the n_group query heads that share the KV head are added.
 *
 * Only rows i >= key_begin are visited: rows before key_begin give nothing to the keys
 * j >= key_begin, and those are the only entries of `scores` that are then meaningful
 * (entries j < key_begin are set to NaN unless key_begin == 0).
 *
 * lse (optional, [n_group, L]) receives log(sum_j exp(s_ij)) of each visited row (natural log).
 * Returns 0, or -1 if the scratch row cannot be allocated.
 * ------------------------------------------------------------------------------------------ */
int lookm_oracle_scores_head(const float *q, long long q_stride_tok, long long q_stride_head,
                             int n_group, const float *k, long long k_stride_tok, int L, int d,
                             double scale, int key_begin, double *scores, double *lse)
{
    double *s = (double *)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1));
    if (!s) return -1;
    for (int j = 0; j < L; ++j) scores[j] = (j < key_begin) ? NAN : 0.0;
    for (int g = 0; g < n_group; ++g) {
        for (int i = key_begin; i < L; ++i) {
            const float *qi = q + (long long)i * q_stride_tok + (long long)g * q_stride_head;
            double row_max = -INFINITY;
            for (int j = 0; j <= i; ++j) {                 /* causal: keys up to and including i */
                const float *kj = k + (long long)j * k_stride_tok;
                double dot = 0.0;
                for (int c = 0; c < d; ++c) dot += (double)qi[c] * (double)kj[c];
                s[j] = dot * scale;
                if (s[j] > row_max) row_max = s[j];
            }
            double denom = 0.0;
            for (int j = 0; j <= i; ++j) { s[j] = exp(s[j] - row_max); denom += s[j]; }
            for (int j = key_begin; j <= i; ++j) scores[j] += s[j] / denom;
            if (lse) lse[(long long)g * L + i] = row_max + log(denom);
        }
    }
    free(s);
    return 0;
}

/* log-sum-exp of selected causal rows of one query head (natural log); rows[] in [0, L). */
int lookm_oracle_lse_rows(const float *q, long long q_stride_tok, const float *k,
                          long long k_stride_tok, int d, double scale, const int *rows, int n_rows,
                          double *lse)
{
    for (int r = 0; r < n_rows; ++r) {
        int i = rows[r];
        const float *qi = q + (long long)i * q_stride_tok;
        double row_max = -INFINITY;
        double *s = (double *)malloc(sizeof(double) * (size_t)(i + 1));
        if (!s) return -1;
        for (int j = 0; j <= i; ++j) {
            const float *kj = k + (long long)j * k_stride_tok;
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += (double)qi[c] * (double)kj[c];
            s[j] = dot * scale;
            if (s[j] > row_max) row_max = s[j];
        }
        double denom = 0.0;
        for (int j = 0; j <= i; ++j) denom += exp(s[j] - row_max);
        lse[r] = row_max + log(denom);
        free(s);
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Steps 2-4. Recent window, text prior and Top-N (Eq. 5-8).
 *
 * The last M tokens are kept.  Among the candidates [0, L-M) the N = B-M best are kept, where
 * "best" orders text tokens before image tokens (the effect of adding T_p = max(A_s) to every
 * text score: all scores are positive, so any boosted score exceeds any unboosted one), then
 * larger A_s first, then lower position first.  T_p is never added numerically.
 *
 * text_prior = 0 leaves Eq. 5 out: the N best are taken by A_s alone (Eq. 8 on the raw scores;
 * the rows of the paper's main-results table that merge without the text prior), ties still to
 * the lower position.
 *
 * mask[j] = 1 for an image token, 0 for text.  B and M are clamped: B <= L, M <= B.
 * kept[] receives the kept positions in ascending order (the N selected, then the window);
 * evicted[] the others in ascending order.  Returns the kept count (= min(B, L)), or -1.
 * ------------------------------------------------------------------------------------------ */
typedef struct { int is_text; double score; int pos; } cand_t;

static int cand_before(const cand_t *a, const cand_t *b)
{
    if (a->is_text != b->is_text) return a->is_text > b->is_text;
    if (a->score != b->score) return a->score > b->score;
    return a->pos < b->pos;
}

int lookm_oracle_select(const double *scores, const uint8_t *mask, int L, int B, int M,
                        int text_prior, int *kept, int *evicted)
{
    if (L <= 0 || B <= 0 || M < 0) return -1;
    if (B > L) B = L;
    if (M > B) M = B;
    int N = B - M, n_cand = L - M;
    cand_t *c = (cand_t *)malloc(sizeof(cand_t) * (size_t)(n_cand > 0 ? n_cand : 1));
    uint8_t *keep = (uint8_t *)calloc((size_t)L, 1);
    if (!c || !keep) { free(c); free(keep); return -1; }
    for (int j = 0; j < n_cand; ++j) { c[j].is_text = (text_prior && !mask[j]) ? 1 : 0; c[j].score = scores[j]; c[j].pos = j; }
    /* insertion of the N best by repeated selection: O(N * L), obviously a full ordering */
    for (int r = 0; r < N; ++r) {
        int best = r;
        for (int j = r + 1; j < n_cand; ++j) if (cand_before(&c[j], &c[best])) best = j;
        cand_t t = c[r]; c[r] = c[best]; c[best] = t;
        keep[c[r].pos] = 1;
    }
    for (int j = L - M; j < L; ++j) keep[j] = 1;
    int nk = 0, ne = 0;
    for (int j = 0; j < L; ++j) { if (keep[j]) kept[nk++] = j; else evicted[ne++] = j; }
    free(c); free(keep);
    return nk;
}

/* ------------------------------------------------------------------------------------------
 * Step 5. Nearest-neighbour matching (Eq. 9): for each evicted key the kept key of largest
 * cosine similarity, on the original keys; lowest kept slot on exact ties; similarity 0 when a
 * norm is 0.  assign[e] is a slot in [0, n_kept); sim[e] the row maximum.
 * sim_matrix (optional, [n_evicted, n_kept]) receives every s_ij.
 * ------------------------------------------------------------------------------------------ */
static double cosine(const float *a, const float *b, int d)
{
    double ab = 0.0, aa = 0.0, bb = 0.0;
    for (int c = 0; c < d; ++c) {
        ab += (double)a[c] * (double)b[c];
        aa += (double)a[c] * (double)a[c];
        bb += (double)b[c] * (double)b[c];
    }
    if (aa == 0.0 || bb == 0.0) return 0.0;
    return ab / (sqrt(aa) * sqrt(bb));
}

void lookm_oracle_match(const float *k, long long k_stride_tok, int d, const int *kept, int n_kept,
                        const int *evicted, int n_evicted, int *assign, double *sim,
                        double *sim_matrix)
{
    for (int e = 0; e < n_evicted; ++e) {
        const float *ke = k + (long long)evicted[e] * k_stride_tok;
        int best = 0;
        double best_sim = -INFINITY;
        for (int c = 0; c < n_kept; ++c) {
            double s = cosine(ke, k + (long long)kept[c] * k_stride_tok, d);
            if (sim_matrix) sim_matrix[(long long)e * n_kept + c] = s;
            if (s > best_sim) { best_sim = s; best = c; }
        }
        assign[e] = best;
        sim[e] = best_sim;
    }
}

/* Row argmax of a given similarity matrix with the same tie rule (lowest slot). */
void lookm_oracle_argmax_rows(const double *sim_matrix, int n_evicted, int n_kept, int *assign,
                              double *sim)
{
    for (int e = 0; e < n_evicted; ++e) {
        int best = 0;
        double best_sim = -INFINITY;
        for (int c = 0; c < n_kept; ++c) {
            double s = sim_matrix[(long long)e * n_kept + c];
            if (s > best_sim) { best_sim = s; best = c; }
        }
        assign[e] = best;
        sim[e] = best_sim;
    }
}

/* ------------------------------------------------------------------------------------------
 * Step 6. Merging (Eq. 10-12) of one tensor x (the keys, then the values, with the same
 * assignment and weights).  For kept slot c with original row x_c and members E_c, n = |E_c|:
 *   mode 0 averaged : (x_c + sum_e x_e) / (n + 1)
 *   mode 1 pivotal  : (x_c + 1/2 sum_e (x_e + x_c)) / (n + 1)
 *   mode 2 weighted : (x_c + sum_e sim[e] x_e) / (n + 1)
 *   mode 3 none     : x_c  (eviction alone, Eq. 6-7: the evicted rows are dropped, not merged)
 * All sums use the original rows.  out is [n_kept, d] in fp64.
 * ------------------------------------------------------------------------------------------ */
int lookm_oracle_merge(const float *x, long long x_stride_tok, int d, const int *kept, int n_kept,
                       const int *evicted, int n_evicted, const int *assign, const double *sim,
                       int mode, double *out)
{
    int *count = (int *)calloc((size_t)(n_kept > 0 ? n_kept : 1), sizeof(int));
    if (!count) return -1;
    for (int c = 0; c < n_kept; ++c) {
        const float *xc = x + (long long)kept[c] * x_stride_tok;
        for (int t = 0; t < d; ++t) out[(long long)c * d + t] = (double)xc[t];
    }
    for (int e = 0; e < n_evicted && mode != 3; ++e) {
        int c = assign[e];
        const float *xe = x + (long long)evicted[e] * x_stride_tok;
        const float *xc = x + (long long)kept[c] * x_stride_tok;
        count[c] += 1;
        for (int t = 0; t < d; ++t) {
            double add;
            if (mode == 0)      add = (double)xe[t];
            else if (mode == 1) add = 0.5 * ((double)xe[t] + (double)xc[t]);
            else                add = sim[e] * (double)xe[t];
            out[(long long)c * d + t] += add;
        }
    }
    for (int c = 0; c < n_kept; ++c)
        for (int t = 0; t < d; ++t) out[(long long)c * d + t] /= (double)(count[c] + 1);
    free(count);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * The step after the path: one token-generation step over a cache (Section 3.1, Eq. 2-3).
 * The new token's key and value rows are appended to the cache first (Eq. 2); the caller passes
 * the cache WITH that row, n rows in all.  Then, for each of the n_group query heads that share
 * this KV head,  out_g = softmax(q_g K^T * scale) V  over all n rows (Eq. 3; no mask: every cached
 * row precedes the new token).  out is [n_group, d] in fp64.  Returns 0, or -1 without memory.
 * ------------------------------------------------------------------------------------------ */
int lookm_oracle_decode_head(const float *q, long long q_stride_head, int n_group, const float *k,
                             long long k_stride_row, const float *v, long long v_stride_row, int n,
                             int d, double scale, double *out)
{
    double *p = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    if (!p) return -1;
    for (int g = 0; g < n_group; ++g) {
        const float *qg = q + (long long)g * q_stride_head;
        double row_max = -INFINITY;
        for (int j = 0; j < n; ++j) {
            const float *kj = k + (long long)j * k_stride_row;
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += (double)qg[c] * (double)kj[c];
            p[j] = dot * scale;
            if (p[j] > row_max) row_max = p[j];
        }
        double denom = 0.0;
        for (int j = 0; j < n; ++j) { p[j] = exp(p[j] - row_max); denom += p[j]; }
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int j = 0; j < n; ++j) acc += p[j] * (double)v[(long long)j * v_stride_row + c];
            out[(long long)g * d + c] = acc / denom;
        }
    }
    free(p);
    return 0;
}
