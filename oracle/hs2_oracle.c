/*
 * CPU oracle for the hybrid sparse-attention path of HySparse2.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the
 * path computes, used to check the CUDA library and timed as the CPU baseline.
 * It shares no code with the CUDA library and the library never calls it.
 *
 * Arithmetic is fp64 on the exact fp32 / bf16 input values.  No blocking, fusion
 * or reordering beyond the definitions below; OpenMP only distributes whole query
 * rows over threads.
 *
 * Definitions followed (paper sections in brackets):
 *   full attention   softmax(scale * Q K^T) V, causal, no positional encoding
 *                    [Section 3.4 "The Role of Full Attention"; Section 4.1: NoPE]
 *   selection score  the full layer's own exact attention scores [Section 3.4];
 *                    per KV head the scores of the query heads that share it are
 *                    aggregated (default: max of the softmax probabilities)
 *   forced window    the most recent w tokens are always selected [Section 3.3,
 *                    "Removing the Separate SWA Branch"]
 *   top-k            the k highest-scoring tokens outside the window, token level
 *                    [Section 3.3, "Token-Level Sparse Selection"]
 *   sparse attention softmax attention restricted to window U top-k, own queries,
 *                    K/V read from the full layer's cache [Section 3.3]; optional
 *                    per-head sink bias in the denominator [Section 4.1]
 *
 * Parity pins (tests/test_oracle_*.py): library SDPA for the full attention,
 * brute-force ranking for the top-k, k >= context -> full attention, k = 0 ->
 * sliding-window attention, hand-worked vectors, closed forms.  The aggregation
 * over a GQA group and the "probabilities, not logits" reading are not fixed by
 * the paper: for those two readings parity is unpinned by the paper itself.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t batch, n_q_heads, n_kv_heads, head_dim;
    int32_t q_len, kv_len;
    int32_t k_sel, window;
    double scale;          /* softmax scale (already resolved, never 0) */
    int32_t dtype;         /* 0 = fp32, 1 = bf16 (raw bits) */
    int32_t agg;           /* 0 = max of probabilities, 1 = max of logits, 2 = sum of probabilities */
    const int32_t *q_start;   /* [batch] or NULL: absolute position of query 0 = kv_lens[b] - q_len */
    const int32_t *kv_lens;   /* [batch] or NULL: kv_len */
} hs2o_problem;

static double load_elem(const void *base, int64_t off, int dtype)
{
    if (dtype == 0) return (double)((const float *)base)[off];
    uint32_t bits = (uint32_t)((const uint16_t *)base)[off] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

static int kvlen_of(const hs2o_problem *p, int b) { return p->kv_lens ? p->kv_lens[b] : p->kv_len; }
static int pos_of(const hs2o_problem *p, int b, int i)
{
    int q0 = p->q_start ? p->q_start[b] : kvlen_of(p, b) - p->q_len;
    return q0 + i;
}

int hs2o_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* q . k_j for query (b,i,h) and key (b,j,g) */
static double dot_qk(const hs2o_problem *p, const void *Q, const void *K, int b, int i, int h, int j)
{
    const int D = p->head_dim, g = h / (p->n_q_heads / p->n_kv_heads);
    int64_t qo = (((int64_t)b * p->q_len + i) * p->n_q_heads + h) * D;
    int64_t ko = (((int64_t)b * p->kv_len + j) * p->n_kv_heads + g) * D;
    double s = 0.0;
    for (int d = 0; d < D; ++d) s += load_elem(Q, qo + d, p->dtype) * load_elem(K, ko + d, p->dtype);
    return s;
}

/*
 * Full causal attention of one query token (all heads) and, optionally, the
 * selection scores of that token for every KV head.
 *   O      [Hq, D]     LSE [Hq]
 *   score  [Hkv, kv_len] or NULL: aggregated score for visible keys, -inf elsewhere
 */
void hs2o_full_attn_row(const hs2o_problem *p, const void *Q, const void *K, const void *V,
                        int b, int i, double *O, double *LSE, double *score)
{
    const int D = p->head_dim, Hq = p->n_q_heads, Hkv = p->n_kv_heads, G = Hq / Hkv;
    const int pos = pos_of(p, b, i);
    int last = pos;                                   /* last visible key */
    if (last > kvlen_of(p, b) - 1) last = kvlen_of(p, b) - 1;
    const int n = last + 1;
    if (score)
        for (int64_t t = 0; t < (int64_t)Hkv * p->kv_len; ++t) score[t] = -INFINITY;
    double *s = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    for (int h = 0; h < Hq; ++h) {
        const int g = h / G;
        double *o = O + (int64_t)h * D;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        if (n <= 0) { LSE[h] = -INFINITY; continue; }
        double m = -INFINITY;
        for (int j = 0; j < n; ++j) {
            s[j] = p->scale * dot_qk(p, Q, K, b, i, h, j);
            if (s[j] > m) m = s[j];
        }
        double l = 0.0;
        for (int j = 0; j < n; ++j) l += exp(s[j] - m);
        const double lse = m + log(l);
        LSE[h] = lse;
        for (int j = 0; j < n; ++j) {
            const double pj = exp(s[j] - lse);
            int64_t vo = (((int64_t)b * p->kv_len + j) * Hkv + g) * D;
            for (int d = 0; d < D; ++d) o[d] += pj * load_elem(V, vo + d, p->dtype);
            if (score) {
                double *a = score + (int64_t)g * p->kv_len + j;
                const int first = (h % G) == 0;
                if (p->agg == 0) { if (first || pj > *a) *a = pj; }
                else if (p->agg == 1) { if (first || s[j] > *a) *a = s[j]; }
                else { *a = first ? pj : *a + pj; }
            }
        }
    }
    free(s);
}

typedef struct { double a; int32_t j; } cand_t;

static int cand_cmp(const void *x, const void *y)
{
    const cand_t *u = (const cand_t *)x, *v = (const cand_t *)y;
    if (u->a > v->a) return -1;            /* higher score first */
    if (u->a < v->a) return 1;
    return (u->j > v->j) - (u->j < v->j);  /* equal score: lower key index first */
}
static int int_cmp(const void *x, const void *y)
{
    int32_t u = *(const int32_t *)x, v = *(const int32_t *)y;
    return (u > v) - (u < v);
}

/*
 * Token-level top-k outside the forced window for one (query, KV head).
 *   score [kv_len]: selection score of every key; pos: absolute query position.
 *   Candidates are keys 0 .. min(pos - window, kvlen - 1).  The first
 *   min(k, #candidates) in (score descending, index ascending) order are kept,
 *   written in ascending index order and padded with -1 to length k.
 */
void hs2o_select_row(const double *score, int kvlen, int pos, int window, int k, int32_t *idx)
{
    int last = pos - window;
    if (last > kvlen - 1) last = kvlen - 1;
    const int nc = last + 1 > 0 ? last + 1 : 0;
    int take = k < nc ? k : nc;
    for (int t = 0; t < k; ++t) idx[t] = -1;
    if (take <= 0) return;
    cand_t *c = (cand_t *)malloc(sizeof(cand_t) * (size_t)nc);
    for (int j = 0; j < nc; ++j) { c[j].a = score[j]; c[j].j = j; }
    qsort(c, (size_t)nc, sizeof(cand_t), cand_cmp);
    for (int t = 0; t < take; ++t) idx[t] = c[t].j;
    qsort(idx, (size_t)take, sizeof(int32_t), int_cmp);
    free(c);
}

/*
 * Sparse attention of one query token (all heads): softmax over
 *   S = {valid selected indices} U {window positions}.
 *   idx  [Hkv, k] rows of this token.  An entry is ignored when it is negative,
 *        inside the window or in the future (> pos - window) or >= kvlen.
 *   sink [Hq] or NULL: e^{sink_h} joins the denominator, with no value.
 *   member [Hkv, kv_len] or NULL: receives 1 for keys in S, else 0 (test introspection).
 */
void hs2o_sparse_attn_row(const hs2o_problem *p, const void *Q, const void *K, const void *V,
                          const int32_t *idx, const double *sink, int b, int i,
                          double *O, double *LSE, uint8_t *member)
{
    const int D = p->head_dim, Hq = p->n_q_heads, Hkv = p->n_kv_heads, G = Hq / Hkv;
    const int kvlen = kvlen_of(p, b), pos = pos_of(p, b, i), w = p->window, k = p->k_sel;
    uint8_t *in_s = (uint8_t *)calloc((size_t)(p->kv_len > 0 ? p->kv_len : 1), 1);
    int32_t *S = (int32_t *)malloc(sizeof(int32_t) * (size_t)(k + w + 1));
    double *s = (double *)malloc(sizeof(double) * (size_t)(k + w + 1));
    for (int g = 0; g < Hkv; ++g) {
        int n = 0;
        memset(in_s, 0, (size_t)(p->kv_len > 0 ? p->kv_len : 1));
        for (int t = 0; t < k; ++t) {                      /* the reused top-k set */
            int32_t j = idx[(int64_t)g * k + t];
            if (j < 0 || j > pos - w || j >= kvlen || in_s[j]) continue;
            in_s[j] = 1; S[n++] = j;
        }
        for (int j = pos - w + 1; j <= pos; ++j) {         /* the forced window */
            if (j < 0 || j >= kvlen || in_s[j]) continue;
            in_s[j] = 1; S[n++] = j;
        }
        if (member) memcpy(member + (int64_t)g * p->kv_len, in_s, (size_t)p->kv_len);
        for (int h = g * G; h < (g + 1) * G; ++h) {
            double *o = O + (int64_t)h * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            double m = sink ? sink[h] : -INFINITY;
            for (int t = 0; t < n; ++t) {
                s[t] = p->scale * dot_qk(p, Q, K, b, i, h, S[t]);
                if (s[t] > m) m = s[t];
            }
            if (m == -INFINITY) { LSE[h] = -INFINITY; continue; }   /* empty set, no sink */
            double l = sink ? exp(sink[h] - m) : 0.0;
            for (int t = 0; t < n; ++t) l += exp(s[t] - m);
            const double lse = m + log(l);
            LSE[h] = lse;
            for (int t = 0; t < n; ++t) {
                const double pj = exp(s[t] - lse);
                int64_t vo = (((int64_t)b * p->kv_len + S[t]) * Hkv + g) * D;
                for (int d = 0; d < D; ++d) o[d] += pj * load_elem(V, vo + d, p->dtype);
            }
        }
    }
    free(s); free(S); free(in_s);
}

/* ---- drivers over lists of (b, i) rows; OpenMP hands out whole rows ---- */

/* O [n,Hq,D], LSE [n,Hq], idx [n,Hkv,k] (nullable), score [n,Hkv,kv_len] (nullable) */
void hs2o_full_attn_select_rows(const hs2o_problem *p, const void *Q, const void *K, const void *V,
                                int n_rows, const int32_t *rows_b, const int32_t *rows_i,
                                double *O, double *LSE, int32_t *idx, double *score)
{
    const int Hq = p->n_q_heads, Hkv = p->n_kv_heads, D = p->head_dim, k = p->k_sel;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
        const int b = rows_b[r], i = rows_i[r];
        double *sc = score ? score + (int64_t)r * Hkv * p->kv_len
                           : (idx ? (double *)malloc(sizeof(double) * (size_t)Hkv * p->kv_len) : NULL);
        hs2o_full_attn_row(p, Q, K, V, b, i, O + (int64_t)r * Hq * D, LSE + (int64_t)r * Hq, sc);
        if (idx)
            for (int g = 0; g < Hkv; ++g)
                hs2o_select_row(sc + (int64_t)g * p->kv_len, kvlen_of(p, b), pos_of(p, b, i), p->window, k,
                                idx + ((int64_t)r * Hkv + g) * k);
        if (!score && sc) free(sc);
    }
}

/* score [n, kv_len] (one row per (query, KV head) pair), pos [n], kvlen [n] -> idx [n, k] */
void hs2o_select_rows(const double *score, int row_stride, int n_rows, const int32_t *pos,
                      const int32_t *kvlen, int window, int k, int32_t *idx)
{
#pragma omp parallel for schedule(dynamic, 4)
    for (int r = 0; r < n_rows; ++r)
        hs2o_select_row(score + (int64_t)r * row_stride, kvlen[r], pos[r], window, k, idx + (int64_t)r * k);
}

/* idx [n,Hkv,k] -> O [n,Hq,D], LSE [n,Hq], member [n,Hkv,kv_len] (nullable) */
void hs2o_sparse_attn_rows(const hs2o_problem *p, const void *Q, const void *K, const void *V,
                           const int32_t *idx, const double *sink,
                           int n_rows, const int32_t *rows_b, const int32_t *rows_i,
                           double *O, double *LSE, uint8_t *member)
{
    const int Hq = p->n_q_heads, Hkv = p->n_kv_heads, D = p->head_dim, k = p->k_sel;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r)
        hs2o_sparse_attn_row(p, Q, K, V, idx + (int64_t)r * Hkv * k, sink, rows_b[r], rows_i[r],
                             O + (int64_t)r * Hq * D, LSE + (int64_t)r * Hq,
                             member ? member + (int64_t)r * Hkv * p->kv_len : NULL);
}
