/*
 * TEST INFRASTRUCTURE ONLY -- the CPU oracle for shared-prefix decode attention.
 *
 * This file is the plain definition of the operator, written out in fp64 so a
 * reader can check it by eye.  It is slow on purpose, shares nothing with the
 * CUDA library, and may only be used by the tests, the smoke check and the
 * CPU-baseline leg of the benchmark.  The product never calls it.
 *
 * Operator (paper, Appendix "Benchmark details", group "attn":
 * softmax(S) . V with S = Q K^T; the same statement appears as the PyTorch
 * reference of attn task 0, a softmax over the key axis followed by a batched
 * product with V).  One decode step: every sample s of prompt p owns one query
 * per query head h and attends, without any mask, to the L_p prompt tokens it
 * shares with its sibling samples followed by its own S_s generated tokens.
 * Query head h reads KV head floor(h / G), G = H_q / H_kv.
 *
 *   x_j   = sm_scale * sum_d q[s,h,d] * k_j[d]
 *   m     = max_j x_j
 *   w_j   = exp(x_j - m),  Z = sum_j w_j
 *   out   = (sum_j w_j v_j) / Z
 *   lse   = m + ln Z                       (natural logarithm)
 *   empty context: out = 0, lse = -inf
 *
 * Cascades: the shared part of a context may itself be layered (demonstrations shared by every task, task
 * text shared by the task's samples: Algorithm 1's sampling step).  A prefix GROUP g is a run of prefix_lens[g]
 * consecutive tokens of the packed prefix arrays attended by samples [first_sample[g], first_sample[g] +
 * n_samples[g]); a sample's context is every group that contains it, in group order, then its own tokens.
 * The flat case (first_sample == NULL) is "group p = prompt p, samples handed out in order".
 *
 * q, k and v arrive as bf16 bit patterns and are widened exactly.
 * Suffix token t of sample s lives in physical page
 * page_indices[page_indptr[s] + t / page_size], slot t % page_size.
 *
 * Every function here is pinned by tests/test_oracle_pins.py against closed
 * forms, brute force, a library softmax and the paper's streaming recurrences.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_f64(uint16_t bits)
{
    uint32_t w = ((uint32_t)bits) << 16; /* bf16 is the top half of an IEEE float */
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

typedef struct {
    int num_prefixes;
    const int32_t *prefix_lens;   /* [P] */
    const int32_t *n_samples;     /* [P] */
    const int32_t *first_sample;  /* [P] or NULL (groups are consecutive prompts) */
    int32_t num_samples;          /* B */
    int num_q_heads, num_kv_heads, head_dim, page_size;
    double sm_scale;
    const uint16_t *q;            /* [B, Hq, D] */
    const uint16_t *prefix_k, *prefix_v; /* token t of prompt p, head kv at (off_p + t)*stride_tok + kv*stride_head */
    int64_t prefix_stride_tok, prefix_stride_head;
    const uint16_t *pool_k, *pool_v;     /* page*stride_page + kv*stride_head + slot*stride_tok */
    int64_t pool_stride_page, pool_stride_head, pool_stride_tok;
    const int32_t *page_indptr;   /* [B+1] */
    const int32_t *page_indices;
    const int32_t *suffix_lens;   /* [B] */
} psa_oracle_problem;

/* Samples [*first, *first + n_samples[g]) of group g. */
static int64_t group_first(const psa_oracle_problem *pb, int g)
{
    if (pb->first_sample) return pb->first_sample[g];
    int64_t first = 0;
    for (int p = 0; p < g; ++p) first += pb->n_samples[p];
    return first;
}

/* Address of key / value number j of the context of sample s, kv head `kv`; *n receives the context length
 * when j < 0.  Walks the groups and then the page table: deliberately the slow, obvious way. */
static const uint16_t *context_row(const psa_oracle_problem *pb, int s, int kv, int64_t j, int want_v, int64_t *n)
{
    int64_t seen = 0, tok_off = 0;
    for (int g = 0; g < pb->num_prefixes; ++g) {
        const int64_t first = group_first(pb, g), L = pb->prefix_lens[g];
        if (s >= first && s < first + pb->n_samples[g]) {
            if (j >= 0 && j < seen + L) {
                const uint16_t *base = want_v ? pb->prefix_v : pb->prefix_k;
                return base + (tok_off + (j - seen)) * pb->prefix_stride_tok + kv * pb->prefix_stride_head;
            }
            seen += L;
        }
        tok_off += L;
    }
    const int64_t S = pb->suffix_lens[s];
    if (j >= 0 && j < seen + S) {
        const int64_t t = j - seen;
        const int64_t page = pb->page_indices[pb->page_indptr[s] + t / pb->page_size];
        const uint16_t *base = want_v ? pb->pool_v : pb->pool_k;
        return base + page * pb->pool_stride_page + kv * pb->pool_stride_head + (t % pb->page_size) * pb->pool_stride_tok;
    }
    if (n) *n = seen + S;
    return NULL;
}

/* One (sample, query head) row, two passes over the concatenated context.
 * weights (optional, length n) receives w_j / Z. Returns the context length. */
static int64_t attend_row(const psa_oracle_problem *pb, int s, int h, double *x /* scratch, >= n */,
                          double *out, double *lse, double *weights)
{
    const int D = pb->head_dim;
    const int G = pb->num_q_heads / pb->num_kv_heads;
    const int kv = h / G;
    int64_t n = 0;
    context_row(pb, s, kv, -1, 0, &n);
    const uint16_t *qrow = pb->q + ((int64_t)s * pb->num_q_heads + h) * D;

    for (int d = 0; d < D; ++d) out[d] = 0.0;
    if (n == 0) { *lse = -INFINITY; return 0; }

    /* pass 1: logits and their maximum */
    double m = -INFINITY;
    for (int64_t j = 0; j < n; ++j) {
        const uint16_t *krow = context_row(pb, s, kv, j, 0, NULL);
        double dot = 0.0;
        for (int d = 0; d < D; ++d) dot += bf16_to_f64(qrow[d]) * bf16_to_f64(krow[d]);
        x[j] = pb->sm_scale * dot;
        if (x[j] > m) m = x[j];
    }
    /* pass 2: weights, normaliser, weighted sum of values */
    double Z = 0.0;
    for (int64_t j = 0; j < n; ++j) {
        const uint16_t *vrow = context_row(pb, s, kv, j, 1, NULL);
        double w = exp(x[j] - m);
        x[j] = w;
        Z += w;
        for (int d = 0; d < D; ++d) out[d] += w * bf16_to_f64(vrow[d]);
    }
    for (int d = 0; d < D; ++d) out[d] /= Z;
    if (weights) for (int64_t j = 0; j < n; ++j) weights[j] = x[j] / Z;
    *lse = m + log(Z);
    return n;
}

/*
 * Attend for a list of rows.  rows[i] = s * Hq + h selects (sample, query head);
 * rows == NULL means all B*Hq rows in order.  out is [n_rows, D] fp64, lse [n_rows].
 * n_threads <= 0 uses every core OpenMP sees.  Returns 0, or -1 on a bad row /
 * allocation failure.  *threads_used (optional) reports the team size.
 */
int psa_oracle_attend(const psa_oracle_problem *pb, const int64_t *rows, int64_t n_rows,
                      double *out, double *lse, int n_threads, int *threads_used)
{
    const int64_t B = pb->num_samples;
    int64_t max_ctx = 1;
    {   /* no context is longer than all prefix tokens plus the longest suffix */
        int64_t sumL = 0, maxS = 0;
        for (int p = 0; p < pb->num_prefixes; ++p) sumL += pb->prefix_lens[p];
        for (int64_t s = 0; s < B; ++s) if (pb->suffix_lens[s] > maxS) maxS = pb->suffix_lens[s];
        max_ctx = sumL + maxS + 1;
    }
    if (rows == NULL) n_rows = B * pb->num_q_heads;
    int failed = 0, team = 1;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#pragma omp parallel
#endif
    {
        double *x = (double *)malloc(sizeof(double) * (size_t)max_ctx);
#ifdef _OPENMP
#pragma omp single
        team = omp_get_num_threads();
#pragma omp for schedule(dynamic, 1)
#endif
        for (int64_t i = 0; i < n_rows; ++i) {
            int64_t r = rows ? rows[i] : i;
            if (!x || r < 0 || r >= B * pb->num_q_heads) { failed = 1; continue; }
            int s = (int)(r / pb->num_q_heads), h = (int)(r % pb->num_q_heads);
            attend_row(pb, s, h, x, out + i * pb->head_dim, lse + i, NULL);
        }
        free(x);
    }
    if (threads_used) *threads_used = team;
    return failed ? -1 : 0;
}

/* Softmax weights w_j / Z of one row over its concatenated context. */
int64_t psa_oracle_weights(const psa_oracle_problem *pb, int s, int h, double *weights, int64_t capacity)
{
    if (s < 0 || s >= pb->num_samples) return -1;
    int64_t n = 0;
    context_row(pb, s, 0, -1, 0, &n);
    if (n > capacity) return -1;
    double *x = (double *)malloc(sizeof(double) * (size_t)(n + 1));
    double *o = (double *)malloc(sizeof(double) * (size_t)pb->head_dim);
    double l;
    if (!x || !o) { free(x); free(o); return -1; }
    attend_row(pb, s, h, x, o, &l, weights);
    free(x); free(o);
    return n;
}

/*
 * The step before the path: causal self-attention of packed prompts (prefill).  Token i of a prompt attends to
 * tokens 0..i of the same prompt; otherwise exactly the operator above (same scale, same GQA mapping, same two
 * passes).  q is [T, Hq, D], k and v are [T, Hkv, D] bf16 bit patterns, prompts packed back to back;
 * rows[i] = token * Hq + head (NULL = all), out [n_rows, D], lse [n_rows].
 */
int psa_oracle_causal(int num_prompts, const int32_t *prompt_lens, int num_q_heads, int num_kv_heads, int head_dim,
                      double sm_scale, const uint16_t *q, const uint16_t *k, const uint16_t *v,
                      const int64_t *rows, int64_t n_rows, double *out, double *lse, int n_threads)
{
    int64_t T = 0, maxL = 1;
    for (int p = 0; p < num_prompts; ++p) { T += prompt_lens[p]; if (prompt_lens[p] > maxL) maxL = prompt_lens[p]; }
    if (rows == NULL) n_rows = T * num_q_heads;
    const int D = head_dim, G = num_q_heads / num_kv_heads;
    int failed = 0;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#pragma omp parallel
#endif
    {
        double *x = (double *)malloc(sizeof(double) * (size_t)maxL);
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
        for (int64_t i = 0; i < n_rows; ++i) {
            const int64_t r = rows ? rows[i] : i;
            if (!x || r < 0 || r >= T * num_q_heads) { failed = 1; continue; }
            const int64_t tok = r / num_q_heads;
            const int h = (int)(r % num_q_heads), kv = h / G;
            int64_t first = 0;                       /* first token of the prompt that holds `tok` */
            for (int p = 0; p < num_prompts; ++p) { if (tok < first + prompt_lens[p]) break; first += prompt_lens[p]; }
            const int64_t n = tok - first + 1;       /* the token's own key is the last one it sees */
            const uint16_t *qrow = q + (tok * num_q_heads + h) * D;
            double m = -INFINITY, Z = 0.0;
            for (int64_t j = 0; j < n; ++j) {
                const uint16_t *krow = k + ((first + j) * num_kv_heads + kv) * D;
                double dot = 0.0;
                for (int d = 0; d < D; ++d) dot += bf16_to_f64(qrow[d]) * bf16_to_f64(krow[d]);
                x[j] = sm_scale * dot;
                if (x[j] > m) m = x[j];
            }
            double *o = out + i * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            for (int64_t j = 0; j < n; ++j) {
                const uint16_t *vrow = v + ((first + j) * num_kv_heads + kv) * D;
                const double w = exp(x[j] - m);
                Z += w;
                for (int d = 0; d < D; ++d) o[d] += w * bf16_to_f64(vrow[d]);
            }
            for (int d = 0; d < D; ++d) o[d] /= Z;
            lse[i] = m + log(Z);
        }
        free(x);
    }
    return failed ? -1 : 0;
}
