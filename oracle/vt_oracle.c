/*
 * CPU oracle for the trimmed-vocabulary draft head.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, double-precision statement of what the head computes, written
 * from the definitions and used to check the CUDA library.  It shares no code,
 * header, table or helper with the CUDA path and must never be called from it.
 * Every floating-point step is fp64 over the exact values of the bf16 inputs;
 * the only concession to speed is a parallel-for over independent vocabulary
 * rows, which does not change any arithmetic.
 *
 * Trimming restricts the index set of the head and approximates nothing, so each
 * function below is the textbook definition of its step:
 *
 *   compact      W_trim[i,:] = W_full[keep_ids[i],:]          (Section 2.1: V_d = the kept tokens)
 *   logits       x[m,i] = sum_j h[m,j] * W_trim[i,j]           (Section 2.3: the d -> k linear head, 2dk FLOPs)
 *   log-softmax  lp[m,i] = x[m,i] - log sum_i' exp(x[m,i'])    (normalised over the kept rows only)
 *   top-k        the k largest x[m,:], ties to the lower draft index
 *   remap        target_id = d2t[draft index]                  (Section 1: draft-to-target index buffer)
 *   coverage     #{t : token_ids[t] in V_d} / N                (Eq. 2, with f = occurrence counts of the stream)
 *
 * Pins (tests with the "not gpu" marker): brute force in exact rational arithmetic
 * on dyadic inputs, one-hot and zero hidden states, exact power-of-two linearity,
 * closed-form two-class and uniform softmax, shift invariance, a k-pass max-scan
 * top-k, the restriction invariant against the full head (bit-for-bit), Eq. 2
 * evaluated from an independent histogram, and O(N*V_trim) membership by brute force.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 is the upper half of an IEEE binary32: widen and convert, both exact. */
double vto_bf16_to_f64(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int vto_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Head compaction: keep the rows named by keep_ids, in that order (Section 2.1). */
void vto_compact(const uint16_t *W_full, int64_t V_full, int64_t d,
                 const int32_t *keep_ids, int64_t V_trim, uint16_t *W_trim)
{
    (void)V_full;
    for (int64_t i = 0; i < V_trim; ++i)
        for (int64_t j = 0; j < d; ++j)
            W_trim[i * d + j] = W_full[(int64_t)keep_ids[i] * d + j];
}

/* logits x[m*V_trim + i] = sum_{j=0}^{d-1} h[m,j] * W[i,j], summed in index order (Section 2.3). */
void vto_logits(const uint16_t *h, const uint16_t *W, int64_t M, int64_t d, int64_t V_trim, double *x)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < V_trim; ++i) {
        for (int64_t m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int64_t j = 0; j < d; ++j)
                acc += vto_bf16_to_f64(h[m * d + j]) * vto_bf16_to_f64(W[i * d + j]);
            x[m * V_trim + i] = acc;
        }
    }
}

/* lse[m] = log sum_i exp(x[m,i]) with the row maximum factored out; lp = x - lse (lp may be NULL). */
void vto_log_softmax(const double *x, int64_t M, int64_t V_trim, double *lp, double *lse)
{
    for (int64_t m = 0; m < M; ++m) {
        const double *row = x + m * V_trim;
        double mx = row[0];
        for (int64_t i = 1; i < V_trim; ++i)
            if (row[i] > mx) mx = row[i];
        double s = 0.0;
        for (int64_t i = 0; i < V_trim; ++i)
            s += exp(row[i] - mx);
        double l = mx + log(s);
        if (lse) lse[m] = l;
        if (lp)
            for (int64_t i = 0; i < V_trim; ++i)
                lp[m * V_trim + i] = row[i] - l;
    }
}

typedef struct { double x; int32_t i; } vto_pair;

static int vto_pair_cmp(const void *a, const void *b)
{
    const vto_pair *p = (const vto_pair *)a, *q = (const vto_pair *)b;
    if (p->x > q->x) return -1;       /* larger logit first */
    if (p->x < q->x) return 1;
    return (p->i > q->i) - (p->i < q->i);   /* equal logits: lower draft index first */
}

/* top-k: order all draft indices by (x descending, index ascending) and keep the first k. */
int vto_topk(const double *x, int64_t M, int64_t V_trim, int64_t k, int32_t *idx)
{
    if (k < 1 || k > V_trim) return 1;
    vto_pair *p = (vto_pair *)malloc((size_t)V_trim * sizeof *p);
    if (!p) return 2;
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t i = 0; i < V_trim; ++i) { p[i].x = x[m * V_trim + i]; p[i].i = (int32_t)i; }
        qsort(p, (size_t)V_trim, sizeof *p, vto_pair_cmp);
        for (int64_t j = 0; j < k; ++j) idx[m * k + j] = p[j].i;
    }
    free(p);
    return 0;
}

/* d2t remap: draft index -> target-vocabulary id (absolute ids). */
void vto_remap(const int32_t *draft_idx, int64_t n, const int32_t *d2t, int32_t *target_ids)
{
    for (int64_t t = 0; t < n; ++t) target_ids[t] = d2t[draft_idx[t]];
}

/* Eq. 2 numerator: occurrences whose id is kept.  Ids outside [0, V_full) are never kept. */
int vto_coverage(const int32_t *token_ids, int64_t N, const int32_t *keep_ids, int64_t V_trim,
                 int64_t V_full, uint64_t *covered)
{
    unsigned char *member = (unsigned char *)calloc((size_t)V_full, 1);
    if (!member) return 2;
    for (int64_t i = 0; i < V_trim; ++i)
        if (keep_ids[i] >= 0 && keep_ids[i] < V_full) member[keep_ids[i]] = 1;
    uint64_t c = 0;
    for (int64_t t = 0; t < N; ++t)
        if (token_ids[t] >= 0 && token_ids[t] < V_full) c += member[token_ids[t]];
    free(member);
    *covered = c;
    return 0;
}

/*
 * The whole call: logits, log-softmax over the kept rows, top-k, log-probs of the
 * winners, remap.  x_out (M*V_trim doubles) receives the logits when non-NULL.
 */
int vto_draft_head(const uint16_t *h, const uint16_t *W_trim, const int32_t *d2t,
                   int64_t M, int64_t d, int64_t V_trim, int64_t k,
                   int32_t *target_ids, double *logprobs, int32_t *draft_ids, double *lse_out,
                   double *x_out)
{
    if (k < 1 || k > V_trim) return 1;
    double *x = x_out ? x_out : (double *)malloc((size_t)(M * V_trim) * sizeof(double));
    double *lse = (double *)malloc((size_t)M * sizeof(double));
    int32_t *idx = (int32_t *)malloc((size_t)(M * k) * sizeof(int32_t));
    if (!x || !lse || !idx) return 2;
    vto_logits(h, W_trim, M, d, V_trim, x);
    vto_log_softmax(x, M, V_trim, NULL, lse);
    int rc = vto_topk(x, M, V_trim, k, idx);
    if (rc == 0) {
        for (int64_t m = 0; m < M; ++m)
            for (int64_t j = 0; j < k; ++j)
                logprobs[m * k + j] = x[m * V_trim + idx[m * k + j]] - lse[m];
        vto_remap(idx, M * k, d2t, target_ids);
        if (draft_ids) memcpy(draft_ids, idx, (size_t)(M * k) * sizeof(int32_t));
        if (lse_out) memcpy(lse_out, lse, (size_t)M * sizeof(double));
    }
    if (!x_out) free(x);
    free(lse);
    free(idx);
    return rc;
}
