/*
 * CPU oracle for the SlimSpec draft LM-head forward.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, fp64.  It exists so that the CUDA library can be checked against
 * something that can be read next to the paper; it shares no code with the CUDA
 * path and must never be called from the product path (only tests, the smoke
 * check and the benchmark's CPU-baseline leg may use it).
 *
 * What it computes (row-vector convention; the paper writes column vectors):
 *   Section 4.1, low-rank head:   logits = W_up W_down h
 *       here  A = W_down^T (d x r),  B = W_up^T (r x V):
 *       z[m][j]     = sum_i h[m][i] * A[i][j]          (rank-r code, never rounded)
 *       logit[m][v] = sum_j z[m][j] * B[j][v]
 *   Section 4.1, standard head:   logits = W_full h,   W = W_full^T (d x V):
 *       logit[m][v] = sum_i h[m][i] * W[i][v]
 *   Section 3.2 names the softmax over the whole vocabulary; the stable form is
 *       mx = max_v logit,  lse = mx + log(sum_v exp(logit - mx)),
 *       logprob[v] = logit[v] - lse
 *   Candidate tokens: the k largest logits of a row, order = (logit descending,
 *       token id ascending), obtained from a full stable sort.
 *
 * Inputs are bf16 bit patterns (uint16_t); each is widened exactly to double.
 * All sums run in double in index order.  Rows may be processed by several
 * OpenMP threads; no sum is split across threads, so results do not depend on
 * the thread count.
 *
 * Pinned by tests/test_oracle_pins.py (identity down-projection, brute force
 * h(AB), a hand-worked integer example, linearity, rank bound, logsumexp = 0,
 * library log-softmax, full-sort top-k, planted ties, a statistical closed form).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_double(uint16_t bits)
{
    uint32_t w = ((uint32_t)bits) << 16;   /* bf16 is the upper half of an IEEE fp32 */
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

int oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* z = h A  (Section 4.1: W_down h).  h: M x d, A: d x r, z: M x r (double). */
void oracle_downproj(const uint16_t *h, const uint16_t *A, int M, int d, int r, double *z)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        double *zm = z + (size_t)m * r;
        for (int j = 0; j < r; ++j) zm[j] = 0.0;
        for (int i = 0; i < d; ++i) {
            double hv = bf16_to_double(h[(size_t)m * d + i]);
            const uint16_t *Ai = A + (size_t)i * r;
            for (int j = 0; j < r; ++j) zm[j] += hv * bf16_to_double(Ai[j]);
        }
    }
}

/* logits = z B  (Section 4.1: W_up applied to the code).  z: M x r double, B: r x V. */
void oracle_upproj(const double *z, const uint16_t *B, int M, int r, int V, double *logits)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        double *lm = logits + (size_t)m * V;
        for (int v = 0; v < V; ++v) lm[v] = 0.0;
        for (int j = 0; j < r; ++j) {
            double zj = z[(size_t)m * r + j];
            const uint16_t *Bj = B + (size_t)j * V;
            for (int v = 0; v < V; ++v) lm[v] += zj * bf16_to_double(Bj[v]);
        }
    }
}

/* Low-rank head logits (Section 4.1).  Returns 0, or -1 if scratch cannot be had. */
int oracle_slimspec_logits(const uint16_t *h, const uint16_t *A, const uint16_t *B,
                           int M, int d, int r, int V, double *logits)
{
    double *z = (double *)malloc((size_t)M * r * sizeof(double));
    if (!z) return -1;
    oracle_downproj(h, A, M, d, r, z);
    oracle_upproj(z, B, M, r, V, logits);
    free(z);
    return 0;
}

/* Standard head logits (Section 4.1: W_full h).  h: M x d, W: d x V. */
void oracle_fullhead_logits(const uint16_t *h, const uint16_t *W, int M, int d, int V,
                            double *logits)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        double *lm = logits + (size_t)m * V;
        for (int v = 0; v < V; ++v) lm[v] = 0.0;
        for (int i = 0; i < d; ++i) {
            double hv = bf16_to_double(h[(size_t)m * d + i]);
            const uint16_t *Wi = W + (size_t)i * V;
            for (int v = 0; v < V; ++v) lm[v] += hv * bf16_to_double(Wi[v]);
        }
    }
}

/* Stable log-softmax over each row; lse (M doubles) may be NULL. */
void oracle_log_softmax(const double *logits, int M, int V, double *logprob, double *lse)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        const double *lm = logits + (size_t)m * V;
        double mx = lm[0];
        for (int v = 1; v < V; ++v) if (lm[v] > mx) mx = lm[v];
        double s = 0.0;
        for (int v = 0; v < V; ++v) s += exp(lm[v] - mx);
        double l = mx + log(s);
        if (lse) lse[m] = l;
        double *pm = logprob + (size_t)m * V;
        for (int v = 0; v < V; ++v) pm[v] = lm[v] - l;
    }
}

typedef struct { double val; int32_t id; } oracle_pair;

static int pair_cmp(const void *a, const void *b)
{
    const oracle_pair *x = (const oracle_pair *)a, *y = (const oracle_pair *)b;
    if (x->val > y->val) return -1;          /* larger value first */
    if (x->val < y->val) return 1;
    return (x->id > y->id) - (x->id < y->id); /* equal values: lower id first */
}

/*
 * Top-k by a full sort of the row.  vals: M x V (any real scores).
 * ids: M x k, topvals: M x k, next_val (M, may be NULL): the (k+1)-th value, or
 * -inf when k == V.  Returns 0, -1 on allocation failure, -2 on bad k.
 */
int oracle_topk(const double *vals, int M, int V, int k, int32_t *ids, double *topvals,
                double *next_val)
{
    if (k < 1 || k > V) return -2;
    int failed = 0;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        oracle_pair *p = (oracle_pair *)malloc((size_t)V * sizeof(oracle_pair));
        if (!p) {
#pragma omp atomic write
            failed = 1;
            continue;
        }
        for (int v = 0; v < V; ++v) { p[v].val = vals[(size_t)m * V + v]; p[v].id = v; }
        qsort(p, (size_t)V, sizeof(oracle_pair), pair_cmp);  /* total order: no ties left */
        for (int j = 0; j < k; ++j) {
            ids[(size_t)m * k + j] = p[j].id;
            topvals[(size_t)m * k + j] = p[j].val;
        }
        if (next_val) next_val[m] = (k < V) ? p[k].val : -INFINITY;
        free(p);
    }
    return failed ? -1 : 0;
}
