/*
 * CPU oracle for scaled dot-product attention.  TEST INFRASTRUCTURE ONLY: this file is the slow,
 * plain statement of what the attention forward pass computes; the tests, the smoke check and the
 * benchmark's CPU-baseline leg are its only callers.  It shares nothing with the CUDA path.
 *
 * What it computes is the definition itself (Eq. 1 of the paper, O = softmax(Q K^T / sqrt(d)) V,
 * with the 1/sqrt(d) factor passed in as `scale` the way Algorithm 1 multiplies S by "scale"):
 * for a query row i and the keys j that row may see,
 *
 *     s_j = scale * sum_t q[i,t] * k[j,t]
 *     p_j = exp(s_j - max_j s_j)
 *     o[i,:] = (sum_j p_j * v[j,:]) / (sum_j p_j)
 *
 * all in fp64, one row at a time, two passes over the keys, no tiling and no running rescale.
 * Under the causal mask row i sees keys 0..i (the diagonal included), so every row sees at least
 * one key and the denominator is never zero.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Number of worker threads the row loop will use. */
int attn_ref_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * One head.  q_rows: [n_rows, d] (the selected query rows, already gathered); row_index[r] is the
 * position of q_rows[r] in the sequence (used only by the causal mask); k, v: [N, d]; out:
 * [n_rows, d].  All row-major fp64.  threads <= 0 means "all the cores OpenMP offers".
 * Returns 0, or -1 on a bad argument or failed scratch allocation.
 */
int attn_ref_rows(const double *q_rows, const int64_t *row_index, int64_t n_rows,
                  const double *k, const double *v, int64_t N, int64_t d,
                  double scale, int causal, int threads, double *out)
{
    if (!q_rows || !row_index || !k || !v || !out || n_rows < 0 || N <= 0 || d <= 0) return -1;
    for (int64_t r = 0; r < n_rows; ++r)
        if (row_index[r] < 0 || row_index[r] >= N) return -1;
    int failed = 0;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#else
    (void)threads;
#endif
#pragma omp parallel
    {
        double *s = (double *)malloc((size_t)N * sizeof(double));
        if (!s) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 4)
        for (int64_t r = 0; r < n_rows; ++r) {
            if (!s) continue;
            const double *qi = q_rows + r * d;
            const int64_t visible = causal ? row_index[r] + 1 : N; /* keys 0 .. visible-1 */
            double smax = -INFINITY;
            for (int64_t j = 0; j < visible; ++j) {
                const double *kj = k + j * d;
                double dot = 0.0;
                for (int64_t t = 0; t < d; ++t) dot += qi[t] * kj[t];
                s[j] = scale * dot;
                if (s[j] > smax) smax = s[j];
            }
            double *oi = out + r * d;
            for (int64_t t = 0; t < d; ++t) oi[t] = 0.0;
            double denom = 0.0;
            for (int64_t j = 0; j < visible; ++j) {
                const double p = exp(s[j] - smax);
                denom += p;
                const double *vj = v + j * d;
                for (int64_t t = 0; t < d; ++t) oi[t] += p * vj[t];
            }
            for (int64_t t = 0; t < d; ++t) oi[t] /= denom;
        }
        free(s);
    }
    return failed ? -1 : 0;
}

/*
 * The softmax denominator of the same definition, as a logarithm: for query row i,
 *
 *     lse[i] = ln sum_j exp(s_j) = max_j s_j + ln sum_j exp(s_j - max_j s_j),   s_j = scale * q[i,:] . k[j,:]
 *
 * over the keys the row may see.  (Not in the paper: it is the per-row quantity a backward pass or a merge of
 * partial attention results needs, and the CUDA path can emit it.)  Arguments as attn_ref_rows; out: [n_rows].
 */
int attn_ref_lse_rows(const double *q_rows, const int64_t *row_index, int64_t n_rows,
                      const double *k, int64_t N, int64_t d, double scale, int causal, int threads, double *out)
{
    if (!q_rows || !row_index || !k || !out || n_rows < 0 || N <= 0 || d <= 0) return -1;
    for (int64_t r = 0; r < n_rows; ++r)
        if (row_index[r] < 0 || row_index[r] >= N) return -1;
    int failed = 0;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#else
    (void)threads;
#endif
#pragma omp parallel
    {
        double *s = (double *)malloc((size_t)N * sizeof(double));
        if (!s) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 4)
        for (int64_t r = 0; r < n_rows; ++r) {
            if (!s) continue;
            const double *qi = q_rows + r * d;
            const int64_t visible = causal ? row_index[r] + 1 : N;
            double smax = -INFINITY;
            for (int64_t j = 0; j < visible; ++j) {
                const double *kj = k + j * d;
                double dot = 0.0;
                for (int64_t t = 0; t < d; ++t) dot += qi[t] * kj[t];
                s[j] = scale * dot;
                if (s[j] > smax) smax = s[j];
            }
            double denom = 0.0;
            for (int64_t j = 0; j < visible; ++j) denom += exp(s[j] - smax);
            out[r] = smax + log(denom);
        }
        free(s);
    }
    return failed ? -1 : 0;
}
