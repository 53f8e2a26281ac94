/* CPU oracle, C restatement of the per-row statistics (test infrastructure only).
 *
 * For every logit row: m = max_v x[v], t = lowest v attaining m, and
 * s = sum_v exp(x[v] - m), all in double precision on the exact input values.
 * These are t* of Algorithm 1 at T = 0 and the soft-max normaliser behind the
 * probabilities of Eq. 3.  It exists because the numpy statement of the same
 * three lines is too slow for the long lock-step runs; the two are pinned to
 * each other and to closed forms in the CPU tests.  Rows are independent and
 * are spread over host threads; nothing else is blocked, fused or reordered:
 * each row is one left-to-right pass for the maximum and one for the sum.
 *
 * This file shares nothing with the CUDA library.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double widen_bf16(uint16_t h)
{
    /* bfloat16 is the upper half of an IEEE binary32 */
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static void one_row_f64(const double *x, int64_t V, double *m, int64_t *t, double *s);

/* dtype: 0 = float32, 1 = bfloat16 (raw 16-bit patterns).
 * `rows` logit rows, row r starting at element offset[r] of `base`.
 * scratch: caller-provided doubles, V per thread (n_threads * V). */
int csd_oracle_row_stats(const void *base, int dtype, int64_t rows, int64_t V,
                         const int64_t *offset, double *m, int64_t *t, double *s,
                         double *scratch, int n_threads)
{
    if (dtype != 0 && dtype != 1) return 1;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int64_t r = 0; r < rows; ++r) {
        int tid = 0;
#ifdef _OPENMP
        tid = omp_get_thread_num();
#endif
        double *x = scratch + (int64_t)tid * V;
        if (dtype == 0) {
            const float *p = (const float *)base + offset[r];
            for (int64_t v = 0; v < V; ++v) x[v] = (double)p[v];
        } else {
            const uint16_t *p = (const uint16_t *)base + offset[r];
            for (int64_t v = 0; v < V; ++v) x[v] = widen_bf16(p[v]);
        }
        one_row_f64(x, V, &m[r], &t[r], &s[r]);
    }
    return 0;
}

static void one_row_f64(const double *x, int64_t V, double *m, int64_t *t, double *s)
{
    double best = x[0];
    int64_t arg = 0;
    for (int64_t v = 1; v < V; ++v) {
        if (x[v] > best) {            /* strict: the lowest index keeps a tie */
            best = x[v];
            arg = v;
        }
    }
    double acc = 0.0;
    for (int64_t v = 0; v < V; ++v) acc += exp(x[v] - best);
    *m = best;
    *t = arg;
    *s = acc;
}

int csd_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
