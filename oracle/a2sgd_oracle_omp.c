/*
 * OpenMP copy of the A2SGD CPU oracle's step — TEST / BENCHMARK INFRASTRUCTURE, not a product path.
 *
 * This file exists for one purpose: the benchmark reports what the host's cores can do on the
 * same path when all of them are used.  It restates a2sgd_oracle_step (Section 3.1, Eq. 2 and
 * Algorithm 1 lines 3-7 of the paper; see a2sgd_oracle.c for the readings taken) with the element
 * loops spread over threads.  The pinned oracle that the parity tests use stays the
 * single-threaded file; this copy shares no code with it and is itself checked against it (the
 * only difference is the order of the fp64 additions inside the group sums, at most an ulp of
 * the fp32 means).
 *
 * Worker p's vector lives at base + p*stride (stride in elements).
 */
#include <stddef.h>
#include <stdint.h>
#include <omp.h>

enum { OMP_MODE_EF = 0, OMP_MODE_ALG1 = 1 };

static inline float value_to_encode(int mode, const float *g, const float *e, int64_t i)
{
    if (mode == OMP_MODE_EF) {
        volatile float v = g[i] + e[i]; /* one fp32 rounding, as on the GPU */
        return v;
    }
    return g[i];
}

int a2sgd_oracle_omp_threads(void) { return omp_get_max_threads(); }

int a2sgd_oracle_omp_step(int mode, uint64_t n, uint32_t P, float *w, int64_t w_stride,
                          const float *grad, int64_t grad_stride, float *err, int64_t err_stride,
                          float lr, float *local_means, float *global_means, uint64_t *pos_counts)
{
    if (n == 0 || P == 0 || !w || !grad || !local_means || !global_means) return -1;
    if (mode == OMP_MODE_EF && !err) return -1;
    /* Algorithm 1 line 3: the two group means of every worker */
    for (uint32_t p = 0; p < P; ++p) {
        const float *g = grad + (int64_t)p * grad_stride;
        const float *e = err ? err + (int64_t)p * err_stride : NULL;
        double s_pos = 0.0, s_neg = 0.0;
        uint64_t n_pos = 0;
#pragma omp parallel for reduction(+ : s_pos, s_neg, n_pos) schedule(static)
        for (int64_t i = 0; i < (int64_t)n; ++i) {
            const float v = value_to_encode(mode, g, e, i);
            if (v >= 0.0f) {
                s_pos += (double)v;
                n_pos += 1;
            } else {
                s_neg += -(double)v;
            }
        }
        const uint64_t n_neg = n - n_pos;
        local_means[2 * p + 0] = n_pos ? (float)(s_pos / (double)n_pos) : 0.0f;
        local_means[2 * p + 1] = n_neg ? (float)(s_neg / (double)n_neg) : 0.0f;
        if (pos_counts) pos_counts[p] = n_pos;
    }
    /* line 5: unweighted average over the workers, in worker order */
    double a_pos = 0.0, a_neg = 0.0;
    for (uint32_t p = 0; p < P; ++p) {
        a_pos += (double)local_means[2 * p + 0];
        a_neg += (double)local_means[2 * p + 1];
    }
    global_means[0] = (float)(a_pos / (double)P);
    global_means[1] = (float)(a_neg / (double)P);
    const double m_pos = (double)global_means[0], m_neg = (double)global_means[1];
    /* lines 4, 6, 7 (or their error-feedback form), element by element */
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)n; ++i) {
        double sum = 0.0;
        for (uint32_t p = 0; p < P; ++p) {
            const float *g = grad + (int64_t)p * grad_stride;
            float *e = err ? err + (int64_t)p * err_stride : NULL;
            const float v = value_to_encode(mode, g, e, i);
            const int is_pos = (v >= 0.0f);
            const double mean_vec = is_pos ? m_pos : -m_neg;
            double g_hat;
            if (mode == OMP_MODE_EF) {
                g_hat = mean_vec;
                e[i] = (float)((double)v - g_hat);
            } else {
                const double enc = is_pos ? (double)local_means[2 * p + 0] : -(double)local_means[2 * p + 1];
                const double eps = (double)v - enc;
                g_hat = eps + mean_vec;
                if (e) e[i] = (float)eps;
            }
            if (w_stride == 0) {
                sum += g_hat;
            } else {
                float *wp = w + (int64_t)p * w_stride;
                wp[i] = (float)((double)wp[i] - (double)lr * g_hat);
            }
        }
        if (w_stride == 0) w[i] = (float)((double)w[i] - (double)lr * sum / (double)P);
    }
    return 0;
}
