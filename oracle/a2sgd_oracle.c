/*
 * A2SGD CPU oracle — TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, single-threaded restatement of what the A2SGD per-worker
 * gradient path computes (two-level gradient averaging: Section 3.1, Eq. 2,
 * Algorithm 1 and Eq. 13 of the paper).  Every loop below is the definition
 * written out: one traversal per worker to form the two group means, one
 * loop over the P pairs of means, one traversal to reconstruct / update.
 * No blocking, no fusion, no reordering, no threads.
 *
 * Only tests, the smoke check and the benchmark's cpu_baseline leg may call
 * this file.  It shares no code, header, table or constant with the CUDA
 * library and includes none of its files.
 *
 * Arithmetic.  Inputs and outputs are fp32 (the paper exchanges "two means,
 * i.e. 64 bits": Section 4.3).  The encoded vector v is formed in fp32 so
 * that the sign decision is taken on the same number the GPU sees; every sum,
 * quotient and update is carried in fp64 and rounded to fp32 once, on store.
 *
 * Two modes (the paper's Algorithm 1 and its prose differ on whether the
 * error vector is carried between iterations):
 *   EF   (mode 0)  v = g + e (retained error added to the fresh gradient),
 *                  g_hat = pos(v)*m_pos - neg(v)*m_neg,  e' = v - g_hat.
 *   ALG1 (mode 1)  v = g; eps = g - enc(g) (Alg. 1 line 4);
 *                  g_hat = eps + pos(g)*m_pos - neg(g)*m_neg (Alg. 1 line 6,
 *                  equivalently Eq. 13: g + (mean vector - enc(g))).
 *
 * Conventions where the paper is silent (none of them is pinned by a value
 * the paper prints — "parity unpinned" for these):
 *   - zero, and IEEE -0.0, belong to the positive group ("positive (>= 0)");
 *     the mask is the IEEE comparison v >= 0, so NaN falls in the negative
 *     group;
 *   - the mean of an empty group is 0, and that worker still counts in the
 *     divide-by-P of the global average;
 *   - with one shared weight vector (w_stride == 0) the P simulated workers
 *     apply the worker-mean of their reconstructed gradients, which is the
 *     mean of the P replicas Algorithm 1 would hold;
 *   - a2sgd_oracle_decode_update_momentum: momentum and weight decay are not
 *     defined by the paper on this path ("parity unpinned" by the paper too);
 *     the heavy-ball reading is stated at that function.
 *
 * Worker p's vector lives at base + p*stride (stride in elements).
 */
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>

enum { ORACLE_MODE_EF = 0, ORACLE_MODE_ALG1 = 1 };

/* The vector that gets encoded.  EF: retained error added to the fresh
 * gradient, rounded to fp32 (one IEEE single-precision add).  ALG1: the
 * gradient itself (Algorithm 1 line 3 takes mu(g_t)). */
static float encoded_value(int mode, const float *g, const float *e, uint64_t i)
{
    if (mode == ORACLE_MODE_EF) {
        volatile float v = g[i] + e[i]; /* volatile: force the fp32 rounding */
        return v;
    }
    return g[i];
}

/*
 * Section 3.1: mu_pos(v) = mean of the entries v_i >= 0, mu_neg(v) = mean of
 * |v_i| over the entries v_i < 0.  Algorithm 1 line 3.
 * local_means[p] = {mu_pos, mu_neg}; pos_counts[p] = #{i : v_i >= 0};
 * pos_mask (optional) packs pos(v): bit b of word j <=> element 32*j + b.
 */
int a2sgd_oracle_encode(int mode, uint64_t n, uint32_t P,
                        const float *grad, int64_t grad_stride,
                        const float *err, int64_t err_stride,
                        float *local_means, uint64_t *pos_counts,
                        uint32_t *pos_mask)
{
    if (n == 0 || P == 0 || !grad || !local_means) return -1;
    if (mode == ORACLE_MODE_EF && !err) return -1;
    const uint64_t words = (n + 31) / 32;
    for (uint32_t p = 0; p < P; ++p) {
        const float *g = grad + (int64_t)p * grad_stride;
        const float *e = err ? err + (int64_t)p * err_stride : NULL;
        double s_pos = 0.0, s_neg = 0.0;
        uint64_t n_pos = 0, n_neg = 0;
        if (pos_mask)
            for (uint64_t j = 0; j < words; ++j) pos_mask[p * words + j] = 0u;
        for (uint64_t i = 0; i < n; ++i) {
            const float v = encoded_value(mode, g, e, i);
            if (v >= 0.0f) {
                s_pos += (double)v;
                n_pos += 1;
                if (pos_mask) pos_mask[p * words + i / 32] |= 1u << (i % 32);
            } else {
                s_neg += -(double)v;
                n_neg += 1;
            }
        }
        local_means[2 * p + 0] = n_pos ? (float)(s_pos / (double)n_pos) : 0.0f;
        local_means[2 * p + 1] = n_neg ? (float)(s_neg / (double)n_neg) : 0.0f;
        if (pos_counts) pos_counts[p] = n_pos;
    }
    return 0;
}

/*
 * Algorithm 1 line 5: Allreduce(average) of the pair of means — the
 * unweighted arithmetic mean over the P workers, summed in worker order.
 */
int a2sgd_oracle_global_average(uint32_t P, const float *local_means,
                                float *global_means)
{
    if (P == 0 || !local_means || !global_means) return -1;
    double s_pos = 0.0, s_neg = 0.0;
    for (uint32_t p = 0; p < P; ++p) {
        s_pos += (double)local_means[2 * p + 0];
        s_neg += (double)local_means[2 * p + 1];
    }
    global_means[0] = (float)(s_pos / (double)P);
    global_means[1] = (float)(s_neg / (double)P);
    return 0;
}

/*
 * Algorithm 1 lines 4, 6, 7 (ALG1) or their error-feedback form (EF):
 * reconstruct g_hat from the two global means, update the residual, apply
 * w <- w - lr * g_hat.  w_stride == 0 selects one shared w (see header).
 * err: EF read-write (required); ALG1 write-only, may be NULL.
 */
int a2sgd_oracle_decode_update(int mode, uint64_t n, uint32_t P,
                               float *w, int64_t w_stride,
                               const float *grad, int64_t grad_stride,
                               float *err, int64_t err_stride,
                               const float *local_means,
                               const float *global_means, float lr)
{
    if (n == 0 || P == 0 || !w || !grad || !global_means) return -1;
    if (mode == ORACLE_MODE_EF && !err) return -1;
    if (mode == ORACLE_MODE_ALG1 && !local_means) return -1;
    const double m_pos = (double)global_means[0];
    const double m_neg = (double)global_means[1];
    double *acc = NULL;
    if (w_stride == 0) {
        acc = (double *)calloc(n, sizeof(double));
        if (!acc) return -6;
    }
    for (uint32_t p = 0; p < P; ++p) {
        const float *g = grad + (int64_t)p * grad_stride;
        float *e = err ? err + (int64_t)p * err_stride : NULL;
        float *wp = w + (int64_t)p * w_stride;
        for (uint64_t i = 0; i < n; ++i) {
            const float v = encoded_value(mode, g, e, i);
            const int is_pos = (v >= 0.0f);
            const double mean_vec = is_pos ? m_pos : -m_neg; /* pos*m+ - neg*m- */
            double g_hat;
            if (mode == ORACLE_MODE_EF) {
                g_hat = mean_vec;
                e[i] = (float)((double)v - g_hat);
            } else {
                const double enc = is_pos ? (double)local_means[2 * p + 0]
                                          : -(double)local_means[2 * p + 1];
                const double eps = (double)v - enc; /* Alg. 1 line 4 */
                g_hat = eps + mean_vec;             /* Alg. 1 line 6 */
                if (e) e[i] = (float)eps;
            }
            if (acc)
                acc[i] += g_hat;
            else
                wp[i] = (float)((double)wp[i] - (double)lr * g_hat); /* line 7 */
        }
    }
    if (acc) {
        for (uint64_t i = 0; i < n; ++i)
            w[i] = (float)((double)w[i] - (double)lr * acc[i] / (double)P);
        free(acc);
    }
    return 0;
}

/*
 * The reconstruct / residual / update step with the optimiser the paper's
 * experiments actually ran on top of Algorithm 1 line 7: SGD with momentum
 * and weight decay (Section 4.1 and Table 1 give the learning-rate policies;
 * Algorithm 1 itself prints the plain step w <- w - lr * g_hat).  The paper
 * compresses the gradient only (Algorithm 1 lines 3-6), so the two terms act
 * on the reconstructed gradient, in the usual heavy-ball form:
 *     u  = g_hat + weight_decay * w        (L2 penalty folded into the gradient)
 *     m <- beta * m + u                    (momentum buffer, no dampening)
 *     w <- w - lr * m
 * "Parity unpinned" by the paper: it defines neither term on this path; the
 * reading above is pinned by beta = weight_decay = 0 (reproduces
 * a2sgd_oracle_decode_update exactly), closed forms and a hand-worked fixture.
 * One shared w (w_stride == 0) has one momentum vector (mom_stride == 0) and
 * receives the worker-mean of g_hat; one replica per worker has one momentum
 * vector per worker.  The residual update is that of a2sgd_oracle_decode_update.
 */
int a2sgd_oracle_decode_update_momentum(int mode, uint64_t n, uint32_t P,
                                        float *w, int64_t w_stride,
                                        float *mom, int64_t mom_stride,
                                        const float *grad, int64_t grad_stride,
                                        float *err, int64_t err_stride,
                                        const float *local_means,
                                        const float *global_means, float lr,
                                        float beta, float weight_decay)
{
    if (n == 0 || P == 0 || !w || !mom || !grad || !global_means) return -1;
    if (mode == ORACLE_MODE_EF && !err) return -1;
    if (mode == ORACLE_MODE_ALG1 && !local_means) return -1;
    if ((w_stride == 0) != (mom_stride == 0) && P > 1) return -1;
    const double m_pos = (double)global_means[0];
    const double m_neg = (double)global_means[1];
    double *acc = NULL;
    if (w_stride == 0) {
        acc = (double *)calloc(n, sizeof(double));
        if (!acc) return -6;
    }
    for (uint32_t p = 0; p < P; ++p) {
        const float *g = grad + (int64_t)p * grad_stride;
        float *e = err ? err + (int64_t)p * err_stride : NULL;
        float *wp = w + (int64_t)p * w_stride;
        float *mp = mom + (int64_t)p * mom_stride;
        for (uint64_t i = 0; i < n; ++i) {
            const float v = encoded_value(mode, g, e, i);
            const int is_pos = (v >= 0.0f);
            const double mean_vec = is_pos ? m_pos : -m_neg;
            double g_hat;
            if (mode == ORACLE_MODE_EF) {
                g_hat = mean_vec;
                e[i] = (float)((double)v - g_hat);
            } else {
                const double enc = is_pos ? (double)local_means[2 * p + 0]
                                          : -(double)local_means[2 * p + 1];
                const double eps = (double)v - enc;
                g_hat = eps + mean_vec;
                if (e) e[i] = (float)eps;
            }
            if (acc) {
                acc[i] += g_hat;
            } else {
                const double u = g_hat + (double)weight_decay * (double)wp[i];
                const double m_new = (double)beta * (double)mp[i] + u;
                mp[i] = (float)m_new;
                wp[i] = (float)((double)wp[i] - (double)lr * m_new);
            }
        }
    }
    if (acc) {
        for (uint64_t i = 0; i < n; ++i) {
            const double u = acc[i] / (double)P + (double)weight_decay * (double)w[i];
            const double m_new = (double)beta * (double)mom[i] + u;
            mom[i] = (float)m_new;
            w[i] = (float)((double)w[i] - (double)lr * m_new);
        }
        free(acc);
    }
    return 0;
}

/*
 * Algorithm 1 lines 9-10: after the last compressed iteration one dense
 * synchronisation — the workers' gradients are averaged element-wise
 * (Allreduce-average of the full vectors) and every worker applies
 * w <- w - lr * mean_p g^p.  This is Eq. 1 (dense distributed SGD) for one
 * step.  w_stride == 0: one shared w; otherwise every replica receives the
 * same averaged update.
 */
int a2sgd_oracle_dense_sync(uint64_t n, uint32_t P, float *w, int64_t w_stride,
                            const float *grad, int64_t grad_stride, float lr)
{
    if (n == 0 || P == 0 || !w || !grad) return -1;
    const uint32_t replicas = (w_stride == 0) ? 1 : P;
    for (uint64_t i = 0; i < n; ++i) {
        double sum = 0.0;
        for (uint32_t p = 0; p < P; ++p)
            sum += (double)grad[(int64_t)p * grad_stride + (int64_t)i];
        const double mean = sum / (double)P;
        for (uint32_t r = 0; r < replicas; ++r) {
            float *wr = w + (int64_t)r * w_stride;
            wr[i] = (float)((double)wr[i] - (double)lr * mean);
        }
    }
    return 0;
}

/* One whole iteration of the loop body of Algorithm 1 for all P workers. */
int a2sgd_oracle_step(int mode, uint64_t n, uint32_t P,
                      float *w, int64_t w_stride,
                      const float *grad, int64_t grad_stride,
                      float *err, int64_t err_stride, float lr,
                      float *local_means, float *global_means,
                      uint64_t *pos_counts)
{
    int rc = a2sgd_oracle_encode(mode, n, P, grad, grad_stride, err, err_stride,
                                 local_means, pos_counts, NULL);
    if (rc) return rc;
    rc = a2sgd_oracle_global_average(P, local_means, global_means);
    if (rc) return rc;
    return a2sgd_oracle_decode_update(mode, n, P, w, w_stride, grad, grad_stride,
                                      err, err_stride, local_means, global_means,
                                      lr);
}
