/*
 * The library driven from plain C through include/a2sgd.h alone: no Python, no torch — device
 * memory from the CUDA runtime, every call through the C ABI.  The data is the hand-worked
 * fixture e1 (one worker, error feedback, two steps; Section 3.1 and Algorithm 1 lines 3-7 worked
 * by hand): after the two steps the weights are back to all ones.
 */
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include "a2sgd.h"

#define CHECK(call)                                                                  \
    do {                                                                             \
        int rc_ = (int)(call);                                                       \
        if (rc_ != 0) {                                                              \
            printf("FAILED %s -> %d (line %d)\n", #call, rc_, __LINE__);            \
            return 1;                                                                \
        }                                                                            \
    } while (0)

static int same(const float *a, const float *b, int n)
{
    for (int i = 0; i < n; ++i)
        if (a[i] != b[i]) return 0;
    return 1;
}

int main(void)
{
    enum { N = 6 };
    const float g_steps[2][N] = {{4, -2, 0, -6, 2, -4}, {-4, 2, 0, 2, -2, 8}};
    const float w_expect[2][N] = {{0, 3, 0, 3, 0, 3}, {1, 1, 1, 1, 1, 1}};
    const float e_expect[2][N] = {{2, 2, -2, -2, 0, 0}, {0, 0, 0, -4, 0, 4}};
    const float means_expect[2][2] = {{2, 4}, {4, 2}};
    const uint64_t count_expect[2] = {3, 3};
    float w_host[N] = {1, 1, 1, 1, 1, 1}, e_host[N] = {0, 0, 0, 0, 0, 0};
    float *g = NULL, *e = NULL, *w = NULL;
    CHECK(cudaMalloc((void **)&g, sizeof(float) * N));
    CHECK(cudaMalloc((void **)&e, sizeof(float) * N));
    CHECK(cudaMalloc((void **)&w, sizeof(float) * N));
    CHECK(cudaMemcpy(w, w_host, sizeof(w_host), cudaMemcpyHostToDevice));
    CHECK(cudaMemcpy(e, e_host, sizeof(e_host), cudaMemcpyHostToDevice));

    a2sgd_ctx *ctx = NULL;
    CHECK(a2sgd_create(&ctx, N, 1, 0, A2SGD_MODE_EF));
    for (int t = 0; t < 2; ++t) {
        CHECK(cudaMemcpy(g, g_steps[t], sizeof(float) * N, cudaMemcpyHostToDevice));
        CHECK(a2sgd_step(ctx, w, 0, g, N, e, N, 0.5f, NULL));
        float lm[2], gm[2];
        uint64_t cnt = 0;
        int status = 1;
        CHECK(a2sgd_read_stats(ctx, lm, gm, &cnt, &status, NULL));
        CHECK(status);
        CHECK(cudaMemcpy(w_host, w, sizeof(w_host), cudaMemcpyDeviceToHost));
        CHECK(cudaMemcpy(e_host, e, sizeof(e_host), cudaMemcpyDeviceToHost));
        if (!same(lm, means_expect[t], 2) || !same(gm, means_expect[t], 2) || cnt != count_expect[t] ||
            !same(w_host, w_expect[t], N) || !same(e_host, e_expect[t], N)) {
            printf("FAILED step %d: means %g %g count %llu\n", t + 1, lm[0], lm[1], (unsigned long long)cnt);
            return 1;
        }
    }
    /* bad arguments come back as status codes, nothing is launched */
    if (a2sgd_step(ctx, w, 0, g, N, NULL, N, 0.5f, NULL) != A2SGD_ERR_ARG) return 1;
    if (strcmp(a2sgd_status_string(A2SGD_OK), "ok") != 0) return 1;
    CHECK(a2sgd_destroy(ctx));
    cudaFree(g);
    cudaFree(e);
    cudaFree(w);
    printf("ok\n");
    return 0;
}
