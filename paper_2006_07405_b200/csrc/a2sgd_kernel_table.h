// The kernels one variant of the library offers (production, or the checked copy used under
// A2SGD_DEBUG_CHECKS), as plain function pointers so that the host dispatch is written once.
#pragma once

#include <stdint.h>

struct a2sgd_kernel_table {
    const void *(*encode)(bool ef, bool mask, int vw);
    const void *(*encode_deferred)(bool err_holds_v);
    const void *(*encode_lowp)(int grad_type, bool ef, int vw);
    const void *(*encode_segments)(bool ef, bool per_tensor_means);
    const void *(*decode_shared)(bool ef, bool store, uint32_t P, int vw, bool momentum);
    const void *(*decode_repl)(bool ef, bool store, int vw, bool momentum);
    const void *(*decode_scalar)(bool ef, bool store, bool momentum);
    const void *(*decode_lowp)(int grad_type, bool ef, bool store, bool shared, uint32_t P, int vw);
    const void *(*decode_deferred)(bool replicated, uint32_t P);
    const void *(*decode_segments)(bool ef, bool store, uint32_t P, bool per_tensor_means);
    const void *(*dense)(uint32_t P, int vw, bool replicated);
    const void *(*coop)(bool ef, bool store, bool shared, uint32_t P);
    const void *(*coop_l2)(bool ef, bool store, bool shared, uint32_t P);
    const void *global_average;           // (const float *local_means, uint32_t P, float *out, float *ctx_copy)
    const void *global_average_from_sums; // (const double *sums, uint32_t workers, float *out, float *ctx_copy)
    const void *materialize_err;          // (float *v, int64_t stride, uint64_t n, const float *means)
    const void *fold_jobs;                // (SegTables)
    const void *fold_segments;            // (SegTables, uint32_t P, int *status)
};
