// Host side of liba2sgd: argument checks, launch geometry, kernel dispatch.
// The operations and their citations are documented in include/a2sgd.h.
#include "../../include/a2sgd.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <new>

#include "a2sgd_kernels.cuh"

using namespace a2sgd;

struct a2sgd_ctx {
    uint64_t n = 0;
    uint32_t P = 0;
    int device = 0;
    uint32_t flags = 0;
    bool alg1 = false;
    int sm_count = 0;
    // scratch (device)
    Partial *partials = nullptr;
    uint32_t g_alloc = 0; // CTAs per worker the partials array can hold
    float *local_means = nullptr;
    float *global_means = nullptr;
    unsigned long long *pos_counts = nullptr;
    unsigned int *tickets = nullptr;
    int *status = nullptr;
    // resident CTAs per SM of each kernel family (occupancy API, queried once)
    int occ_encode = 0;
    int occ_decode_shared = 0;
    int occ_decode_repl = 0;
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        target = dev;
    }
    ~DeviceGuard()
    {
        if (ok && prev >= 0 && prev != target) cudaSetDevice(prev);
    }
    int target = -1;
};

#define A2_CUDA(call)                                  \
    do {                                               \
        if ((call) != cudaSuccess) {                   \
            (void)cudaGetLastError();                  \
            return A2SGD_ERR_CUDA;                     \
        }                                              \
    } while (0)

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

inline bool stride_ok(int64_t stride, uint64_t n, uint32_t P)
{
    return P == 1 || (stride >= 0 && (uint64_t)stride >= n);
}

// 16-byte aligned base and (for P > 1) worker stride a multiple of 4 elements
inline bool vec_ok(const void *p, int64_t stride, uint32_t P)
{
    return p == nullptr || (aligned(p, 16) && (P == 1 || stride % 4 == 0));
}

// CTAs per worker for a (G, P) grid that fills the device exactly once.
inline uint32_t per_worker_grid(const a2sgd_ctx *c, int occ, uint64_t items)
{
    const uint64_t slots = (uint64_t)c->sm_count * (uint64_t)std::max(occ, 1);
    uint64_t G = std::max<uint64_t>(1, slots / c->P);
    const uint64_t need = std::max<uint64_t>(1, (items + kBlock - 1) / kBlock);
    G = std::min(G, need);
    return (uint32_t)std::min<uint64_t>(G, c->g_alloc);
}

inline uint32_t flat_grid(const a2sgd_ctx *c, int occ, uint64_t items)
{
    const uint64_t slots = (uint64_t)c->sm_count * (uint64_t)std::max(occ, 1);
    const uint64_t need = std::max<uint64_t>(1, (items + kBlock - 1) / kBlock);
    return (uint32_t)std::min(slots, need);
}

template <typename K>
int occupancy(K kernel)
{
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kBlock, 0) != cudaSuccess) {
        (void)cudaGetLastError();
        return 1;
    }
    return std::max(occ, 1);
}

// ---------------------------------------------------------------- launches
int launch_encode(a2sgd_ctx *c, const float *grad, int64_t gs, const float *err, int64_t es,
                  float *local_means, unsigned long long *pos_counts, uint32_t *pos_mask,
                  float *global_means, cudaStream_t s)
{
    const bool ef = !c->alg1;
    const bool vec = vec_ok(grad, gs, c->P) && (!ef || vec_ok(err, es, c->P));
    EncodeArgs a{};
    a.grad = grad;
    a.grad_stride = gs;
    a.err = ef ? err : nullptr;
    a.err_stride = es;
    a.n = c->n;
    a.P = c->P;
    a.partials = c->partials;
    a.tickets = c->tickets;
    a.status = c->status;
    a.local_means = local_means;
    a.pos_counts = pos_counts;
    a.pos_mask = pos_mask;
    a.global_means = global_means;
    a.ctx_local_means = c->local_means;
    a.ctx_pos_counts = c->pos_counts;
    const uint64_t items = vec ? (c->n + 3) / 4 : c->n;
    const dim3 grid(per_worker_grid(c, c->occ_encode, items), c->P);
    const bool mask = pos_mask != nullptr;
#define A2_ENC(KERNEL)                                                      \
    do {                                                                    \
        if (ef && mask) KERNEL<true, true><<<grid, kBlock, 0, s>>>(a);      \
        else if (ef) KERNEL<true, false><<<grid, kBlock, 0, s>>>(a);        \
        else if (mask) KERNEL<false, true><<<grid, kBlock, 0, s>>>(a);      \
        else KERNEL<false, false><<<grid, kBlock, 0, s>>>(a);               \
    } while (0)
    if (vec) A2_ENC(k_encode_vec);
    else A2_ENC(k_encode_scalar);
#undef A2_ENC
    A2_CUDA(cudaGetLastError());
    return A2SGD_OK;
}

template <bool EF, bool STORE>
void launch_decode_shared(const DecodeArgs &a, uint32_t grid, cudaStream_t s)
{
    switch (a.P) {
    case 1: k_decode_shared_vec<EF, STORE, 1><<<grid, kBlock, 0, s>>>(a); break;
    case 2: k_decode_shared_vec<EF, STORE, 2><<<grid, kBlock, 0, s>>>(a); break;
    case 4: k_decode_shared_vec<EF, STORE, 4><<<grid, kBlock, 0, s>>>(a); break;
    case 8: k_decode_shared_vec<EF, STORE, 8><<<grid, kBlock, 0, s>>>(a); break;
    default: k_decode_shared_vec<EF, STORE, 0><<<grid, kBlock, 0, s>>>(a); break;
    }
}

int launch_decode(a2sgd_ctx *c, float *w, int64_t ws, const float *grad, int64_t gs, float *err,
                  int64_t es, const float *local_means, const float *global_means, float lr,
                  cudaStream_t s)
{
    const bool ef = !c->alg1;
    const bool store = ef || err != nullptr;
    const bool shared = ws == 0;
    const bool vec = vec_ok(grad, gs, c->P) && vec_ok(err, es, c->P) && vec_ok(w, shared ? 4 : ws, c->P);
    DecodeArgs a{};
    a.w = w;
    a.w_stride = ws;
    a.grad = grad;
    a.grad_stride = gs;
    a.err = err;
    a.err_stride = es;
    a.n = c->n;
    a.P = c->P;
    a.local_means = local_means;
    a.global_means = global_means;
    a.lr = lr;
    if (vec && shared) {
        const uint32_t grid = flat_grid(c, c->occ_decode_shared, (c->n + 3) / 4);
        if (ef) launch_decode_shared<true, true>(a, grid, s);
        else if (store) launch_decode_shared<false, true>(a, grid, s);
        else launch_decode_shared<false, false>(a, grid, s);
    } else if (vec) {
        const dim3 grid(per_worker_grid(c, c->occ_decode_repl, (c->n + 3) / 4), c->P);
        if (ef) k_decode_repl_vec<true, true><<<grid, kBlock, 0, s>>>(a);
        else if (store) k_decode_repl_vec<false, true><<<grid, kBlock, 0, s>>>(a);
        else k_decode_repl_vec<false, false><<<grid, kBlock, 0, s>>>(a);
    } else {
        const dim3 grid = shared ? dim3(flat_grid(c, 8, c->n), 1)
                                 : dim3(per_worker_grid(c, 8, c->n), c->P);
        if (ef) k_decode_scalar<true, true><<<grid, kBlock, 0, s>>>(a);
        else if (store) k_decode_scalar<false, true><<<grid, kBlock, 0, s>>>(a);
        else k_decode_scalar<false, false><<<grid, kBlock, 0, s>>>(a);
    }
    A2_CUDA(cudaGetLastError());
    return A2SGD_OK;
}

int check_common(const a2sgd_ctx *c, const float *grad, int64_t gs, const float *err, int64_t es,
                 bool err_required)
{
    if (!c || !grad) return A2SGD_ERR_ARG;
    if (err_required && !err) return A2SGD_ERR_ARG;
    if (!stride_ok(gs, c->n, c->P)) return A2SGD_ERR_ARG;
    if (err && !stride_ok(es, c->n, c->P)) return A2SGD_ERR_ARG;
    if (!aligned(grad, 4) || (err && !aligned(err, 4))) return A2SGD_ERR_ALIGN;
    return A2SGD_OK;
}

} // namespace

// ---------------------------------------------------------------- public API
extern "C" int a2sgd_create(a2sgd_ctx **out, uint64_t n, uint32_t P, int device, uint32_t flags)
{
    if (!out) return A2SGD_ERR_ARG;
    *out = nullptr;
    const uint32_t known = A2SGD_MODE_ALG1 | A2SGD_FORCE_TWO_PASS | A2SGD_FORCE_COOPERATIVE;
    if (n == 0 || n >= (1ull << 40) || P == 0 || P > (uint32_t)kMaxP || (flags & ~known)) return A2SGD_ERR_ARG;
    if ((flags & A2SGD_FORCE_TWO_PASS) && (flags & A2SGD_FORCE_COOPERATIVE)) return A2SGD_ERR_ARG;
    int count = 0;
    A2_CUDA(cudaGetDeviceCount(&count));
    if (device < 0 || device >= count) return A2SGD_ERR_ARG;
    DeviceGuard guard(device);
    if (!guard.ok) return A2SGD_ERR_CUDA;

    a2sgd_ctx *c = new (std::nothrow) a2sgd_ctx();
    if (!c) return A2SGD_ERR_NOMEM;
    c->n = n;
    c->P = P;
    c->device = device;
    c->flags = flags;
    c->alg1 = (flags & A2SGD_MODE_ALG1) != 0;
    if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
        delete c;
        return A2SGD_ERR_CUDA;
    }
    if (c->alg1) {
        c->occ_encode = occupancy(k_encode_vec<false, false>);
        c->occ_decode_repl = occupancy(k_decode_repl_vec<false, true>);
    } else {
        c->occ_encode = occupancy(k_encode_vec<true, false>);
        c->occ_decode_repl = occupancy(k_decode_repl_vec<true, true>);
    }
    switch (P) {
    case 1: c->occ_decode_shared = c->alg1 ? occupancy(k_decode_shared_vec<false, true, 1>) : occupancy(k_decode_shared_vec<true, true, 1>); break;
    case 2: c->occ_decode_shared = c->alg1 ? occupancy(k_decode_shared_vec<false, true, 2>) : occupancy(k_decode_shared_vec<true, true, 2>); break;
    case 4: c->occ_decode_shared = c->alg1 ? occupancy(k_decode_shared_vec<false, true, 4>) : occupancy(k_decode_shared_vec<true, true, 4>); break;
    case 8: c->occ_decode_shared = c->alg1 ? occupancy(k_decode_shared_vec<false, true, 8>) : occupancy(k_decode_shared_vec<true, true, 8>); break;
    default: c->occ_decode_shared = c->alg1 ? occupancy(k_decode_shared_vec<false, true, 0>) : occupancy(k_decode_shared_vec<true, true, 0>); break;
    }
    // partials: room for a (G, P) grid that fills the device at the highest possible occupancy
    const uint32_t max_slots = (uint32_t)c->sm_count * (2048 / kBlock);
    c->g_alloc = std::max<uint32_t>(1, max_slots / P);
    bool ok = true;
    ok = ok && cudaMalloc(&c->partials, sizeof(Partial) * (size_t)c->g_alloc * P) == cudaSuccess;
    ok = ok && cudaMalloc(&c->local_means, sizeof(float) * 2 * P) == cudaSuccess;
    ok = ok && cudaMalloc(&c->global_means, sizeof(float) * 2) == cudaSuccess;
    ok = ok && cudaMalloc(&c->pos_counts, sizeof(unsigned long long) * P) == cudaSuccess;
    ok = ok && cudaMalloc(&c->tickets, sizeof(unsigned int) * (P + 1)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->status, sizeof(int)) == cudaSuccess;
    ok = ok && cudaMemset(c->local_means, 0, sizeof(float) * 2 * P) == cudaSuccess;
    ok = ok && cudaMemset(c->global_means, 0, sizeof(float) * 2) == cudaSuccess;
    ok = ok && cudaMemset(c->pos_counts, 0, sizeof(unsigned long long) * P) == cudaSuccess;
    ok = ok && cudaMemset(c->tickets, 0, sizeof(unsigned int) * (P + 1)) == cudaSuccess;
    ok = ok && cudaMemset(c->status, 0, sizeof(int)) == cudaSuccess;
    ok = ok && cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) {
        (void)cudaGetLastError();
        a2sgd_destroy(c);
        return A2SGD_ERR_NOMEM;
    }
    *out = c;
    return A2SGD_OK;
}

extern "C" int a2sgd_destroy(a2sgd_ctx *c)
{
    if (!c) return A2SGD_OK;
    DeviceGuard guard(c->device);
    cudaFree(c->partials);
    cudaFree(c->local_means);
    cudaFree(c->global_means);
    cudaFree(c->pos_counts);
    cudaFree(c->tickets);
    cudaFree(c->status);
    (void)cudaGetLastError();
    delete c;
    return A2SGD_OK;
}

extern "C" int a2sgd_encode(a2sgd_ctx *c, const float *grad, int64_t grad_stride, const float *err,
                            int64_t err_stride, float *local_means, uint64_t *pos_counts,
                            uint32_t *pos_mask, void *stream)
{
    if (!c || !local_means) return A2SGD_ERR_ARG;
    const int rc = check_common(c, grad, grad_stride, err, err_stride, !c->alg1);
    if (rc) return rc;
    if (!aligned(local_means, 4) || (pos_counts && !aligned(pos_counts, 8)) || (pos_mask && !aligned(pos_mask, 4)))
        return A2SGD_ERR_ALIGN;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    return launch_encode(c, grad, grad_stride, err, err_stride, local_means,
                         reinterpret_cast<unsigned long long *>(pos_counts), pos_mask, nullptr,
                         static_cast<cudaStream_t>(stream));
}

extern "C" int a2sgd_global_average(a2sgd_ctx *c, const float *local_means, float *global_means, void *stream)
{
    if (!c || !local_means || !global_means) return A2SGD_ERR_ARG;
    if (!aligned(local_means, 4) || !aligned(global_means, 4)) return A2SGD_ERR_ALIGN;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    k_global_average<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(local_means, c->P, global_means,
                                                                     c->global_means);
    A2_CUDA(cudaGetLastError());
    return A2SGD_OK;
}

extern "C" int a2sgd_decode_update(a2sgd_ctx *c, float *w, int64_t w_stride, const float *grad,
                                   int64_t grad_stride, float *err, int64_t err_stride,
                                   const float *local_means, const float *global_means, float lr,
                                   void *stream)
{
    if (!c || !w || !global_means) return A2SGD_ERR_ARG;
    const int rc = check_common(c, grad, grad_stride, err, err_stride, !c->alg1);
    if (rc) return rc;
    if (c->alg1 && !local_means) return A2SGD_ERR_ARG;
    if (w_stride != 0 && !stride_ok(w_stride, c->n, c->P)) return A2SGD_ERR_ARG;
    if (!aligned(w, 4) || !aligned(global_means, 4) || (local_means && !aligned(local_means, 4)))
        return A2SGD_ERR_ALIGN;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    return launch_decode(c, w, (c->P == 1) ? 0 : w_stride, grad, grad_stride, err, err_stride, local_means,
                         global_means, lr, static_cast<cudaStream_t>(stream));
}

extern "C" int a2sgd_step(a2sgd_ctx *c, float *w, int64_t w_stride, const float *grad, int64_t grad_stride,
                          float *err, int64_t err_stride, float lr, void *stream)
{
    if (!c || !w) return A2SGD_ERR_ARG;
    const int rc = check_common(c, grad, grad_stride, err, err_stride, !c->alg1);
    if (rc) return rc;
    if (w_stride != 0 && !stride_ok(w_stride, c->n, c->P)) return A2SGD_ERR_ARG;
    if (!aligned(w, 4)) return A2SGD_ERR_ALIGN;
    if (c->flags & A2SGD_FORCE_COOPERATIVE) return A2SGD_ERR_TOO_LARGE;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int r1 = launch_encode(c, grad, grad_stride, err, err_stride, c->local_means, c->pos_counts, nullptr,
                                 c->global_means, s);
    if (r1) return r1;
    return launch_decode(c, w, (c->P == 1) ? 0 : w_stride, grad, grad_stride, err, err_stride, c->local_means,
                         c->global_means, lr, s);
}

extern "C" int a2sgd_step_host(a2sgd_ctx *c, float *w, int64_t w_stride, const float *grad_host,
                               int64_t grad_host_stride, float *grad_staging, int64_t grad_stride,
                               float *err, int64_t err_stride, float lr, float *means_host, void *stream)
{
    if (!c || !grad_host || !grad_staging || !means_host) return A2SGD_ERR_ARG;
    if (!stride_ok(grad_host_stride, c->n, c->P)) return A2SGD_ERR_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    {
        // validate the device-side arguments before any copy is enqueued
        const int rc = check_common(c, grad_staging, grad_stride, err, err_stride, !c->alg1);
        if (rc) return rc;
        if (!w || (w_stride != 0 && !stride_ok(w_stride, c->n, c->P))) return A2SGD_ERR_ARG;
    }
    for (uint32_t p = 0; p < c->P; ++p)
        A2_CUDA(cudaMemcpyAsync(grad_staging + (int64_t)p * grad_stride, grad_host + (int64_t)p * grad_host_stride,
                                sizeof(float) * c->n, cudaMemcpyHostToDevice, s));
    const int rc = a2sgd_step(c, w, w_stride, grad_staging, grad_stride, err, err_stride, lr, stream);
    if (rc) return rc;
    A2_CUDA(cudaMemcpyAsync(means_host, c->local_means, sizeof(float) * 2 * c->P, cudaMemcpyDeviceToHost, s));
    A2_CUDA(cudaMemcpyAsync(means_host + 2 * c->P, c->global_means, sizeof(float) * 2, cudaMemcpyDeviceToHost, s));
    A2_CUDA(cudaStreamSynchronize(s));
    return A2SGD_OK;
}

extern "C" int a2sgd_read_stats(a2sgd_ctx *c, float *local_means_host, float *global_means_host,
                                uint64_t *pos_counts_host, int *device_status, void *stream)
{
    if (!c) return A2SGD_ERR_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (local_means_host)
        A2_CUDA(cudaMemcpyAsync(local_means_host, c->local_means, sizeof(float) * 2 * c->P, cudaMemcpyDeviceToHost, s));
    if (global_means_host)
        A2_CUDA(cudaMemcpyAsync(global_means_host, c->global_means, sizeof(float) * 2, cudaMemcpyDeviceToHost, s));
    if (pos_counts_host)
        A2_CUDA(cudaMemcpyAsync(pos_counts_host, c->pos_counts, sizeof(uint64_t) * c->P, cudaMemcpyDeviceToHost, s));
    int st = 0;
    A2_CUDA(cudaMemcpyAsync(&st, c->status, sizeof(int), cudaMemcpyDeviceToHost, s));
    A2_CUDA(cudaMemsetAsync(c->status, 0, sizeof(int), s));
    A2_CUDA(cudaStreamSynchronize(s));
    if (device_status) *device_status = st;
    return A2SGD_OK;
}

extern "C" int a2sgd_launch_info(a2sgd_ctx *c, int64_t w_stride, uint32_t out[5])
{
    if (!c || !out) return A2SGD_ERR_ARG;
    const uint64_t items = (c->n + 3) / 4;
    out[0] = per_worker_grid(c, c->occ_encode, items) * c->P;
    out[1] = (w_stride == 0 || c->P == 1) ? flat_grid(c, c->occ_decode_shared, items)
                                          : per_worker_grid(c, c->occ_decode_repl, items) * c->P;
    out[2] = kBlock;
    out[3] = 0;
    out[4] = (uint32_t)c->sm_count;
    return A2SGD_OK;
}

extern "C" const char *a2sgd_status_string(int status)
{
    switch (status) {
    case A2SGD_OK: return "ok";
    case A2SGD_ERR_ARG: return "invalid argument";
    case A2SGD_ERR_ALIGN: return "pointer not aligned to its element type";
    case A2SGD_ERR_CUDA: return "CUDA runtime error";
    case A2SGD_ERR_TIMEOUT: return "bounded device-side wait ran out";
    case A2SGD_ERR_NONFINITE: return "non-finite group sum";
    case A2SGD_ERR_NOMEM: return "scratch allocation failed";
    case A2SGD_ERR_TOO_LARGE: return "n*P too large for the single-launch path";
    default: return "unknown status";
    }
}
