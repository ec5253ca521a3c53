// a2sgd_encode_noalloc: the encode-reduce step for callers that must not allocate.
//
// The regular entry points need a context, and creating one calls cudaMalloc
// for the reduction scratch (per-CTA partial sums, tickets, status word).
// Some callers cannot do that: a training framework that has handed the
// whole device to its own caching allocator (a raw cudaMalloc then fails or
// fragments the pool), a latency-critical loop in which cudaMalloc's implicit
// device synchronisation is not acceptable, or a plug-in that runs under a
// "no allocation after start-up" rule.  For them this file keeps the scratch
// in a fixed file-scope device array: it is part of the library image, so
// every GPU that loads the library holds these 64 KiB until the process
// exits, and no call here allocates or frees anything.
//
// The array's name is only a host-side stand-in in host code, so its device
// address is looked up with cudaGetSymbolAddress — once per device, on the
// first call made with that device current — and that address is what the
// kernel receives.
#include "../../include/a2sgd.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <mutex>

#define A2SGD_NS a2sgd
#define A2SGD_CHECKED 0
#include "a2sgd_kernels.cuh"

using namespace a2sgd;

namespace {

constexpr uint32_t kNoAllocMaxP = A2SGD_NOALLOC_MAX_P;      // workers per call
constexpr uint32_t kNoAllocMaxCtas = 2048;                  // partial sums the array can hold
constexpr size_t kPartialsBytes = sizeof(Partial) * kNoAllocMaxCtas;            // 49152
constexpr size_t kTicketsOffset = kPartialsBytes;
constexpr size_t kTicketsBytes = sizeof(unsigned int) * (kNoAllocMaxP + 1);     // 260
constexpr size_t kStatusOffset = (kTicketsOffset + kTicketsBytes + 15) / 16 * 16;
constexpr size_t kScratchBytes = 64 * 1024;
static_assert(kStatusOffset + sizeof(int) <= kScratchBytes, "scratch layout exceeds the static array");

// Shared by every call on a device; keeps whatever the last call left in it.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
struct DeviceSetup {
    bool ready = false;
    unsigned char *scratch = nullptr; // device address of g_noalloc_scratch on this device
    int sm_count = 0;
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

// First call on a device: resolve the array's device address and the SM count.
int setup_current_device(int device, DeviceSetup **out)
{
    if (device < 0 || device >= kMaxDevices) return A2SGD_ERR_ARG;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    DeviceSetup &s = g_setup[device];
    if (!s.ready) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) {
            (void)cudaGetLastError();
            return A2SGD_ERR_CUDA;
        }
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms <= 0) {
            (void)cudaGetLastError();
            return A2SGD_ERR_CUDA;
        }
        s.scratch = static_cast<unsigned char *>(ptr);
        s.sm_count = sms;
        s.ready = true;
    }
    *out = &s;
    return A2SGD_OK;
}

inline bool aligned_to(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

inline int width_of(const void *p, int64_t stride, uint32_t P)
{
    if (aligned_to(p, 32) && (P == 1 || stride % 8 == 0)) return 8;
    if (aligned_to(p, 16) && (P == 1 || stride % 4 == 0)) return 4;
    return 0;
}

const void *pick_kernel(bool ef, int vw)
{
    if (ef) {
        return vw == 8 ? (const void *)k_encode_vec<true, false, 8>
                       : vw == 4 ? (const void *)k_encode_vec<true, false, 4>
                                 : (const void *)k_encode_scalar<true, false>;
    }
    return vw == 8 ? (const void *)k_encode_vec<false, false, 8>
                   : vw == 4 ? (const void *)k_encode_vec<false, false, 4>
                             : (const void *)k_encode_scalar<false, false>;
}

} // namespace

extern "C" int a2sgd_encode_noalloc(uint64_t n, uint32_t P, uint32_t mode, const float *grad,
                                    int64_t grad_stride, const float *err, int64_t err_stride,
                                    float *local_means, uint64_t *pos_counts, void *stream)
{
    if (mode != A2SGD_MODE_EF && mode != A2SGD_MODE_ALG1) return A2SGD_ERR_ARG;
    const bool ef = mode == A2SGD_MODE_EF;
    if (n == 0 || n >= (1ull << 40) || P == 0 || !grad || !local_means || (ef && !err)) return A2SGD_ERR_ARG;
    if (P > kNoAllocMaxP) return A2SGD_ERR_TOO_LARGE; // the static scratch has room for this many workers only
    if (P > 1 && (grad_stride < 0 || (uint64_t)grad_stride < n)) return A2SGD_ERR_ARG;
    if (ef && P > 1 && (err_stride < 0 || (uint64_t)err_stride < n)) return A2SGD_ERR_ARG;
    if (!aligned_to(grad, 4) || (ef && !aligned_to(err, 4)) || !aligned_to(local_means, 4) ||
        (pos_counts && !aligned_to(pos_counts, 8)))
        return A2SGD_ERR_ALIGN;

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) {
        (void)cudaGetLastError();
        return A2SGD_ERR_CUDA;
    }
    DeviceSetup *setup = nullptr;
    const int rc = setup_current_device(device, &setup);
    if (rc != A2SGD_OK) return rc;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int vw = width_of(grad, grad_stride, P);
    if (ef) vw = std::min(vw, width_of(err, err_stride, P));
    const void *fn = pick_kernel(ef, vw);
    int occ = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, fn, kBlock, 0) != cudaSuccess) {
        (void)cudaGetLastError();
        occ = 1;
    }
    const uint64_t items = vw ? (n + vw - 1) / vw : (n + kScalarU - 1) / kScalarU;
    const uint64_t slots = (uint64_t)setup->sm_count * (uint64_t)std::max(occ, 1);
    uint64_t G = std::max<uint64_t>(1, std::min<uint64_t>(slots, kNoAllocMaxCtas) / P);
    G = std::min<uint64_t>(G, std::max<uint64_t>(1, (items + kBlock - 1) / kBlock));

    EncodeArgs a{};
    a.grad = grad;
    a.grad_stride = grad_stride;
    a.err = ef ? err : nullptr;
    a.err_stride = err_stride;
    a.n = n;
    a.P = P;
    a.partials = reinterpret_cast<Partial *>(setup->scratch);
    a.tickets = reinterpret_cast<unsigned int *>(setup->scratch + kTicketsOffset);
    a.status = reinterpret_cast<int *>(setup->scratch + kStatusOffset);
    a.local_means = local_means;
    a.pos_counts = reinterpret_cast<unsigned long long *>(pos_counts);
    a.pos_mask = nullptr;
    a.global_means = nullptr;
    a.ctx_local_means = nullptr;
    a.ctx_pos_counts = nullptr;

    // The tickets must start at zero; whatever an earlier (possibly interrupted) call left is cleared.
    if (cudaMemsetAsync(setup->scratch + kTicketsOffset, 0, kStatusOffset + sizeof(int) - kTicketsOffset, s) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return A2SGD_ERR_CUDA;
    }
    void *params[] = {&a};
    if (cudaLaunchKernel(fn, dim3((unsigned)G, P), dim3(kBlock), params, 0, s) != cudaSuccess) {
        (void)cudaGetLastError();
        return A2SGD_ERR_CUDA;
    }
    return A2SGD_OK;
}
