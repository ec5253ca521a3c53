// Host side of liba2sgd: argument checks, launch geometry, kernel dispatch.
// The operations and their citations are documented in include/a2sgd.h.
#include "../../include/a2sgd.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <new>
#include <unordered_map>
#include <vector>

#include "a2sgd_kernel_table.h"
#define A2SGD_NS a2sgd
#define A2SGD_CHECKED 0
#include "a2sgd_kernels.cuh"
#include "a2sgd_segments.cuh"
#include "a2sgd_select.cuh"

using namespace a2sgd;

// The checked copy of the kernels lives in its own translation unit (a2sgd_checked.cu).
const a2sgd_kernel_table *a2sgd_checked_kernels();
cudaError_t a2sgd_checked_arm(const void *descriptor, size_t bytes, cudaStream_t stream);

// Grid shapes (measured on B200, CUDA events, c2-c5 workloads):
//  * decode: one vector per thread, as many CTAs as that takes.  A persistent grid of
//    148 x occupancy CTAs with an equal static share each ran the same kernel at 6.2 TB/s; the
//    SMs do not stream at equal speed (two dies, shared channels), so the slowest share set the
//    time.  Letting the hardware CTA scheduler hand out small CTAs reaches 6.9-7.0 TB/s.
//  * encode: per-CTA partial sums must stay few and their order fixed, so the grid stays
//    proportional to the resident-CTA count: 16 CTAs per resident slot, 32 from half a billion
//    worker-elements up (c5, us per launch at 2 / 4 / 8 / 16 / 32 / 64: 6853 / 6796 / 6772 / 6773 /
//    6685 / 6668; c4: 620 / 617 / 617 / 612 / 606 / 610; c2: 300 / 303 / 305 / 300 / 304 / 329 —
//    smaller CTAs shorten the tail of the grid, more of them lengthen the last CTA's fold of the
//    partial sums, which the small configurations feel first).  The deferred-residual encode also
//    writes v, a read/write mix, and gains the same way (c2: 626 us per step at 1, 583 at 16 and 32,
//    599 at 64).
constexpr int kWavesK1 = 16;
constexpr int kWavesK1Large = 32;
constexpr uint64_t kLargeWorkerElements = 1ull << 29;
constexpr int kWavesK1Deferred = 16;
constexpr int kWavesK3 = 1 << 20; // effectively: cover every vector with its own thread
constexpr int kMaxVecWidth = 8;   // widest access the dispatcher picks: 256-bit

struct a2sgd_ctx {
    uint64_t n = 0;
    uint32_t P = 0;
    int device = 0;
    uint32_t flags = 0;
    bool alg1 = false;
    int sm_count = 0;
    bool coop_supported = false;
    size_t l2_bytes = 0;
    // scratch (device)
    Partial *partials = nullptr;
    uint32_t g_alloc = 0; // CTAs per worker the partials array can hold
    float *local_means = nullptr;
    float *global_means = nullptr;
    unsigned long long *pos_counts = nullptr;
    unsigned int *tickets = nullptr;
    unsigned int *barrier = nullptr; // 2 words: arrival counter, generation counter
    int *status = nullptr;
    // deferred-residual representation (A2SGD_DEFERRED_RESIDUAL)
    uint32_t *sign_mask = nullptr; // [P][ceil(n/32)]
    float *prev_means = nullptr;   // [2]
    bool err_holds_v = false;      // the caller's error buffer currently holds v, not e
    const a2sgd_kernel_table *k = nullptr; // production kernels, or the checked copy (A2SGD_DEBUG_CHECKS)
    // resident CTAs per SM of every kernel instance used so far (occupancy API, cached)
    std::unordered_map<const void *, int> occ;
};

inline int encode_waves(const a2sgd_ctx *c)
{
    return c->n * (uint64_t)c->P >= kLargeWorkerElements ? kWavesK1Large : kWavesK1;
}

struct a2sgd_segments {
    a2sgd_ctx *ctx = nullptr;
    uint32_t S = 0;
    bool replicated = false;
    bool has_err = false;
    // device tables
    SegTile *tiles = nullptr;
    SegStart *starts = nullptr; // [S + 1]
    uint64_t n_tiles = 0;
    // scratch of the per-tensor-means variant, allocated by its first call
    FoldJob *fold_jobs = nullptr;              // [n_jobs], built with the plan
    uint32_t n_jobs = 0;
    Partial *tile_partials = nullptr;          // [P][n_tiles]
    Partial *job_partials = nullptr;           // [P][n_jobs]
    float *seg_local_means = nullptr;          // [S][P][2]
    unsigned long long *seg_counts = nullptr;  // [S][P]
    float *seg_global_means = nullptr;         // [S][2]
    uint64_t *numel = nullptr;
    const float **grad = nullptr;
    float **err = nullptr;
    float **w = nullptr;
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

// Widest vector access (elements) this pointer / worker stride allows: 8, 4 or 0 (scalar).
inline int vec_width(const void *p, int64_t stride, uint32_t P)
{
    if (p == nullptr) return 8;
    if (kMaxVecWidth >= 8 && aligned(p, 32) && (P == 1 || stride % 8 == 0)) return 8;
    if (aligned(p, 16) && (P == 1 || stride % 4 == 0)) return 4;
    return 0;
}

// Launch with programmatic stream serialisation (see pdl_wait_prior_grid in the kernels).
cudaError_t launch_pdl(const void *fn, dim3 grid, void **params, cudaStream_t s)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kBlock);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelExC(&cfg, fn, params);
}

int occupancy(a2sgd_ctx *c, const void *kernel)
{
    auto it = c->occ.find(kernel);
    if (it != c->occ.end()) return it->second;
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kBlock, 0) != cudaSuccess) {
        (void)cudaGetLastError();
        occ = 1;
    }
    occ = std::max(occ, 1);
    c->occ[kernel] = occ;
    return occ;
}

// CTAs per worker for a (G, P) grid that fills the device exactly once.
inline uint32_t per_worker_grid(const a2sgd_ctx *c, int occ, uint64_t items, int waves = 1)
{
    const uint64_t slots = (uint64_t)c->sm_count * (uint64_t)std::max(occ, 1) * (uint64_t)waves;
    uint64_t G = std::max<uint64_t>(1, slots / c->P);
    const uint64_t need = std::max<uint64_t>(1, (items + kBlock - 1) / kBlock);
    G = std::min(G, need);
    return (uint32_t)std::min<uint64_t>(G, 0x7fffffffu);
}

inline uint32_t flat_grid(const a2sgd_ctx *c, int occ, uint64_t items, int waves = 1)
{
    const uint64_t slots = (uint64_t)c->sm_count * (uint64_t)std::max(occ, 1) * (uint64_t)waves;
    const uint64_t need = std::max<uint64_t>(1, (items + kBlock - 1) / kBlock);
    return (uint32_t)std::min<uint64_t>(std::min(slots, need), 0x7fffffffu);
}

// a 16-bit row allows 8-element vectors when it is 16-byte aligned with a stride multiple of 8
inline int vec_width_bf16(const void *p, int64_t stride, uint32_t P)
{
    return (aligned(p, 16) && (P == 1 || stride % 8 == 0)) ? 8 : 0;
}


// ---------------------------------------------------------------- launches
EncodeArgs make_encode_args(a2sgd_ctx *c, const float *grad, int64_t gs, const float *err, int64_t es,
                            float *local_means, unsigned long long *pos_counts, uint32_t *pos_mask,
                            float *global_means)
{
    EncodeArgs a{};
    a.grad = grad;
    a.grad_stride = gs;
    a.err = c->alg1 ? nullptr : err;
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
    return a;
}

DecodeArgs make_decode_args(a2sgd_ctx *c, float *w, int64_t ws, const float *grad, int64_t gs, float *err,
                            int64_t es, const float *local_means, const float *global_means, float lr)
{
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
    return a;
}

int encode_vec_width(const a2sgd_ctx *c, const float *grad, int64_t gs, const float *err, int64_t es)
{
    int vw = vec_width(grad, gs, c->P);
    if (!c->alg1) vw = std::min(vw, vec_width(err, es, c->P));
    return vw;
}

int decode_vec_width(const a2sgd_ctx *c, const float *w, int64_t ws, const float *grad, int64_t gs,
                     const float *err, int64_t es)
{
    int vw = std::min(vec_width(grad, gs, c->P), vec_width(err, es, c->P));
    return std::min(vw, vec_width(w, ws == 0 ? 8 : ws, c->P));
}

int launch_encode(a2sgd_ctx *c, const float *grad, int64_t gs, const float *err, int64_t es,
                  float *local_means, unsigned long long *pos_counts, uint32_t *pos_mask,
                  float *global_means, cudaStream_t s)
{
    const int vw = encode_vec_width(c, grad, gs, err, es);
    EncodeArgs a = make_encode_args(c, grad, gs, err, es, local_means, pos_counts, pos_mask, global_means);
    const void *fn = c->k->encode(!c->alg1, pos_mask != nullptr, vw);
    const uint64_t items = vw ? (c->n + vw - 1) / vw : (c->n + kScalarU - 1) / kScalarU;
    const dim3 grid(std::min(per_worker_grid(c, occupancy(c, fn), items, encode_waves(c)), c->g_alloc), c->P);
    void *params[] = {&a};
    A2_CUDA(launch_pdl(fn, grid, params, s));
    return A2SGD_OK;
}

// Momentum / weight-decay form of the update: the buffer (layout of w) and the two coefficients.
struct MomentumArgs {
    float *mom = nullptr;
    int64_t mom_stride = 0;
    float beta = 0.f;
    float weight_decay = 0.f;
};

int launch_decode(a2sgd_ctx *c, float *w, int64_t ws, const float *grad, int64_t gs, float *err,
                  int64_t es, const float *local_means, const float *global_means, float lr,
                  cudaStream_t s, const MomentumArgs *mo = nullptr)
{
    const bool ef = !c->alg1;
    const bool store = ef || err != nullptr;
    const bool shared = ws == 0;
    const bool mom = mo != nullptr;
    int vw = decode_vec_width(c, w, ws, grad, gs, err, es);
    if (mom) vw = std::min(vw, vec_width(mo->mom, ws == 0 ? 8 : mo->mom_stride, c->P));
    DecodeArgs a = make_decode_args(c, w, ws, grad, gs, err, es, local_means, global_means, lr);
    if (mom) {
        a.mom = mo->mom;
        a.mom_stride = shared ? 0 : mo->mom_stride;
        a.beta = mo->beta;
        a.weight_decay = mo->weight_decay;
    }
    void *params[] = {&a};
    const void *fn;
    dim3 grid;
    if (vw && shared) {
        fn = c->k->decode_shared(ef, store, c->P, vw, mom);
        grid = dim3(flat_grid(c, occupancy(c, fn), (c->n + vw - 1) / vw, kWavesK3));
    } else if (vw) {
        fn = c->k->decode_repl(ef, store, vw, mom);
        grid = dim3(per_worker_grid(c, occupancy(c, fn), (c->n + vw - 1) / vw, kWavesK3), c->P);
    } else {
        fn = c->k->decode_scalar(ef, store, mom);
        const uint64_t items = (c->n + kDecScalarU - 1) / kDecScalarU; // one tile of kBlock * kDecScalarU per CTA
        grid = shared ? dim3(flat_grid(c, occupancy(c, fn), items, kWavesK3), 1)
                      : dim3(per_worker_grid(c, occupancy(c, fn), items, kWavesK3), c->P);
    }
    A2_CUDA(launch_pdl(fn, grid, params, s));
    return A2SGD_OK;
}

// The single-launch path.  Register-resident form: at most kCoopVecPerThread 128-bit vectors of v
// per thread.  L2-resident form: g, e and w together within 70 % of the L2 capacity.
// Returns the kernel and its grid, or nullptr when (n, P, alignment) does not qualify.
//
// Which sizes take it by default is decided by measurement (B200, CUDA graphs of 50 steps, us per
// step, single launch vs two launches).  With one CTA per SM (v of all workers fits the registers of
// 148 CTAs: n * P <= 1.2 M elements) the single launch wins for every worker count: P = 1, 1 M: 8.7 vs
// 10.8; P = 2, 0.6 M: 9.2 vs 10.4; P = 4, 0.3 M: 9.9 vs 10.9; P = 8, 0.15 M: 9.9 vs 12.4.  Needing
// two or three CTAs per SM it still wins for one worker (1.5 M: 10.5 vs 10.8; 2 M: 11.5 vs 13.9) but
// not in general for several (P = 4, 0.5 M: 14.2 vs 12.4; P = 2, 0.8 M: 12.3 vs 10.9): the arrivals
// at the grid barrier double or triple, and the two-launch path hands its decode work to the
// hardware CTA scheduler, which balances the SMs better than equal static shares.  So: automatic
// for the register form when one CTA per SM is enough or P = 1; everything else that fits
// (including the L2-resident form: 1 M x 4: 17.1 vs 15.8) is available through A2SGD_FORCE_COOPERATIVE.
const void *coop_plan(a2sgd_ctx *c, bool store, bool shared, int vw, uint32_t *grid_out)
{
    if (!c->coop_supported || vw < 4) return nullptr;
    const bool forced = (c->flags & A2SGD_FORCE_COOPERATIVE) != 0;
    const void *fn = c->k->coop(!c->alg1, store, shared, c->P);
    if (!fn) return nullptr;
    const uint64_t n4 = (c->n + 3) / 4;
    const uint64_t need = std::max<uint64_t>(1, (n4 + kBlock - 1) / kBlock);
    // The smallest co-resident grid whose registers hold v: one CTA per SM where that is enough (half
    // the arrivals at the grid barrier: c1 9.6 -> 8.7 us per step), full occupancy otherwise.
    for (const int ctas_per_sm : {1, occupancy(c, fn)}) {
        const uint64_t resident = (uint64_t)c->sm_count * ctas_per_sm;
        const uint64_t per_thread = kCoopVecPerThread / c->P;
        const uint64_t grid = std::min<uint64_t>(resident, need);
        if (n4 <= resident * kBlock * per_thread && grid <= c->g_alloc) {
            if (!forced && ctas_per_sm != 1 && c->P != 1) return nullptr; // measured slower than two launches
            *grid_out = (uint32_t)grid;
            return fn;
        }
    }
    if (!forced) return nullptr;
    const void *fn2 = c->k->coop_l2(!c->alg1, store, shared, c->P);
    const uint64_t rows = (uint64_t)c->P * (c->alg1 ? (store ? 2 : 1) : 2) + (shared ? 1 : c->P);
    const double footprint = (double)rows * (double)c->n * 4.0;
    if (!fn2 || footprint > 0.70 * (double)c->l2_bytes) return nullptr;
    const uint64_t grid = std::min<uint64_t>(std::min<uint64_t>((uint64_t)c->sm_count * occupancy(c, fn2), need), c->g_alloc);
    *grid_out = (uint32_t)grid;
    return fn2;
}

int launch_coop(a2sgd_ctx *c, const void *fn, uint32_t grid, float *w, int64_t ws, const float *grad, int64_t gs,
                float *err, int64_t es, float lr, cudaStream_t s)
{
    CoopArgs a{};
    a.enc = make_encode_args(c, grad, gs, err, es, c->local_means, c->pos_counts, nullptr, c->global_means);
    a.dec = make_decode_args(c, w, ws, grad, gs, err, es, c->local_means, c->global_means, lr);
    a.barrier = c->barrier;
    const bool never_opens = (c->flags & A2SGD_TEST_BARRIER_NEVER_OPENS) != 0;
    a.expected = never_opens ? grid + 1 : grid;
    a.spin_limit = never_opens ? (1u << 12) : (1u << 24); // x 40 ns sleep: ~0.2 ms / ~1 s
    void *params[] = {&a};
    // cooperative (all CTAs co-resident: the grid barrier needs it) and, like the other kernels,
    // with programmatic stream serialisation: the CTAs of the next step may become resident while
    // this grid drains; they wait for it before their first memory access, ahead of the barrier
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kBlock);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    A2_CUDA(cudaLaunchKernelExC(&cfg, fn, params));
    return A2SGD_OK;
}

// One step in the deferred-residual representation (see k_encode_vec / k_decode_deferred).
int deferred_step(a2sgd_ctx *c, float *w, int64_t ws, const float *grad, int64_t gs, float *err, int64_t es,
                  float lr, cudaStream_t s)
{
    // this form has 256-bit kernels only
    if (vec_width(grad, gs, c->P) < 8 || vec_width(err, es, c->P) < 8 || vec_width(w, ws == 0 ? 8 : ws, c->P) < 8)
        return A2SGD_ERR_ALIGN;
    {
        EncodeArgs a = make_encode_args(c, grad, gs, err, es, c->local_means, c->pos_counts, c->sign_mask,
                                        c->global_means);
        a.prev_means = c->prev_means;
        const void *fn = c->k->encode_deferred(c->err_holds_v);
        const dim3 grid(std::min(per_worker_grid(c, occupancy(c, fn), (c->n + 7) / 8, kWavesK1Deferred), c->g_alloc), c->P);
        void *params[] = {&a};
        A2_CUDA(launch_pdl(fn, grid, params, s));
    }
    {
        DeferredDecodeArgs a{};
        a.w = w;
        a.w_stride = ws;
        a.v = err;
        a.v_stride = es;
        a.mask = c->sign_mask;
        a.n = c->n;
        a.P = c->P;
        a.global_means = c->global_means;
        a.prev_means = c->prev_means;
        a.lr = lr;
        const void *fn = c->k->decode_deferred(ws != 0, c->P);
        const dim3 grid(flat_grid(c, occupancy(c, fn), std::max<uint64_t>(1, (c->n / 32) * 4), kWavesK3));
        void *params[] = {&a};
        A2_CUDA(launch_pdl(fn, grid, params, s));
    }
    c->err_holds_v = true;
    return A2SGD_OK;
}

// A2SGD_CHECK_POINTERS: is this address device (or managed) memory that the context's device can use?
bool device_pointer_ok(const a2sgd_ctx *c, const void *p)
{
    if (!(c->flags & A2SGD_CHECK_POINTERS) || p == nullptr) return true;
    cudaPointerAttributes attr{};
    if (cudaPointerGetAttributes(&attr, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return false;
    }
    if (attr.type == cudaMemoryTypeManaged) return true;
    return attr.type == cudaMemoryTypeDevice && attr.device == c->device;
}

// A2SGD_DEBUG_CHECKS: for the duration of one call's launches the device-side descriptor of the
// checked kernels holds the extents of the call's buffers; the destructor switches it off again
// (stream-ordered after the kernels).  Buffers are added as `rows` rows of `n` elements of `elem`
// bytes, `stride` elements apart.
struct DebugScope {
    a2sgd_ctx *c;
    cudaStream_t s;
    DebugChecks d{};
    bool armed = false;
    DebugScope(a2sgd_ctx *ctx, cudaStream_t stream) : c(ctx), s(stream) {}
    void add(const void *base, uint64_t rows, int64_t stride, uint64_t n, uint32_t elem)
    {
        if (!(c->flags & A2SGD_DEBUG_CHECKS) || !base || d.count >= kDebugMaxRanges) return;
        DebugRange &r = d.range[d.count++];
        r.base = (uint64_t)reinterpret_cast<uintptr_t>(base);
        r.rows = rows;
        r.stride_bytes = rows > 1 ? (uint64_t)stride * elem : 0;
        r.row_bytes = n * elem;
        if ((c->flags & A2SGD_TEST_SHRINK_EXTENTS) && n > 1) r.row_bytes -= elem;
    }
    // mode 1: the address ranges added so far; mode 2: index checks only (segment lists)
    bool arm(int mode)
    {
        if (!(c->flags & A2SGD_DEBUG_CHECKS)) return true;
        // the descriptor is copied from this (stack) object: a captured copy would read it again at
        // every replay, long after it is gone — checking contexts are refused during stream capture
        cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(s, &capturing) != cudaSuccess || capturing != cudaStreamCaptureStatusNone) {
            (void)cudaGetLastError();
            return false;
        }
        d.on = mode;
        d.status = c->status;
        armed = a2sgd_checked_arm(&d, sizeof(d), s) == cudaSuccess;
        if (!armed) (void)cudaGetLastError();
        return armed;
    }
    ~DebugScope()
    {
        if (!armed) return;
        const DebugChecks off{};
        if (a2sgd_checked_arm(&off, sizeof(off), s) != cudaSuccess) (void)cudaGetLastError();
    }
};

int check_common(const a2sgd_ctx *c, const float *grad, int64_t gs, const float *err, int64_t es,
                 bool err_required)
{
    if (!c || !grad) return A2SGD_ERR_ARG;
    if (!device_pointer_ok(c, grad) || !device_pointer_ok(c, err)) return A2SGD_ERR_ARG;
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
    const uint32_t known = A2SGD_MODE_ALG1 | A2SGD_FORCE_TWO_PASS | A2SGD_FORCE_COOPERATIVE |
                           A2SGD_TEST_BARRIER_NEVER_OPENS | A2SGD_DEFERRED_RESIDUAL | A2SGD_CHECK_POINTERS |
                           A2SGD_DEBUG_CHECKS | A2SGD_TEST_SHRINK_EXTENTS;
    if ((flags & A2SGD_DEFERRED_RESIDUAL) && (flags & (A2SGD_MODE_ALG1 | A2SGD_FORCE_COOPERATIVE))) return A2SGD_ERR_ARG;
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
    static const a2sgd_kernel_table production = a2sgd::kernel_table();
    c->k = (flags & A2SGD_DEBUG_CHECKS) ? a2sgd_checked_kernels() : &production;
    if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
        delete c;
        return A2SGD_ERR_CUDA;
    }
    {
        int coop = 0;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, device) != cudaSuccess) (void)cudaGetLastError();
        c->coop_supported = coop != 0;
        int l2 = 0;
        if (cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, device) != cudaSuccess) (void)cudaGetLastError();
        c->l2_bytes = (size_t)std::max(l2, 0);
    }
    // partials: room for a (G, P) grid that fills the device at the highest possible occupancy
    const uint32_t max_slots = (uint32_t)c->sm_count * (2048 / kBlock) * std::max(kWavesK1Large, kWavesK1Deferred);
    c->g_alloc = std::max<uint32_t>(1, max_slots / P);
    bool ok = true;
    ok = ok && cudaMalloc(&c->partials, sizeof(Partial) * (size_t)c->g_alloc * P) == cudaSuccess;
    ok = ok && cudaMalloc(&c->local_means, sizeof(float) * 2 * P) == cudaSuccess;
    ok = ok && cudaMalloc(&c->global_means, sizeof(float) * 2) == cudaSuccess;
    ok = ok && cudaMalloc(&c->pos_counts, sizeof(unsigned long long) * P) == cudaSuccess;
    ok = ok && cudaMalloc(&c->tickets, sizeof(unsigned int) * (P + 1)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->status, sizeof(int)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->barrier, sizeof(unsigned int) * 2) == cudaSuccess;
    if (flags & A2SGD_DEFERRED_RESIDUAL) {
        ok = ok && cudaMalloc(&c->sign_mask, sizeof(uint32_t) * (size_t)P * ((n + 31) / 32)) == cudaSuccess;
        ok = ok && cudaMalloc(&c->prev_means, sizeof(float) * 2) == cudaSuccess;
        ok = ok && cudaMemset(c->prev_means, 0, sizeof(float) * 2) == cudaSuccess;
    }
    ok = ok && cudaMemset(c->barrier, 0, sizeof(unsigned int) * 2) == cudaSuccess;
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
    cudaFree(c->barrier);
    cudaFree(c->sign_mask);
    cudaFree(c->prev_means);
    (void)cudaGetLastError();
    delete c;
    return A2SGD_OK;
}

extern "C" int a2sgd_encode(a2sgd_ctx *c, const float *grad, int64_t grad_stride, const float *err,
                            int64_t err_stride, float *local_means, uint64_t *pos_counts,
                            uint32_t *pos_mask, void *stream)
{
    if (!c || !local_means) return A2SGD_ERR_ARG;
    if (c->flags & A2SGD_DEFERRED_RESIDUAL) return A2SGD_ERR_ARG; // the error buffer may not hold a residual
    const int rc = check_common(c, grad, grad_stride, err, err_stride, !c->alg1);
    if (rc) return rc;
    if (!aligned(local_means, 4) || (pos_counts && !aligned(pos_counts, 8)) || (pos_mask && !aligned(pos_mask, 4)))
        return A2SGD_ERR_ALIGN;
    if (!device_pointer_ok(c, local_means) || !device_pointer_ok(c, pos_counts) || !device_pointer_ok(c, pos_mask))
        return A2SGD_ERR_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    DebugScope dbg(c, static_cast<cudaStream_t>(stream));
    dbg.add(grad, c->P, grad_stride, c->n, 4);
    if (!c->alg1) dbg.add(err, c->P, err_stride, c->n, 4);
    dbg.add(pos_mask, c->P, (int64_t)((c->n + 31) / 32), (c->n + 31) / 32, 4);
    if (!dbg.arm(1)) return A2SGD_ERR_CUDA;
    return launch_encode(c, grad, grad_stride, err, err_stride, local_means,
                         reinterpret_cast<unsigned long long *>(pos_counts), pos_mask, nullptr,
                         static_cast<cudaStream_t>(stream));
}

extern "C" int a2sgd_global_average(a2sgd_ctx *c, const float *local_means, float *global_means, void *stream)
{
    if (!c || !local_means || !global_means) return A2SGD_ERR_ARG;
    if (!aligned(local_means, 4) || !aligned(global_means, 4)) return A2SGD_ERR_ALIGN;
    if (!device_pointer_ok(c, local_means) || !device_pointer_ok(c, global_means)) return A2SGD_ERR_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    {
        uint32_t P = c->P;
        float *ctx_copy = c->global_means;
        void *params[] = {&local_means, &P, &global_means, &ctx_copy};
        A2_CUDA(cudaLaunchKernel(c->k->global_average, dim3(1), dim3(32), params, 0, static_cast<cudaStream_t>(stream)));
    }
    return A2SGD_OK;
}

extern "C" int a2sgd_global_average_from_sums(a2sgd_ctx *c, const double *sums, uint32_t workers,
                                              float *global_means, void *stream)
{
    if (!c || !sums || !global_means || workers == 0) return A2SGD_ERR_ARG;
    if (!aligned(sums, 8) || !aligned(global_means, 4)) return A2SGD_ERR_ALIGN;
    if (!device_pointer_ok(c, sums) || !device_pointer_ok(c, global_means)) return A2SGD_ERR_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    {
        float *ctx_copy = c->global_means;
        void *params[] = {&sums, &workers, &global_means, &ctx_copy};
        A2_CUDA(cudaLaunchKernel(c->k->global_average_from_sums, dim3(1), dim3(32), params, 0,
                                 static_cast<cudaStream_t>(stream)));
    }
    return A2SGD_OK;
}

extern "C" int a2sgd_decode_update(a2sgd_ctx *c, float *w, int64_t w_stride, const float *grad,
                                   int64_t grad_stride, float *err, int64_t err_stride,
                                   const float *local_means, const float *global_means, float lr,
                                   void *stream)
{
    if (!c || !w || !global_means) return A2SGD_ERR_ARG;
    if (c->flags & A2SGD_DEFERRED_RESIDUAL) return A2SGD_ERR_ARG;
    const int rc = check_common(c, grad, grad_stride, err, err_stride, !c->alg1);
    if (rc) return rc;
    if (c->alg1 && !local_means) return A2SGD_ERR_ARG;
    if (w_stride != 0 && !stride_ok(w_stride, c->n, c->P)) return A2SGD_ERR_ARG;
    if (!aligned(w, 4) || !aligned(global_means, 4) || (local_means && !aligned(local_means, 4)))
        return A2SGD_ERR_ALIGN;
    if (!device_pointer_ok(c, w) || !device_pointer_ok(c, global_means) || !device_pointer_ok(c, local_means))
        return A2SGD_ERR_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    DebugScope dbg(c, static_cast<cudaStream_t>(stream));
    dbg.add(grad, c->P, grad_stride, c->n, 4);
    dbg.add(err, c->P, err_stride, c->n, 4);
    dbg.add(w, (w_stride == 0 || c->P == 1) ? 1 : c->P, w_stride, c->n, 4);
    if (!dbg.arm(1)) return A2SGD_ERR_CUDA;
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
    if (!device_pointer_ok(c, w)) return A2SGD_ERR_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int64_t ws = (c->P == 1) ? 0 : w_stride;
    DebugScope dbg(c, s);
    dbg.add(grad, c->P, grad_stride, c->n, 4);
    dbg.add(err, c->P, err_stride, c->n, 4);
    dbg.add(w, ws == 0 ? 1 : c->P, ws, c->n, 4);
    dbg.add(c->sign_mask, c->P, (int64_t)((c->n + 31) / 32), (c->n + 31) / 32, 4);
    if (!dbg.arm(1)) return A2SGD_ERR_CUDA;
    if (c->flags & A2SGD_DEFERRED_RESIDUAL) return deferred_step(c, w, ws, grad, grad_stride, err, err_stride, lr, s);
    if (!(c->flags & A2SGD_FORCE_TWO_PASS)) {
        const bool store = !c->alg1 || err != nullptr;
        const int vw = decode_vec_width(c, w, ws, grad, grad_stride, err, err_stride);
        uint32_t grid = 0;
        const void *fn = coop_plan(c, store, ws == 0, vw, &grid);
        if (fn) return launch_coop(c, fn, grid, w, ws, grad, grad_stride, err, err_stride, lr, s);
        if (c->flags & A2SGD_FORCE_COOPERATIVE) return A2SGD_ERR_TOO_LARGE;
    }
    const int r1 = launch_encode(c, grad, grad_stride, err, err_stride, c->local_means, c->pos_counts, nullptr,
                                 c->global_means, s);
    if (r1) return r1;
    return launch_decode(c, w, ws, grad, grad_stride, err, err_stride, c->local_means, c->global_means, lr, s);
}

// Argument checks shared by the two momentum entry points.
static int check_momentum(const a2sgd_ctx *c, const float *w, int64_t w_stride, const float *mom, int64_t mom_stride,
                          float beta, float weight_decay)
{
    if (!w || !mom) return A2SGD_ERR_ARG;
    if (c->flags & A2SGD_DEFERRED_RESIDUAL) return A2SGD_ERR_ARG;
    if (w_stride != 0 && !stride_ok(w_stride, c->n, c->P)) return A2SGD_ERR_ARG;
    if (c->P > 1 && (w_stride == 0) != (mom_stride == 0)) return A2SGD_ERR_ARG; // same layout as w
    if (mom_stride != 0 && !stride_ok(mom_stride, c->n, c->P)) return A2SGD_ERR_ARG;
    if (!(beta >= 0.0f && beta < 1.0f) || !(weight_decay >= 0.0f)) return A2SGD_ERR_ARG;
    if (!aligned(w, 4) || !aligned(mom, 4)) return A2SGD_ERR_ALIGN;
    if (!device_pointer_ok(c, w) || !device_pointer_ok(c, mom)) return A2SGD_ERR_ARG;
    return A2SGD_OK;
}

extern "C" int a2sgd_decode_update_momentum(a2sgd_ctx *c, float *w, int64_t w_stride, float *mom, int64_t mom_stride,
                                            const float *grad, int64_t grad_stride, float *err, int64_t err_stride,
                                            const float *local_means, const float *global_means, float lr,
                                            float beta, float weight_decay, void *stream)
{
    if (!c || !global_means) return A2SGD_ERR_ARG;
    int rc = check_common(c, grad, grad_stride, err, err_stride, !c->alg1);
    if (rc) return rc;
    rc = check_momentum(c, w, w_stride, mom, mom_stride, beta, weight_decay);
    if (rc) return rc;
    if (c->alg1 && !local_means) return A2SGD_ERR_ARG;
    if (!aligned(global_means, 4) || (local_means && !aligned(local_means, 4))) return A2SGD_ERR_ALIGN;
    if (!device_pointer_ok(c, global_means) || !device_pointer_ok(c, local_means)) return A2SGD_ERR_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    MomentumArgs mo;
    mo.mom = mom;
    mo.mom_stride = mom_stride;
    mo.beta = beta;
    mo.weight_decay = weight_decay;
    DebugScope dbg(c, static_cast<cudaStream_t>(stream));
    dbg.add(grad, c->P, grad_stride, c->n, 4);
    dbg.add(err, c->P, err_stride, c->n, 4);
    dbg.add(w, (w_stride == 0 || c->P == 1) ? 1 : c->P, w_stride, c->n, 4);
    dbg.add(mom, (w_stride == 0 || c->P == 1) ? 1 : c->P, mom_stride, c->n, 4);
    if (!dbg.arm(1)) return A2SGD_ERR_CUDA;
    return launch_decode(c, w, (c->P == 1) ? 0 : w_stride, grad, grad_stride, err, err_stride, local_means,
                         global_means, lr, static_cast<cudaStream_t>(stream), &mo);
}

extern "C" int a2sgd_step_momentum(a2sgd_ctx *c, float *w, int64_t w_stride, float *mom, int64_t mom_stride,
                                   const float *grad, int64_t grad_stride, float *err, int64_t err_stride,
                                   float lr, float beta, float weight_decay, void *stream)
{
    if (!c) return A2SGD_ERR_ARG;
    int rc = check_common(c, grad, grad_stride, err, err_stride, !c->alg1);
    if (rc) return rc;
    rc = check_momentum(c, w, w_stride, mom, mom_stride, beta, weight_decay);
    if (rc) return rc;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    MomentumArgs mo;
    mo.mom = mom;
    mo.mom_stride = mom_stride;
    mo.beta = beta;
    mo.weight_decay = weight_decay;
    DebugScope dbg(c, s);
    dbg.add(grad, c->P, grad_stride, c->n, 4);
    dbg.add(err, c->P, err_stride, c->n, 4);
    dbg.add(w, (w_stride == 0 || c->P == 1) ? 1 : c->P, w_stride, c->n, 4);
    dbg.add(mom, (w_stride == 0 || c->P == 1) ? 1 : c->P, mom_stride, c->n, 4);
    if (!dbg.arm(1)) return A2SGD_ERR_CUDA;
    const int r1 = launch_encode(c, grad, grad_stride, err, err_stride, c->local_means, c->pos_counts, nullptr,
                                 c->global_means, s);
    if (r1) return r1;
    return launch_decode(c, w, (c->P == 1) ? 0 : w_stride, grad, grad_stride, err, err_stride, c->local_means,
                         c->global_means, lr, s, &mo);
}

static int step_lowp(a2sgd_ctx *c, float *w, int64_t w_stride, const uint16_t *grad, int64_t grad_stride,
                     float *err, int64_t err_stride, float lr, void *stream, int gt);

extern "C" int a2sgd_step_bf16(a2sgd_ctx *c, float *w, int64_t w_stride, const uint16_t *grad, int64_t grad_stride,
                               float *err, int64_t err_stride, float lr, void *stream)
{
    return step_lowp(c, w, w_stride, grad, grad_stride, err, err_stride, lr, stream, 1);
}

extern "C" int a2sgd_step_f16(a2sgd_ctx *c, float *w, int64_t w_stride, const uint16_t *grad, int64_t grad_stride,
                              float *err, int64_t err_stride, float lr, void *stream)
{
    return step_lowp(c, w, w_stride, grad, grad_stride, err, err_stride, lr, stream, 2);
}

static int step_lowp(a2sgd_ctx *c, float *w, int64_t w_stride, const uint16_t *grad, int64_t grad_stride,
                     float *err, int64_t err_stride, float lr, void *stream, int gt)
{
    if (!c || !w || !grad) return A2SGD_ERR_ARG;
    if (!c->alg1 && !err) return A2SGD_ERR_ARG;
    if (c->flags & A2SGD_DEFERRED_RESIDUAL) return A2SGD_ERR_ARG;
    if (!stride_ok(grad_stride, c->n, c->P) || (err && !stride_ok(err_stride, c->n, c->P))) return A2SGD_ERR_ARG;
    if (w_stride != 0 && !stride_ok(w_stride, c->n, c->P)) return A2SGD_ERR_ARG;
    if (!aligned(grad, 2) || (err && !aligned(err, 4)) || !aligned(w, 4)) return A2SGD_ERR_ALIGN;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool ef = !c->alg1;
    const bool store = ef || err != nullptr;
    const int64_t ws = (c->P == 1) ? 0 : w_stride;
    const float *g = reinterpret_cast<const float *>(grad); // element type is carried by the kernel template
    if (!device_pointer_ok(c, grad) || !device_pointer_ok(c, err) || !device_pointer_ok(c, w)) return A2SGD_ERR_ARG;
    DebugScope dbg(c, s);
    dbg.add(grad, c->P, grad_stride, c->n, 2);
    dbg.add(err, c->P, err_stride, c->n, 4);
    dbg.add(w, ws == 0 ? 1 : c->P, ws, c->n, 4);
    if (!dbg.arm(1)) return A2SGD_ERR_CUDA;
    int vw_enc = vec_width_bf16(grad, grad_stride, c->P);
    if (ef && vec_width(err, err_stride, c->P) < 8) vw_enc = 0;
    int vw_dec = vw_enc;
    if (vec_width(err, err_stride, c->P) < 8 || vec_width(w, ws == 0 ? 8 : ws, c->P) < 8) vw_dec = 0;
    {
        EncodeArgs a = make_encode_args(c, g, grad_stride, err, err_stride, c->local_means, c->pos_counts, nullptr,
                                        c->global_means);
        const void *fn = c->k->encode_lowp(gt, ef, vw_enc);
        const uint64_t items = vw_enc ? (c->n + 7) / 8 : (c->n + kScalarU - 1) / kScalarU;
        const dim3 grid(std::min(per_worker_grid(c, occupancy(c, fn), items, encode_waves(c)), c->g_alloc), c->P);
        void *params[] = {&a};
        A2_CUDA(launch_pdl(fn, grid, params, s));
    }
    {
        DecodeArgs a = make_decode_args(c, w, ws, g, grad_stride, err, err_stride, c->local_means, c->global_means, lr);
        const void *fn = c->k->decode_lowp(gt, ef, store, ws == 0, c->P, vw_dec);
        const uint64_t items = vw_dec ? (c->n + 7) / 8 : (c->n + kDecScalarU - 1) / kDecScalarU;
        const dim3 grid = (ws == 0) ? dim3(flat_grid(c, occupancy(c, fn), items, kWavesK3))
                                    : dim3(per_worker_grid(c, occupancy(c, fn), items, kWavesK3), c->P);
        void *params[] = {&a};
        A2_CUDA(launch_pdl(fn, grid, params, s));
    }
    return A2SGD_OK;
}

extern "C" int a2sgd_materialize_err(a2sgd_ctx *c, float *err, int64_t err_stride, void *stream)
{
    if (!c || !err) return A2SGD_ERR_ARG;
    if (!(c->flags & A2SGD_DEFERRED_RESIDUAL)) return A2SGD_ERR_ARG;
    if (!stride_ok(err_stride, c->n, c->P)) return A2SGD_ERR_ARG;
    if (vec_width(err, err_stride, c->P) < 8) return A2SGD_ERR_ALIGN;
    if (!c->err_holds_v) return A2SGD_OK; // already a true residual
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    if (!device_pointer_ok(c, err)) return A2SGD_ERR_ARG;
    DebugScope dbg(c, static_cast<cudaStream_t>(stream));
    dbg.add(err, c->P, err_stride, c->n, 4);
    if (!dbg.arm(1)) return A2SGD_ERR_CUDA;
    const uint64_t need = std::max<uint64_t>(1, (c->n / 8 + kBlock - 1) / kBlock);
    const dim3 grid((unsigned)std::min<uint64_t>(need, 0x7fffffffu), c->P);
    {
        uint64_t n = c->n;
        const float *means = c->global_means;
        void *params[] = {&err, &err_stride, &n, &means};
        A2_CUDA(cudaLaunchKernel(c->k->materialize_err, grid, dim3(kBlock), params, 0, static_cast<cudaStream_t>(stream)));
    }
    c->err_holds_v = false;
    return A2SGD_OK;
}

static int dense_sync_impl(a2sgd_ctx *c, float *w, int64_t w_stride, const float *grad, int64_t grad_stride,
                           float lr, float divisor, void *stream);

extern "C" int a2sgd_dense_sync(a2sgd_ctx *c, float *w, int64_t w_stride, const float *grad, int64_t grad_stride,
                               float lr, void *stream)
{
    if (!c) return A2SGD_ERR_ARG;
    return dense_sync_impl(c, w, w_stride, grad, grad_stride, lr, (float)c->P, stream);
}

extern "C" int a2sgd_dense_sync_reduced(a2sgd_ctx *c, float *w, const float *grad_sum, uint32_t workers, float lr,
                                       void *stream)
{
    if (!c || c->P != 1 || workers == 0) return A2SGD_ERR_ARG;
    return dense_sync_impl(c, w, 0, grad_sum, 0, lr, (float)workers, stream);
}

static int dense_sync_impl(a2sgd_ctx *c, float *w, int64_t w_stride, const float *grad, int64_t grad_stride,
                           float lr, float divisor, void *stream)
{
    if (!c || !w || !grad) return A2SGD_ERR_ARG;
    if (!stride_ok(grad_stride, c->n, c->P)) return A2SGD_ERR_ARG;
    if (w_stride != 0 && !stride_ok(w_stride, c->n, c->P)) return A2SGD_ERR_ARG;
    if (!aligned(w, 4) || !aligned(grad, 4)) return A2SGD_ERR_ALIGN;
    if (!device_pointer_ok(c, w) || !device_pointer_ok(c, grad)) return A2SGD_ERR_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    const int64_t ws = (c->P == 1) ? 0 : w_stride;
    const int vw = std::min(vec_width(grad, grad_stride, c->P), vec_width(w, ws == 0 ? 8 : ws, c->P));
    DebugScope dbg(c, static_cast<cudaStream_t>(stream));
    dbg.add(grad, c->P, grad_stride, c->n, 4);
    dbg.add(w, ws == 0 ? 1 : c->P, ws, c->n, 4);
    if (!dbg.arm(1)) return A2SGD_ERR_CUDA;
    DenseArgs a{};
    a.w = w;
    a.w_stride = ws;
    a.grad = grad;
    a.grad_stride = grad_stride;
    a.n = c->n;
    a.P = c->P;
    a.lr = lr;
    a.divisor = divisor;
    const void *fn = c->k->dense(c->P, vw, ws != 0);
    const uint64_t items = vw ? (c->n + vw - 1) / vw : c->n;
    const dim3 grid(flat_grid(c, occupancy(c, fn), items, kWavesK3));
    void *params[] = {&a};
    A2_CUDA(launch_pdl(fn, grid, params, static_cast<cudaStream_t>(stream)));
    return A2SGD_OK;
}

// ---------------------------------------------------------------- segment lists
extern "C" int a2sgd_segments_create(a2sgd_ctx *c, uint32_t S, const uint64_t *numel, const float *const *grad,
                                     float *const *err, float *const *w, int w_replicated, a2sgd_segments **out)
{
    if (!out) return A2SGD_ERR_ARG;
    *out = nullptr;
    if (!c || S == 0 || !numel || !grad || !w) return A2SGD_ERR_ARG;
    if (c->flags & A2SGD_DEFERRED_RESIDUAL) return A2SGD_ERR_ARG;
    if (!c->alg1 && !err) return A2SGD_ERR_ARG;
    const uint32_t P = c->P;
    const bool repl = w_replicated != 0 && P > 1;
    uint64_t total = 0;
    std::vector<SegTile> tiles;
    std::vector<SegStart> starts;
    std::vector<FoldJob> jobs;
    for (uint32_t s = 0; s < S; ++s) {
        if (numel[s] == 0) return A2SGD_ERR_ARG;
        total += numel[s];
        bool vec = true;
        for (uint32_t p = 0; p < P; ++p) {
            const float *g = grad[(size_t)p * S + s];
            const float *e = err ? err[(size_t)p * S + s] : nullptr;
            if (!g || (err && !e)) return A2SGD_ERR_ARG; // an error table, when given, has no NULL entries
            if (!device_pointer_ok(c, g) || !device_pointer_ok(c, e)) return A2SGD_ERR_ARG;
            if (!aligned(g, 4) || (e && !aligned(e, 4))) return A2SGD_ERR_ALIGN;
            vec = vec && aligned(g, 32) && (!e || aligned(e, 32));
        }
        const uint32_t w_rows = repl ? P : 1;
        for (uint32_t r = 0; r < w_rows; ++r) {
            const float *wp = w[(size_t)r * S + s];
            if (!wp || !device_pointer_ok(c, wp)) return A2SGD_ERR_ARG;
            if (!aligned(wp, 4)) return A2SGD_ERR_ALIGN;
            vec = vec && aligned(wp, 32);
        }
        starts.push_back(SegStart{(uint64_t)tiles.size(), numel[s], vec ? kSegFlagVec : 0u, (uint32_t)jobs.size(), {0u, 0u}});
        const uint64_t first_tile = tiles.size();
        for (uint64_t off = 0; off < numel[s]; off += kSegTile) tiles.push_back(SegTile{s, vec ? kSegFlagVec : 0u, off});
        for (uint64_t ft = first_tile; ft < tiles.size(); ft += kFoldJobTiles)
            jobs.push_back(FoldJob{ft, (uint32_t)std::min<uint64_t>(kFoldJobTiles, tiles.size() - ft), s});
    }
    if (total != c->n) return A2SGD_ERR_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    a2sgd_segments *sg = new (std::nothrow) a2sgd_segments();
    if (!sg) return A2SGD_ERR_NOMEM;
    sg->ctx = c;
    sg->S = S;
    sg->replicated = repl;
    sg->has_err = err != nullptr;
    sg->n_tiles = tiles.size();
    const size_t w_count = (size_t)(repl ? P : 1) * S;
    bool ok = true;
    ok = ok && cudaMalloc(&sg->tiles, sizeof(SegTile) * tiles.size()) == cudaSuccess;
    ok = ok && cudaMalloc(&sg->numel, sizeof(uint64_t) * S) == cudaSuccess;
    ok = ok && cudaMalloc(&sg->grad, sizeof(float *) * (size_t)P * S) == cudaSuccess;
    ok = ok && cudaMalloc(&sg->w, sizeof(float *) * w_count) == cudaSuccess;
    if (err) ok = ok && cudaMalloc(&sg->err, sizeof(float *) * (size_t)P * S) == cudaSuccess;
    ok = ok && cudaMemcpy(sg->tiles, tiles.data(), sizeof(SegTile) * tiles.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    starts.push_back(SegStart{(uint64_t)tiles.size(), 0, 0u, (uint32_t)jobs.size(), {0u, 0u}}); // end marker
    sg->n_jobs = (uint32_t)jobs.size();
    ok = ok && cudaMalloc(&sg->starts, sizeof(SegStart) * starts.size()) == cudaSuccess;
    ok = ok && cudaMemcpy(sg->starts, starts.data(), sizeof(SegStart) * starts.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMalloc(&sg->fold_jobs, sizeof(FoldJob) * jobs.size()) == cudaSuccess;
    ok = ok && cudaMemcpy(sg->fold_jobs, jobs.data(), sizeof(FoldJob) * jobs.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(sg->numel, numel, sizeof(uint64_t) * S, cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(sg->grad, grad, sizeof(float *) * (size_t)P * S, cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(sg->w, w, sizeof(float *) * w_count, cudaMemcpyHostToDevice) == cudaSuccess;
    if (err) ok = ok && cudaMemcpy(sg->err, err, sizeof(float *) * (size_t)P * S, cudaMemcpyHostToDevice) == cudaSuccess;
    if (!ok) {
        (void)cudaGetLastError();
        a2sgd_segments_destroy(sg);
        return A2SGD_ERR_NOMEM;
    }
    *out = sg;
    return A2SGD_OK;
}

extern "C" int a2sgd_segments_destroy(a2sgd_segments *sg)
{
    if (!sg) return A2SGD_OK;
    DeviceGuard guard(sg->ctx->device);
    cudaFree(sg->tiles);
    cudaFree(sg->starts);
    cudaFree(sg->fold_jobs);
    cudaFree(sg->job_partials);
    cudaFree(sg->tile_partials);
    cudaFree(sg->seg_local_means);
    cudaFree(sg->seg_counts);
    cudaFree(sg->seg_global_means);
    cudaFree(sg->numel);
    cudaFree(sg->grad);
    cudaFree(sg->err);
    cudaFree(sg->w);
    (void)cudaGetLastError();
    delete sg;
    return A2SGD_OK;
}

static SegTables seg_tables(const a2sgd_segments *sg, const float *lr_per_segment)
{
    SegTables t{};
    t.tiles = sg->tiles;
    t.starts = sg->S <= kSegScanMax ? sg->starts : nullptr; // beyond that the decode kernel reads the tile table
    t.all_starts = sg->starts;
    t.fold_jobs = sg->fold_jobs;
    t.n_jobs = sg->n_jobs;
    t.tile_partials = sg->tile_partials;
    t.job_partials = sg->job_partials;
    t.seg_local_means = sg->seg_local_means;
    t.seg_counts = sg->seg_counts;
    t.seg_global_means = sg->seg_global_means;
    t.n_tiles = sg->n_tiles;
    t.numel = sg->numel;
    t.grad = sg->grad;
    t.err = sg->err;
    t.w = sg->w;
    t.S = sg->S;
    t.w_replicated = sg->replicated ? 1u : 0u;
    t.lr_per_segment = lr_per_segment;
    return t;
}

static int launch_encode_segments(a2sgd_ctx *c, a2sgd_segments *sg, float *local_means,
                                  unsigned long long *pos_counts, float *global_means, cudaStream_t s,
                                  bool per_tensor = false)
{
    SegTables t = seg_tables(sg, nullptr);
    EncodeArgs a = make_encode_args(c, nullptr, 0, nullptr, 0, local_means, pos_counts, nullptr, global_means);
    const void *fn = c->k->encode_segments(!c->alg1, per_tensor);
    const uint64_t slots = (uint64_t)c->sm_count * occupancy(c, fn) * kWavesK1; // 32 measured slower here (c5: 19.8 vs 19.5 ms per step)
    uint64_t G = std::max<uint64_t>(1, slots / c->P);
    G = std::min<uint64_t>(std::min<uint64_t>(G, sg->n_tiles), c->g_alloc);
    void *params[] = {&a, &t};
    A2_CUDA(launch_pdl(fn, dim3((unsigned)G, c->P), params, s));
    return A2SGD_OK;
}

static int launch_decode_segments(a2sgd_ctx *c, a2sgd_segments *sg, const float *local_means,
                                  const float *global_means, float lr, const float *lr_per_segment, cudaStream_t s,
                                  bool per_tensor = false)
{
    const bool ef = !c->alg1;
    const bool store = ef || sg->has_err;
    SegTables t = seg_tables(sg, lr_per_segment);
    DecodeArgs a = make_decode_args(c, nullptr, sg->replicated ? 1 : 0, nullptr, 0, nullptr, 0, local_means,
                                    global_means, lr);
    const void *fn = c->k->decode_segments(ef, store, c->P, per_tensor);
    const uint64_t grid = std::min<uint64_t>(sg->n_tiles, 0x7fffffffu);
    void *params[] = {&a, &t};
    A2_CUDA(launch_pdl(fn, dim3((unsigned)grid), params, s));
    return A2SGD_OK;
}

static int step_segments_impl(a2sgd_ctx *c, a2sgd_segments *sg, float lr, const float *lr_per_segment, void *stream)
{
    if (!c || !sg || sg->ctx != c) return A2SGD_ERR_ARG;
    if (lr_per_segment && !device_pointer_ok(c, lr_per_segment)) return A2SGD_ERR_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    DebugScope dbg(c, s);
    if (!dbg.arm(2)) return A2SGD_ERR_CUDA;
    const int rc = launch_encode_segments(c, sg, c->local_means, c->pos_counts, c->global_means, s);
    if (rc) return rc;
    return launch_decode_segments(c, sg, c->local_means, c->global_means, lr, lr_per_segment, s);
}

extern "C" int a2sgd_step_segments(a2sgd_ctx *c, a2sgd_segments *sg, float lr, void *stream)
{
    return step_segments_impl(c, sg, lr, nullptr, stream);
}

extern "C" int a2sgd_step_segments_lr(a2sgd_ctx *c, a2sgd_segments *sg, const float *lr_per_segment, void *stream)
{
    if (!lr_per_segment || !aligned(lr_per_segment, 4)) return lr_per_segment ? A2SGD_ERR_ALIGN : A2SGD_ERR_ARG;
    return step_segments_impl(c, sg, 0.0f, lr_per_segment, stream);
}

// Scratch of the per-tensor-means variant: one partial per (worker, tile), the per-tensor means and counts.
static int ensure_per_tensor_scratch(a2sgd_ctx *c, a2sgd_segments *sg)
{
    if (sg->tile_partials) return A2SGD_OK;
    const size_t P = c->P, S = sg->S;
    bool ok = true;
    ok = ok && cudaMalloc(&sg->tile_partials, sizeof(Partial) * P * sg->n_tiles) == cudaSuccess;
    ok = ok && cudaMalloc(&sg->job_partials, sizeof(Partial) * P * sg->n_jobs) == cudaSuccess;
    ok = ok && cudaMalloc(&sg->seg_local_means, sizeof(float) * 2 * P * S) == cudaSuccess;
    ok = ok && cudaMalloc(&sg->seg_counts, sizeof(unsigned long long) * P * S) == cudaSuccess;
    ok = ok && cudaMalloc(&sg->seg_global_means, sizeof(float) * 2 * S) == cudaSuccess;
    if (!ok) {
        (void)cudaGetLastError();
        cudaFree(sg->tile_partials);
        cudaFree(sg->job_partials);
        sg->job_partials = nullptr;
        cudaFree(sg->seg_local_means);
        cudaFree(sg->seg_counts);
        cudaFree(sg->seg_global_means);
        sg->tile_partials = nullptr;
        sg->seg_local_means = sg->seg_global_means = nullptr;
        sg->seg_counts = nullptr;
        (void)cudaGetLastError();
        return A2SGD_ERR_NOMEM;
    }
    return A2SGD_OK;
}

extern "C" int a2sgd_step_segments_per_tensor(a2sgd_ctx *c, a2sgd_segments *sg, float lr, const float *lr_per_segment,
                                              void *stream)
{
    if (!c || !sg || sg->ctx != c) return A2SGD_ERR_ARG;
    if (lr_per_segment && !aligned(lr_per_segment, 4)) return A2SGD_ERR_ALIGN;
    if (lr_per_segment && !device_pointer_ok(c, lr_per_segment)) return A2SGD_ERR_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    const int rc0 = ensure_per_tensor_scratch(c, sg);
    if (rc0) return rc0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    DebugScope dbg(c, s);
    if (!dbg.arm(2)) return A2SGD_ERR_CUDA;
    const int rc = launch_encode_segments(c, sg, c->local_means, c->pos_counts, nullptr, s, true);
    if (rc) return rc;
    {
        SegTables t = seg_tables(sg, nullptr);
        uint32_t P = c->P;
        int *status = c->status;
        void *params1[] = {&t};
        A2_CUDA(launch_pdl(c->k->fold_jobs, dim3(sg->n_jobs, c->P), params1, s));
        void *params[] = {&t, &P, &status};
        A2_CUDA(launch_pdl(c->k->fold_segments, dim3(sg->S), params, s));
    }
    return launch_decode_segments(c, sg, nullptr, nullptr, lr, lr_per_segment, s, true);
}

extern "C" int a2sgd_read_segment_stats(a2sgd_ctx *c, a2sgd_segments *sg, float *local_means_host,
                                        float *global_means_host, uint64_t *pos_counts_host, void *stream)
{
    if (!c || !sg || sg->ctx != c) return A2SGD_ERR_ARG;
    if (!sg->tile_partials) return A2SGD_ERR_ARG; // no per-tensor step has run on this plan
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t P = c->P, S = sg->S;
    if (local_means_host)
        A2_CUDA(cudaMemcpyAsync(local_means_host, sg->seg_local_means, sizeof(float) * 2 * P * S, cudaMemcpyDeviceToHost, s));
    if (global_means_host)
        A2_CUDA(cudaMemcpyAsync(global_means_host, sg->seg_global_means, sizeof(float) * 2 * S, cudaMemcpyDeviceToHost, s));
    if (pos_counts_host)
        A2_CUDA(cudaMemcpyAsync(pos_counts_host, sg->seg_counts, sizeof(uint64_t) * P * S, cudaMemcpyDeviceToHost, s));
    A2_CUDA(cudaStreamSynchronize(s));
    return A2SGD_OK;
}

extern "C" int a2sgd_encode_segments(a2sgd_ctx *c, a2sgd_segments *sg, float *local_means, uint64_t *pos_counts,
                                     void *stream)
{
    if (!c || !sg || sg->ctx != c || !local_means) return A2SGD_ERR_ARG;
    if (!aligned(local_means, 4) || (pos_counts && !aligned(pos_counts, 8))) return A2SGD_ERR_ALIGN;
    if (!device_pointer_ok(c, local_means) || !device_pointer_ok(c, pos_counts)) return A2SGD_ERR_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    DebugScope dbg(c, static_cast<cudaStream_t>(stream));
    if (!dbg.arm(2)) return A2SGD_ERR_CUDA;
    return launch_encode_segments(c, sg, local_means, reinterpret_cast<unsigned long long *>(pos_counts), nullptr,
                                  static_cast<cudaStream_t>(stream));
}

extern "C" int a2sgd_decode_update_segments(a2sgd_ctx *c, a2sgd_segments *sg, const float *local_means,
                                            const float *global_means, float lr, const float *lr_per_segment,
                                            void *stream)
{
    if (!c || !sg || sg->ctx != c || !global_means) return A2SGD_ERR_ARG;
    if (c->alg1 && !local_means) return A2SGD_ERR_ARG;
    if (!aligned(global_means, 4) || (local_means && !aligned(local_means, 4)) ||
        (lr_per_segment && !aligned(lr_per_segment, 4)))
        return A2SGD_ERR_ALIGN;
    if (!device_pointer_ok(c, global_means) || !device_pointer_ok(c, local_means) ||
        !device_pointer_ok(c, lr_per_segment))
        return A2SGD_ERR_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    DebugScope dbg(c, static_cast<cudaStream_t>(stream));
    if (!dbg.arm(2)) return A2SGD_ERR_CUDA;
    return launch_decode_segments(c, sg, local_means, global_means, lr, lr_per_segment,
                                  static_cast<cudaStream_t>(stream));
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
    if (st == A2SGD_ERR_TIMEOUT) {
        // CTAs that gave up left their arrivals in the barrier counter
        A2_CUDA(cudaMemsetAsync(c->barrier, 0, sizeof(unsigned int), s));
        A2_CUDA(cudaStreamSynchronize(s));
    }
    if (device_status) *device_status = st;
    return A2SGD_OK;
}

extern "C" int a2sgd_launch_info(a2sgd_ctx *c, int64_t w_stride, uint32_t out[5])
{
    if (!c || !out) return A2SGD_ERR_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return A2SGD_ERR_CUDA;
    // geometry for best-aligned buffers (what a caller that pads rows to 128 bytes gets)
    const bool ef = !c->alg1;
    const bool shared = w_stride == 0 || c->P == 1;
    const int vw = kMaxVecWidth >= 8 ? 8 : 4;
    const uint64_t items = (c->n + vw - 1) / vw;
    out[0] = std::min(per_worker_grid(c, occupancy(c, c->k->encode(ef, false, vw)), items, encode_waves(c)),
                      c->g_alloc) * c->P;
    out[1] = shared ? flat_grid(c, occupancy(c, c->k->decode_shared(ef, true, c->P, vw, false)), items, kWavesK3)
                    : per_worker_grid(c, occupancy(c, c->k->decode_repl(ef, true, vw, false)), items, kWavesK3) * c->P;
    out[2] = kBlock;
    out[3] = 0;
    if (!(c->flags & A2SGD_FORCE_TWO_PASS)) {
        uint32_t grid = 0;
        if (coop_plan(c, true, shared, vw, &grid)) {
            out[3] = 1;
            out[0] = out[1] = grid;
        }
    }
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
    case A2SGD_ERR_TOO_LARGE: return "too large: n*P for the single-launch path, or P for the fixed scratch";
    case A2SGD_ERR_BOUNDS: return "debug checks: an access outside the buffers of the call was skipped";
    default: return "unknown status";
    }
}
