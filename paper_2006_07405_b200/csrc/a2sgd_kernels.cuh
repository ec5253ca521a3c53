// Device code of the A2SGD gradient path for sm_100a.
//
// K1  encode-reduce   one streaming pass per worker over v (= g + e, or g):
//                     S_pos, S_neg, n_pos  -> two local means (Section 3.1,
//                     Algorithm 1 line 3), optional packed pos mask.
// K2  global average  mean of the 2P scalars in worker order (Algorithm 1
//                     line 5); also folded into the last CTA of K1.
// K3  decode-update   reconstruct g_hat, update the residual, SGD step
//                     (Algorithm 1 lines 4, 6, 7), one streaming pass.
//
// Everything here is bound by HBM bandwidth, so the kernels are built around
// 128/256-bit coalesced accesses with many independent loads in flight per
// thread, streaming cache policy, and no tensor cores (nothing on this path
// is a contraction).  Grids: the reduction kernels run a few CTAs per
// resident slot with grid-stride loops (few, fixed-order partial sums); the
// element-wise decode kernels are launched with one vector per thread, which
// lets the hardware CTA scheduler even out SMs that stream at different
// speeds (the host picks the grid; the loops here accept any grid).
//
// Summation.  Within one unrolled batch (8 elements) a thread adds non-negative
// fp32 values pairwise (depth 3, relative error <= 3 * 2^-24 of the batch sum);
// everything above that level — the thread's running sum, the warp and block
// trees, the cross-CTA combine — is fp64 in a fixed order.  Counts are
// integers.  No floating-point atomics: each CTA stores one partial, and the
// CTA that draws the last ticket folds all partials in index order, so the
// result depends only on (n, P, grid), never on scheduling.
//
// This header is compiled twice into the library, into two namespaces: the production kernels
// (A2SGD_NS = a2sgd, A2SGD_CHECKED = 0) and a checked copy of exactly the same code
// (a2sgd_chk, A2SGD_CHECKED = 1) in which every access made through the helpers below is first
// tested against the extents of the call's buffers (A2SGD_DEBUG_CHECKS).  Keeping the two apart
// at compile time leaves the production kernels' instructions and register counts untouched.
// No include guard: the including file sets the two macros.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "a2sgd_debug_check.h"

#ifndef A2SGD_NS
#define A2SGD_NS a2sgd
#endif
#ifndef A2SGD_CHECKED
#define A2SGD_CHECKED 0
#endif

namespace A2SGD_NS {

constexpr int kBlock = 256;
constexpr int kWarps = kBlock / 32;
constexpr int kMaxP = 1024;

// status word values (mirrors the public enum; kept separate so that this
// header depends on nothing outside the CUDA toolkit)
constexpr int kDevOk = 0;
constexpr int kDevTimeout = -4;
constexpr int kDevNonFinite = -5;
constexpr int kDevBounds = -8;

// ------------------------------------------------------------------ A2SGD_DEBUG_CHECKS
// The stand-in for a memory checker on systems where none can be run.  In the checked copy of
// the kernels, while the descriptor below is switched on (by a context created with
// A2SGD_DEBUG_CHECKS, for the duration of its launches), every access that goes through the
// helpers of this file is first checked against the extents of the buffers the call was given
// — inside the live elements of one row of one buffer — and an access that is not is SKIPPED
// (loads return 0) and latches kDevBounds in the context's status word.  Nothing traps, so a
// defect shows up as a status code instead of a fault.  One descriptor per device: launches of a
// checking context must not overlap other checked launches on the same device.
using a2sgd_check::DebugRange;
using a2sgd_check::kDebugMaxRanges;
struct DebugChecks {
    int on;    // 0 off, 1 address ranges below, 2 index checks only (the tensors of a segment list)
    int count;
    int *status;
    DebugRange range[kDebugMaxRanges];
};
#if A2SGD_CHECKED
static __constant__ DebugChecks c_debug;

static __device__ __noinline__ bool debug_access_failed(const void *p, unsigned bytes)
{
    if (a2sgd_check::debug_any_range_contains(c_debug.range, c_debug.count, (uint64_t)(uintptr_t)p, bytes)) return false;
    atomicCAS(c_debug.status, kDevOk, kDevBounds);
    return true;
}
// true: the access may be made
__device__ __forceinline__ bool access_ok(const void *p, unsigned bytes)
{
    if (c_debug.on != 1) return true;
    return !debug_access_failed(p, bytes);
}
// the index form, for the tensors of a segment list
__device__ __forceinline__ bool span_ok(uint64_t first, uint64_t count, uint64_t numel)
{
    if (c_debug.on == 0 || a2sgd_check::debug_span_inside(first, count, numel)) return true;
    atomicCAS(c_debug.status, kDevOk, kDevBounds);
    return false;
}
#else
__device__ __forceinline__ bool access_ok(const void *, unsigned) { return true; }
__device__ __forceinline__ bool span_ok(uint64_t, uint64_t, uint64_t) { return true; }
#endif

struct __align__(8) Partial {
    double s_pos;
    double s_neg;
    unsigned long long n_pos;
};

// ------------------------------------------------------------------ programmatic dependent launch
// The two kernels of a step (and the steps of a loop) are launched with programmatic stream
// serialisation: a kernel's CTAs may become resident while the previous kernel drains, which
// hides the launch latency at each kernel boundary.  Every kernel therefore waits for the
// previous grid (completion and memory flush) before its first global access, and then lets
// its own successor start being scheduled.
__device__ __forceinline__ void pdl_wait_prior_grid()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
__device__ __forceinline__ void pdl_release_next_grid()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ------------------------------------------------------------------ memory access helpers
// Streaming vector accesses, VW = 4 (128-bit) or 8 (256-bit, new on sm_100).
// Every byte on this path is touched at most twice per step (once by K1, once
// by K3) with gigabytes in between, so nothing is allocated in L1; the 256-bit
// forms also mark their L2 lines evict-first (the ISA ties that hint to the
// 256-bit width).
template <int VW>
struct Vec {
    float v[VW];
};

template <int VW>
__device__ __forceinline__ Vec<VW> ld_vec(const float *p);
template <>
__device__ __forceinline__ Vec<4> ld_vec<4>(const float *p)
{
    Vec<4> r;
    if (!access_ok(p, 16)) {
        r.v[0] = r.v[1] = r.v[2] = r.v[3] = 0.f;
        return r;
    }
    asm volatile("ld.global.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3])
                 : "l"(p));
    return r;
}
template <>
__device__ __forceinline__ Vec<8> ld_vec<8>(const float *p)
{
    Vec<8> r;
    if (!access_ok(p, 32)) {
#pragma unroll
        for (int k = 0; k < 8; ++k) r.v[k] = 0.f;
        return r;
    }
    asm volatile("ld.global.L1::no_allocate.L2::evict_first.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]), "=f"(r.v[5]),
                   "=f"(r.v[6]), "=f"(r.v[7])
                 : "l"(p));
    return r;
}
template <int VW>
__device__ __forceinline__ void st_vec(float *p, const Vec<VW> &x);
template <>
__device__ __forceinline__ void st_vec<4>(float *p, const Vec<4> &x)
{
    if (!access_ok(p, 16)) return;
    asm volatile("st.global.L1::no_allocate.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(p), "f"(x.v[0]), "f"(x.v[1]),
                 "f"(x.v[2]), "f"(x.v[3])
                 : "memory");
}
template <>
__device__ __forceinline__ void st_vec<8>(float *p, const Vec<8> &x)
{
    if (!access_ok(p, 32)) return;
    asm volatile("st.global.L1::no_allocate.L2::evict_first.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p),
                 "f"(x.v[0]), "f"(x.v[1]), "f"(x.v[2]), "f"(x.v[3]), "f"(x.v[4]), "f"(x.v[5]), "f"(x.v[6]),
                 "f"(x.v[7])
                 : "memory");
}
__device__ __forceinline__ float ld_stream1(const float *p)
{
    float r;
    if (!access_ok(p, 4)) return 0.f;
    asm volatile("ld.global.L1::no_allocate.f32 %0, [%1];" : "=f"(r) : "l"(p));
    return r;
}
__device__ __forceinline__ void st_stream1(float *p, float v)
{
    if (!access_ok(p, 4)) return;
    asm volatile("st.global.L1::no_allocate.f32 [%0], %1;" ::"l"(p), "f"(v) : "memory");
}

// Plain (cached) single-element accesses: the read-modify-write tails and the mask words.
__device__ __forceinline__ float ld1(const float *p) { return access_ok(p, 4) ? *p : 0.f; }
__device__ __forceinline__ void st1(float *p, float v)
{
    if (access_ok(p, 4)) *p = v;
}
__device__ __forceinline__ void st_word(uint32_t *p, uint32_t v)
{
    if (access_ok(p, 4)) *p = v;
}

// A gradient row whose elements are fp32 (GB = 0), bfloat16 (GB = 1) or IEEE half (GB = 2);
// Section 1 of the paper names the combination with quantisation as a natural extension.  Widening either
// 16-bit format to fp32 is exact (bfloat16 is the upper half of an fp32; every half value,
// subnormals included, is an fp32 value), so v = float(g) + e is formed from exactly the value the
// caller stored.
template <int GB>
struct GradRow {
    const char *base;
    __device__ __forceinline__ GradRow(const float *grad_base, int64_t row_offset_elems)
        : base(reinterpret_cast<const char *>(grad_base) + row_offset_elems * (GB ? 2 : 4))
    {
    }
    __device__ __forceinline__ float one(uint64_t elem) const
    {
        if (GB) {
            unsigned short h = 0;
            if (access_ok(base + 2 * elem, 2))
                asm volatile("ld.global.L1::no_allocate.u16 %0, [%1];" : "=h"(h) : "l"(base + 2 * elem));
            return GB == 1 ? __uint_as_float((unsigned)h << 16) : __half2float(__ushort_as_half(h));
        }
        return ld_stream1(reinterpret_cast<const float *>(base) + elem);
    }
    template <int VW>
    __device__ __forceinline__ Vec<VW> vec(uint64_t elem) const
    {
        if (GB) {
            static_assert(!GB || VW == 8, "16-bit gradients use 8-element (128-bit) vectors");
            unsigned x[4] = {0u, 0u, 0u, 0u};
            if (access_ok(base + 2 * elem, 16))
                asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                             : "=r"(x[0]), "=r"(x[1]), "=r"(x[2]), "=r"(x[3])
                             : "l"(base + 2 * elem));
            Vec<VW> r;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (GB == 1) {
                    r.v[2 * k] = __uint_as_float(x[k] << 16);
                    r.v[2 * k + 1] = __uint_as_float(x[k] & 0xffff0000u);
                } else {
                    r.v[2 * k] = __half2float(__ushort_as_half((unsigned short)(x[k] & 0xffffu)));
                    r.v[2 * k + 1] = __half2float(__ushort_as_half((unsigned short)(x[k] >> 16)));
                }
            }
            return r;
        }
        return ld_vec<VW>(reinterpret_cast<const float *>(base) + elem);
    }
};

// ------------------------------------------------------------------ per-element arithmetic
// The partition of Section 3.1: positive group is the IEEE comparison v >= 0
// (+0 and -0 are positive, NaN is not).  Flush-to-zero must stay off: a
// negative subnormal keeps its sign and its group.
struct Acc {
    double s_pos = 0.0;
    double s_neg = 0.0;
    unsigned int n_pos = 0;
};

__device__ __forceinline__ void split1(float v, float &sp, float &sn, unsigned &c, unsigned &bit)
{
    const bool p = v >= 0.0f;
    sp = p ? v : 0.0f;
    sn = p ? 0.0f : -v;
    c += p ? 1u : 0u;
    bit = p ? 1u : 0u;
}

// Pairwise fp32 sum of VW values (VW a power of two).
template <int VW>
__device__ __forceinline__ float tree_sum(const float *x)
{
    if (VW == 1) return x[0];
    return tree_sum<(VW > 1 ? VW / 2 : 1)>(x) + tree_sum<(VW > 1 ? VW / 2 : 1)>(x + VW / 2);
}

// One vector: pairwise fp32 sums of the two groups, count, VW-bit pos field.
template <int VW>
__device__ __forceinline__ void split_vec(const Vec<VW> &v, float &sp, float &sn, unsigned &c, unsigned &bits)
{
    float ps[VW], ns[VW];
    bits = 0;
#pragma unroll
    for (int k = 0; k < VW; ++k) {
        unsigned b;
        split1(v.v[k], ps[k], ns[k], c, b);
        bits |= b << k;
    }
    sp = tree_sum<VW>(ps);
    sn = tree_sum<VW>(ns);
}

template <int VW>
__device__ __forceinline__ Vec<VW> add_vec(const Vec<VW> &a, const Vec<VW> &b)
{
    Vec<VW> r;
#pragma unroll
    for (int k = 0; k < VW; ++k) r.v[k] = a.v[k] + b.v[k];
    return r;
}

// ------------------------------------------------------------------ fixed-order block reduction
__device__ __forceinline__ double shfl_down_f64(double x, int off)
{
    return __shfl_down_sync(0xffffffffu, x, off);
}

// Result valid in thread 0.  Order: butterfly-down inside each warp, then the
// kWarps warp results in lane order inside warp 0 — the same tree every time.
__device__ __forceinline__ void block_reduce(double &s_pos, double &s_neg, unsigned long long &n_pos,
                                             double (*sh_d)[kWarps], unsigned long long *sh_n)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        s_pos += shfl_down_f64(s_pos, off);
        s_neg += shfl_down_f64(s_neg, off);
        n_pos += __shfl_down_sync(0xffffffffu, n_pos, off);
    }
    if (lane == 0) {
        sh_d[0][warp] = s_pos;
        sh_d[1][warp] = s_neg;
        sh_n[warp] = n_pos;
    }
    __syncthreads();
    if (warp == 0) {
        s_pos = lane < kWarps ? sh_d[0][lane] : 0.0;
        s_neg = lane < kWarps ? sh_d[1][lane] : 0.0;
        n_pos = lane < kWarps ? sh_n[lane] : 0ull;
#pragma unroll
        for (int off = kWarps / 2; off > 0; off >>= 1) {
            s_pos += shfl_down_f64(s_pos, off);
            s_neg += shfl_down_f64(s_neg, off);
            n_pos += __shfl_down_sync(0xffffffffu, n_pos, off);
        }
    }
    __syncthreads();
}

// ------------------------------------------------------------------ K1: encode-reduce
struct EncodeArgs {
    const float *grad;
    int64_t grad_stride;
    const float *err;
    int64_t err_stride;
    uint64_t n;
    uint32_t P;
    // scratch owned by the context
    Partial *partials;          // [P][gridDim.x]
    unsigned int *tickets;      // [P + 1], all zero between launches
    int *status;
    // outputs
    float *local_means;         // [P][2]
    unsigned long long *pos_counts; // [P] or nullptr
    uint32_t *pos_mask;         // [P][ceil(n/32)] or nullptr
    float *global_means;        // [2] or nullptr: fold the global average into the last CTA
    const float *prev_means;    // [2]: last step's global means (deferred-residual form only)
    // second copies kept in the context for read_stats (may alias the above or be nullptr)
    float *ctx_local_means;
    unsigned long long *ctx_pos_counts;
};

// Writes the worker's means once every CTA of that worker has stored its
// partial; optionally the CTA finishing the last worker also forms the
// global means (K2 folded in).  Called by all threads of the CTA.
__device__ __forceinline__ void finish_worker(const EncodeArgs &a, uint32_t p, double s_pos, double s_neg,
                                              unsigned long long n_pos, double (*sh_d)[kWarps],
                                              unsigned long long *sh_n, int *sh_flag)
{
    const uint32_t G = gridDim.x;
    Partial *mine = a.partials + (uint64_t)p * G;
    if (threadIdx.x == 0) {
        mine[blockIdx.x].s_pos = s_pos;
        mine[blockIdx.x].s_neg = s_neg;
        mine[blockIdx.x].n_pos = n_pos;
        __threadfence();
        const unsigned int t = atomicAdd(&a.tickets[p], 1u);
        *sh_flag = (t == G - 1) ? 1 : 0;
    }
    __syncthreads();
    if (*sh_flag == 0) return;
    __threadfence();
    // last CTA of this worker: fold the G partials, thread t takes t, t+kBlock, ... in order.
    // The loads of a batch are issued together (one L2 round trip per four partials, not four);
    // the additions stay in index order.
    double fp = 0.0, fn = 0.0;
    unsigned long long fc = 0;
    for (uint32_t base = threadIdx.x; base < G; base += 4 * kBlock) {
        double bp[4], bn[4];
        unsigned long long bc[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t i = base + u * kBlock;
            bp[u] = i < G ? __ldcg(&mine[i].s_pos) : 0.0;
            bn[u] = i < G ? __ldcg(&mine[i].s_neg) : 0.0;
            bc[u] = i < G ? __ldcg(&mine[i].n_pos) : 0ull;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            fp += bp[u];
            fn += bn[u];
            fc += bc[u];
        }
    }
    __syncthreads();
    block_reduce(fp, fn, fc, sh_d, sh_n);
    if (threadIdx.x == 0) {
        const unsigned long long n_neg = a.n - fc;
        const float mu_pos = fc ? (float)(fp / (double)fc) : 0.0f;
        const float mu_neg = n_neg ? (float)(fn / (double)n_neg) : 0.0f;
        if (!isfinite(fp) || !isfinite(fn)) atomicCAS(a.status, kDevOk, kDevNonFinite);
        a.local_means[2 * p + 0] = mu_pos;
        a.local_means[2 * p + 1] = mu_neg;
        if (a.pos_counts) a.pos_counts[p] = fc;
        if (a.ctx_local_means && a.ctx_local_means != a.local_means) {
            a.ctx_local_means[2 * p + 0] = mu_pos;
            a.ctx_local_means[2 * p + 1] = mu_neg;
        }
        if (a.ctx_pos_counts && a.ctx_pos_counts != a.pos_counts) a.ctx_pos_counts[p] = fc;
        a.tickets[p] = 0; // ready for the next launch
        int last_of_all = 0;
        if (a.global_means) {
            __threadfence();
            last_of_all = atomicAdd(&a.tickets[a.P], 1u) == a.P - 1 ? 1 : 0;
        }
        *sh_flag = last_of_all;
    }
    __syncthreads();
    if (*sh_flag == 0) return;
    // The CTA that finished the last worker averages the 2P scalars (Algorithm 1 line 5).  The
    // loads are spread over the CTA (P can be 1024); the sum itself runs in worker order in fp64.
    __threadfence();
    __shared__ float sh_mu[2][kMaxP];
    for (uint32_t q = threadIdx.x; q < a.P; q += kBlock) {
        sh_mu[0][q] = __ldcg(&a.local_means[2 * q + 0]);
        sh_mu[1][q] = __ldcg(&a.local_means[2 * q + 1]);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double gp = 0.0, gn = 0.0;
        for (uint32_t q = 0; q < a.P; ++q) { // worker order
            gp += (double)sh_mu[0][q];
            gn += (double)sh_mu[1][q];
        }
        a.global_means[0] = (float)(gp / (double)a.P);
        a.global_means[1] = (float)(gn / (double)a.P);
        a.tickets[a.P] = 0;
    }
}

// Fast path, VW floats per access: bases aligned to 4*VW bytes, worker strides
// multiples of VW elements.  grid = (G, P).  Lanes are handled in groups of
// 32/VW (= one 32-element mask word) whose loop bounds are uniform across the
// group, so the sub-warp shuffles that assemble a mask word always see the
// whole group.
//
// DEFER selects the deferred-residual representation of the error buffer (EF mode, MASK on,
// VW = 8 only).  There the buffer holds, between steps, the compensated vector v of the last
// step instead of the residual e' = v - g_hat(v); the residual is formed here, one step late,
// with the previous step's global means (a.prev_means) — the same fp32 subtraction the decode
// kernel would have done, so every value is bit-identical — and the new v is written back in
// place.  The decode kernel then needs only the sign mask and w.  DEFER = 1: the buffer still
// holds a true residual (first step, or after a2sgd_materialize_err); DEFER = 2: it holds v.
template <bool EF, bool MASK, int VW, int GB = 0, int DEFER = 0>
__global__ void __launch_bounds__(kBlock) k_encode_vec(EncodeArgs a)
{
    static_assert(DEFER == 0 || (EF && MASK && VW == 8 && !GB), "deferred residual: EF, mask, 256-bit, fp32 gradients");
    pdl_wait_prior_grid();
    pdl_release_next_grid();

    constexpr int LPW = 32 / VW;  // lanes per mask word
    constexpr int U = 8 / VW;     // vectors per trip: 8 elements per thread per batch.  One 256-bit vector of g
                                  // and of e per trip keeps the kernel at 48 registers (5 CTAs per SM); two per
                                  // trip (64 B + 64 B in flight per thread, 4 CTAs per SM) measured 1-2 % slower
    __shared__ double sh_d[2][kWarps];
    __shared__ unsigned long long sh_n[kWarps];
    __shared__ int sh_flag;

    const uint32_t p = blockIdx.y;
    const GradRow<GB> g(a.grad, (int64_t)p * a.grad_stride);
    const float *e = EF ? a.err + (int64_t)p * a.err_stride : nullptr;
    float *e_out = DEFER ? const_cast<float *>(e) : nullptr; // deferred form rewrites the buffer in place
    float dm_pos = 0.f, dm_neg = 0.f;
    if (DEFER == 2) {
        dm_pos = __ldcg(a.prev_means);
        dm_neg = -__ldcg(a.prev_means + 1);
    }
    // the residual owed from the previous step: x - (x >= 0 ? m_pos : -m_neg)
    auto owed = [&](float x) { return DEFER == 2 ? x - (x >= 0.0f ? dm_pos : dm_neg) : x; };
    auto owed_vec = [&](Vec<VW> x) {
        if (DEFER == 2) {
#pragma unroll
            for (int k = 0; k < VW; ++k) x.v[k] = owed(x.v[k]);
        }
        return x;
    };
    const uint64_t nv = a.n / VW;
    const uint64_t full_words = a.n >> 5;
    uint32_t *mask = MASK ? a.pos_mask + (uint64_t)p * ((a.n + 31) >> 5) : nullptr;

    const unsigned lane = threadIdx.x & 31u;
    const unsigned sub = lane & (LPW - 1);
    const unsigned group_mask = ((1u << LPW) - 1u) << (lane & ~(unsigned)(LPW - 1));
    const uint64_t stride = (uint64_t)gridDim.x * kBlock;
    uint64_t j = (uint64_t)blockIdx.x * kBlock + threadIdx.x;

    Acc acc;

    auto emit_word = [&](unsigned bits, uint64_t jv) {
        if (MASK) {
            unsigned w = bits << (VW * sub);
#pragma unroll
            for (int x = 1; x < LPW; x <<= 1) w |= __shfl_xor_sync(group_mask, w, x);
            const uint64_t word = jv / LPW;
            if (sub == 0 && word < full_words) st_word(mask + word, w);
        }
    };

    // main loop: U vectors per thread per trip, all loads issued before use
    for (; (j - sub + (LPW - 1)) + (U - 1) * stride < nv; j += U * stride) {
        Vec<VW> gv[U], ev[U];
#pragma unroll
        for (int u = 0; u < U; ++u) gv[u] = g.template vec<VW>(VW * (j + u * stride));
        if (EF) {
#pragma unroll
            for (int u = 0; u < U; ++u) ev[u] = ld_vec<VW>(e + VW * (j + u * stride));
        }
        float sp[U], sn[U];
        unsigned bits[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const Vec<VW> v = EF ? add_vec<VW>(gv[u], owed_vec(ev[u])) : gv[u];
            if (DEFER) st_vec<VW>(e_out + VW * (j + u * stride), v);
            split_vec<VW>(v, sp[u], sn[u], acc.n_pos, bits[u]);
        }
        acc.s_pos += (double)tree_sum<U>(sp);
        acc.s_neg += (double)tree_sum<U>(sn);
#pragma unroll
        for (int u = 0; u < U; ++u) emit_word(bits[u], j + u * stride);
    }
    // remainder: one vector per trip, bounds uniform per lane group
    for (; (j - sub) < nv; j += stride) {
        float sp = 0.f, sn = 0.f;
        unsigned bits = 0;
        if (j < nv) {
            Vec<VW> v = g.template vec<VW>(VW * j);
            if (EF) v = add_vec<VW>(v, owed_vec(ld_vec<VW>(e + VW * j)));
            if (DEFER) st_vec<VW>(e_out + VW * j, v);
            split_vec<VW>(v, sp, sn, acc.n_pos, bits);
        }
        acc.s_pos += (double)sp;
        acc.s_neg += (double)sn;
        emit_word(bits, j);
    }
    if (blockIdx.x == 0) {
        // the n % VW trailing elements
        const uint64_t i = nv * VW + threadIdx.x;
        if (threadIdx.x < VW && i < a.n) {
            float v = g.one(i);
            if (EF) v += owed(ld_stream1(e + i));
            if (DEFER) st_stream1(e_out + i, v);
            float sp, sn;
            unsigned bit;
            split1(v, sp, sn, acc.n_pos, bit);
            acc.s_pos += (double)sp;
            acc.s_neg += (double)sn;
        }
        // the last, partial mask word (n % 32 elements): one warp re-reads them.  Not in the
        // deferred form (the buffer is being rewritten): its decode reads v itself for those elements.
        if (MASK && !DEFER && threadIdx.x < 32 && (a.n & 31u)) {
            const uint64_t i2 = (full_words << 5) + lane;
            bool pos = false;
            if (i2 < a.n) {
                float v = g.one(i2);
                if (EF) v += ld_stream1(e + i2);
                pos = v >= 0.0f;
            }
            const unsigned w = __ballot_sync(0xffffffffu, pos);
            if (lane == 0) st_word(mask + full_words, w);
        }
    }
    double s_pos = acc.s_pos, s_neg = acc.s_neg;
    unsigned long long n_pos = acc.n_pos;
    block_reduce(s_pos, s_neg, n_pos, sh_d, sh_n);
    finish_worker(a, p, s_pos, s_neg, n_pos, sh_d, sh_n, &sh_flag);
}

// General path: any 4-byte alignment, coalesced 32-bit accesses.  grid = (G, P).
// A CTA walks tiles of kBlock * kScalarU consecutive elements; within a tile a thread takes the
// elements tid, tid + kBlock, ... so that every load instruction of a warp is one contiguous
// 128-byte piece whatever the row's alignment.  All loads of a tile are issued before the first
// use, the kScalarU values are summed pairwise in fp32 and enter the fp64 running sums once per
// tile — the same arithmetic shape as the vector kernel, only with narrower accesses.
constexpr int kScalarU = 8;

template <bool EF, bool MASK, int GB = 0>
__global__ void __launch_bounds__(kBlock) k_encode_scalar(EncodeArgs a)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();

    __shared__ double sh_d[2][kWarps];
    __shared__ unsigned long long sh_n[kWarps];
    __shared__ int sh_flag;

    const uint32_t p = blockIdx.y;
    const GradRow<GB> g(a.grad, (int64_t)p * a.grad_stride);
    const float *__restrict__ e = EF ? a.err + (int64_t)p * a.err_stride : nullptr;
    uint32_t *mask = MASK ? a.pos_mask + (uint64_t)p * ((a.n + 31) >> 5) : nullptr;
    const unsigned lane = threadIdx.x & 31u;
    constexpr uint64_t kTile = (uint64_t)kBlock * kScalarU;
    const uint64_t tiles = (a.n + kTile - 1) / kTile;
    Acc acc;
    for (uint64_t t = blockIdx.x; t < tiles; t += gridDim.x) {
        const uint64_t base = t * kTile + threadIdx.x;
        float gv[kScalarU], ev[kScalarU];
        const bool whole = (t + 1) * kTile <= a.n;
        if (whole) {
#pragma unroll
            for (int k = 0; k < kScalarU; ++k) gv[k] = g.one(base + (uint64_t)k * kBlock);
            if (EF) {
#pragma unroll
                for (int k = 0; k < kScalarU; ++k) ev[k] = ld_stream1(e + base + (uint64_t)k * kBlock);
            }
        } else {
#pragma unroll
            for (int k = 0; k < kScalarU; ++k) {
                const uint64_t i = base + (uint64_t)k * kBlock;
                gv[k] = i < a.n ? g.one(i) : 0.f;
                ev[k] = (EF && i < a.n) ? ld_stream1(e + i) : 0.f;
            }
        }
        float sp[kScalarU], sn[kScalarU];
#pragma unroll
        for (int k = 0; k < kScalarU; ++k) {
            const uint64_t i = base + (uint64_t)k * kBlock;
            const float v = EF ? gv[k] + ev[k] : gv[k];
            unsigned bit = 0;
            sp[k] = sn[k] = 0.f;
            if (whole || i < a.n) split1(v, sp[k], sn[k], acc.n_pos, bit);
            if (MASK && (whole || (i - lane) < a.n)) {       // warp-uniform: the warp's 32 elements share a word
                const unsigned w = __ballot_sync(0xffffffffu, bit != 0);
                if (lane == 0) st_word(mask + (i >> 5), w);
            }
        }
        acc.s_pos += (double)tree_sum<kScalarU>(sp);
        acc.s_neg += (double)tree_sum<kScalarU>(sn);
    }
    double s_pos = acc.s_pos, s_neg = acc.s_neg;
    unsigned long long n_pos = acc.n_pos;
    block_reduce(s_pos, s_neg, n_pos, sh_d, sh_n);
    finish_worker(a, p, s_pos, s_neg, n_pos, sh_d, sh_n, &sh_flag);
}

// ------------------------------------------------------------------ K2: global average (stand-alone form)
static __global__ void k_global_average(const float *__restrict__ local_means, uint32_t P, float *global_means,
                                 float *ctx_global_means)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();

    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    double gp = 0.0, gn = 0.0;
    for (uint32_t q = 0; q < P; ++q) { // worker order
        gp += (double)local_means[2 * q + 0];
        gn += (double)local_means[2 * q + 1];
    }
    const float m_pos = (float)(gp / (double)P), m_neg = (float)(gn / (double)P);
    global_means[0] = m_pos;
    global_means[1] = m_neg;
    if (ctx_global_means && ctx_global_means != global_means) {
        ctx_global_means[0] = m_pos;
        ctx_global_means[1] = m_neg;
    }
}

// Algorithm 1 line 5 when the workers sit on different GPUs and a collective has already formed
// the sums of the two means over all workers (fp64): divide by the worker count, round once.
static __global__ void k_global_average_from_sums(const double *__restrict__ sums, uint32_t workers,
                                                  float *global_means, float *ctx_global_means)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const float m_pos = (float)(sums[0] / (double)workers), m_neg = (float)(sums[1] / (double)workers);
    global_means[0] = m_pos;
    global_means[1] = m_neg;
    if (ctx_global_means && ctx_global_means != global_means) {
        ctx_global_means[0] = m_pos;
        ctx_global_means[1] = m_neg;
    }
}

// ------------------------------------------------------------------ K3: decode + residual + SGD
struct DecodeArgs {
    float *w;
    int64_t w_stride; // 0 = shared
    const float *grad;
    int64_t grad_stride;
    float *err; // EF: in/out; ALG1: out or nullptr
    int64_t err_stride;
    uint64_t n;
    uint32_t P;
    const float *local_means;  // [P][2] (ALG1)
    const float *global_means; // [2]
    float lr;
    // momentum / weight-decay form of the update (MOM kernels only); mom has the layout of w
    float *mom;
    int64_t mom_stride;
    float beta;
    float weight_decay;
};

// The update applied to one weight once its reconstructed gradient is known.
//   plain (Algorithm 1 line 7):  w <- w + scale * g_sum          (scale = -lr, or -lr/P for a shared w)
//   MOM (heavy-ball momentum and weight decay acting on the reconstructed gradient):
//        u = g_sum / p + wd * w;   m <- beta * m + u;   w <- w - lr * m
struct UpdateConst {
    float scale;  // plain form
    float p;      // MOM: divisor of g_sum (1 for a replica, P for a shared w)
    float beta, wd, neg_lr;
};

template <bool MOM>
__device__ __forceinline__ float update1(const UpdateConst &u, float g_sum, float w, float &m)
{
    if (MOM) {
        const float gbar = u.p == 1.0f ? g_sum : g_sum / u.p;
        m = fmaf(u.beta, m, fmaf(u.wd, w, gbar));
        return fmaf(u.neg_lr, m, w);
    }
    return fmaf(u.scale, g_sum, w);
}

template <bool MOM, int VW>
__device__ __forceinline__ Vec<VW> update_vec(const UpdateConst &u, const Vec<VW> &g_sum, const Vec<VW> &w, Vec<VW> &m)
{
    Vec<VW> r;
#pragma unroll
    for (int k = 0; k < VW; ++k) r.v[k] = update1<MOM>(u, g_sum.v[k], w.v[k], m.v[k]);
    return r;
}

__device__ __forceinline__ UpdateConst update_const(const DecodeArgs &a, float divisor)
{
    UpdateConst u;
    u.scale = -a.lr / divisor;
    u.p = divisor;
    u.beta = a.beta;
    u.wd = a.weight_decay;
    u.neg_lr = -a.lr;
    return u;
}

// Per-worker constants of the reconstruction.
//   EF  : g_hat = pos ? m_pos : -m_neg                      e' = v - g_hat
//   ALG1: g_hat = v + (pos ? m_pos - mu_pos : mu_neg - m_neg)   eps = v - (pos ? mu_pos : -mu_neg)
// (the ALG1 form adds the net gain of Eq. 13 to g in one rounding; with P = 1
// the gain is exactly zero and g_hat == g.)
struct WorkerConst {
    float a_pos, a_neg; // EF: the two values of g_hat; ALG1: the two values of the net gain
    float b_pos, b_neg; // ALG1: the two values of enc(g)
};

template <bool EF>
__device__ __forceinline__ WorkerConst worker_const(const DecodeArgs &a, uint32_t p, float m_pos, float m_neg)
{
    WorkerConst c;
    if (EF) {
        c.a_pos = m_pos;
        c.a_neg = -m_neg;
        c.b_pos = c.b_neg = 0.f;
    } else {
        const float mu_pos = __ldg(a.local_means + 2 * p), mu_neg = __ldg(a.local_means + 2 * p + 1);
        c.a_pos = m_pos - mu_pos;
        c.a_neg = mu_neg - m_neg;
        c.b_pos = mu_pos;
        c.b_neg = -mu_neg;
    }
    return c;
}

// v (already g + e in EF mode) -> g_hat, and the residual to store.
template <bool EF>
__device__ __forceinline__ void decode1(float v, const WorkerConst &c, float &g_hat, float &resid)
{
    const bool p = v >= 0.0f;
    if (EF) {
        g_hat = p ? c.a_pos : c.a_neg;
        resid = v - g_hat;
    } else {
        g_hat = v + (p ? c.a_pos : c.a_neg);
        resid = v - (p ? c.b_pos : c.b_neg);
    }
}

template <bool EF, int VW>
__device__ __forceinline__ void decode_vec(const Vec<VW> &v, const WorkerConst &c, Vec<VW> &g_hat, Vec<VW> &resid)
{
#pragma unroll
    for (int k = 0; k < VW; ++k) decode1<EF>(v.v[k], c, g_hat.v[k], resid.v[k]);
}

template <int VW>
__device__ __forceinline__ Vec<VW> axpy_vec(float alpha, const Vec<VW> &x, const Vec<VW> &y)
{
    Vec<VW> r;
#pragma unroll
    for (int k = 0; k < VW; ++k) r.v[k] = fmaf(alpha, x.v[k], y.v[k]);
    return r;
}

template <int VW>
__device__ __forceinline__ Vec<VW> zero_vec()
{
    Vec<VW> r;
#pragma unroll
    for (int k = 0; k < VW; ++k) r.v[k] = 0.f;
    return r;
}

// One shared w: each thread owns a VW-vector of the model and walks the P
// workers in order (fixed summation order), so w is read and written once
// per model element.  PT > 0: P known at compile time (all 2P+1 loads of a
// vector are issued before any is used); PT == 0: run-time P.
template <bool EF, bool STORE, int PT, int VW, int GB = 0, bool MOM = false>
__global__ void __launch_bounds__(kBlock) k_decode_shared_vec(DecodeArgs a)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();

    __shared__ WorkerConst sh_c[PT > 0 ? 1 : kMaxP];
    const uint32_t P = PT > 0 ? PT : a.P;
    const float m_pos = __ldg(a.global_means), m_neg = __ldg(a.global_means + 1);
    const UpdateConst uc = update_const(a, (float)P);
    const uint64_t nv = a.n / VW;
    const uint64_t stride = (uint64_t)gridDim.x * kBlock;

    if (PT > 0) {
        constexpr int PP = PT > 0 ? PT : 1;
        WorkerConst c[PP];
#pragma unroll
        for (int p = 0; p < PP; ++p) c[p] = worker_const<EF>(a, p, m_pos, m_neg);
        for (uint64_t j = (uint64_t)blockIdx.x * kBlock + threadIdx.x; j < nv; j += stride) {
            // workers whose loads are in flight together; 4 measured better than 8 at P = 8
            // (6.55 -> 6.77 TB/s): fewer concurrent streams per thread, lower register count
            constexpr int PB = PP < 4 ? PP : 4;
            const Vec<VW> wv = ld_vec<VW>(a.w + VW * j);
            Vec<VW> mv = MOM ? ld_vec<VW>(a.mom + VW * j) : zero_vec<VW>();
            Vec<VW> sum = zero_vec<VW>();
#pragma unroll
            for (int p0 = 0; p0 < PP; p0 += PB) {
                Vec<VW> gv[PB], ev[PB];
#pragma unroll
                for (int q = 0; q < PB; ++q)
                    gv[q] = GradRow<GB>(a.grad, (int64_t)(p0 + q) * a.grad_stride).template vec<VW>(VW * j);
                if (EF) {
#pragma unroll
                    for (int q = 0; q < PB; ++q)
                        ev[q] = ld_vec<VW>(a.err + (int64_t)(p0 + q) * a.err_stride + VW * j);
                }
#pragma unroll
                for (int q = 0; q < PB; ++q) {
                    const Vec<VW> v = EF ? add_vec<VW>(gv[q], ev[q]) : gv[q];
                    Vec<VW> gh, rs;
                    decode_vec<EF, VW>(v, c[p0 + q], gh, rs);
                    sum = add_vec<VW>(sum, gh);
                    if (STORE) st_vec<VW>(a.err + (int64_t)(p0 + q) * a.err_stride + VW * j, rs);
                }
            }
            st_vec<VW>(a.w + VW * j, update_vec<MOM, VW>(uc, sum, wv, mv));
            if (MOM) st_vec<VW>(a.mom + VW * j, mv);
        }
    } else {
        for (uint32_t p = threadIdx.x; p < P; p += kBlock) sh_c[p] = worker_const<EF>(a, p, m_pos, m_neg);
        __syncthreads();
        for (uint64_t j = (uint64_t)blockIdx.x * kBlock + threadIdx.x; j < nv; j += stride) {
            const Vec<VW> wv = ld_vec<VW>(a.w + VW * j);
            Vec<VW> mv = MOM ? ld_vec<VW>(a.mom + VW * j) : zero_vec<VW>();
            Vec<VW> sum = zero_vec<VW>();
            for (uint32_t p = 0; p < P; ++p) {
                Vec<VW> v = GradRow<GB>(a.grad, (int64_t)p * a.grad_stride).template vec<VW>(VW * j);
                if (EF) v = add_vec<VW>(v, ld_vec<VW>(a.err + (int64_t)p * a.err_stride + VW * j));
                Vec<VW> gh, rs;
                decode_vec<EF, VW>(v, sh_c[p], gh, rs);
                sum = add_vec<VW>(sum, gh);
                if (STORE) st_vec<VW>(a.err + (int64_t)p * a.err_stride + VW * j, rs);
            }
            st_vec<VW>(a.w + VW * j, update_vec<MOM, VW>(uc, sum, wv, mv));
            if (MOM) st_vec<VW>(a.mom + VW * j, mv);
        }
    }
    // the n % VW trailing elements
    if (blockIdx.x == 0 && threadIdx.x < VW) {
        const uint64_t i = nv * VW + threadIdx.x;
        if (i < a.n) {
            float sum = 0.f;
            for (uint32_t p = 0; p < P; ++p) {
                const WorkerConst c = worker_const<EF>(a, p, m_pos, m_neg);
                float v = GradRow<GB>(a.grad, (int64_t)p * a.grad_stride).one(i);
                if (EF) v += ld_stream1(a.err + (int64_t)p * a.err_stride + i);
                float gh, rs;
                decode1<EF>(v, c, gh, rs);
                sum += gh;
                if (STORE) st_stream1(a.err + (int64_t)p * a.err_stride + i, rs);
            }
            float m = MOM ? ld1(a.mom + i) : 0.f;
            st1(a.w + i, update1<MOM>(uc, sum, ld1(a.w + i), m));
            if (MOM) st1(a.mom + i, m);
        }
    }
}

// One w replica per worker (Algorithm 1's layout).  grid = (G, P).
template <bool EF, bool STORE, int VW, int GB = 0, bool MOM = false>
__global__ void __launch_bounds__(kBlock) k_decode_repl_vec(DecodeArgs a)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();

    const uint32_t p = blockIdx.y;
    const float m_pos = __ldg(a.global_means), m_neg = __ldg(a.global_means + 1);
    const WorkerConst c = worker_const<EF>(a, p, m_pos, m_neg);
    const GradRow<GB> g(a.grad, (int64_t)p * a.grad_stride);
    float *e = (EF || STORE) ? a.err + (int64_t)p * a.err_stride : nullptr;
    float *w = a.w + (int64_t)p * a.w_stride;
    float *mom = MOM ? a.mom + (int64_t)p * a.mom_stride : nullptr;
    const UpdateConst uc = update_const(a, 1.0f);
    const uint64_t nv = a.n / VW;
    const uint64_t stride = (uint64_t)gridDim.x * kBlock;
    uint64_t j = (uint64_t)blockIdx.x * kBlock + threadIdx.x;
    constexpr int U = 8 / VW;
    for (; j + (U - 1) * stride < nv; j += U * stride) {
        Vec<VW> gv[U], ev[U], wv[U], mv[U];
#pragma unroll
        for (int u = 0; u < U; ++u) gv[u] = g.template vec<VW>(VW * (j + u * stride));
        if (EF) {
#pragma unroll
            for (int u = 0; u < U; ++u) ev[u] = ld_vec<VW>(e + VW * (j + u * stride));
        }
#pragma unroll
        for (int u = 0; u < U; ++u) wv[u] = ld_vec<VW>(w + VW * (j + u * stride));
#pragma unroll
        for (int u = 0; u < U; ++u) mv[u] = MOM ? ld_vec<VW>(mom + VW * (j + u * stride)) : zero_vec<VW>();
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const Vec<VW> v = EF ? add_vec<VW>(gv[u], ev[u]) : gv[u];
            Vec<VW> gh, rs;
            decode_vec<EF, VW>(v, c, gh, rs);
            if (STORE) st_vec<VW>(e + VW * (j + u * stride), rs);
            st_vec<VW>(w + VW * (j + u * stride), update_vec<MOM, VW>(uc, gh, wv[u], mv[u]));
            if (MOM) st_vec<VW>(mom + VW * (j + u * stride), mv[u]);
        }
    }
    for (; j < nv; j += stride) {
        Vec<VW> v = g.template vec<VW>(VW * j);
        if (EF) v = add_vec<VW>(v, ld_vec<VW>(e + VW * j));
        const Vec<VW> wv = ld_vec<VW>(w + VW * j);
        Vec<VW> mv = MOM ? ld_vec<VW>(mom + VW * j) : zero_vec<VW>();
        Vec<VW> gh, rs;
        decode_vec<EF, VW>(v, c, gh, rs);
        if (STORE) st_vec<VW>(e + VW * j, rs);
        st_vec<VW>(w + VW * j, update_vec<MOM, VW>(uc, gh, wv, mv));
        if (MOM) st_vec<VW>(mom + VW * j, mv);
    }
    if (blockIdx.x == 0 && threadIdx.x < VW) {
        const uint64_t i = nv * VW + threadIdx.x;
        if (i < a.n) {
            float v = g.one(i);
            if (EF) v += ld_stream1(e + i);
            float gh, rs;
            decode1<EF>(v, c, gh, rs);
            if (STORE) st_stream1(e + i, rs);
            float m = MOM ? ld1(mom + i) : 0.f;
            st1(w + i, update1<MOM>(uc, gh, ld1(w + i), m));
            if (MOM) st1(mom + i, m);
        }
    }
}

// General path: any 4-byte alignment, both weight layouts, coalesced 32-bit accesses.
// One tile of kBlock * kDecScalarU consecutive model elements per CTA (grid.x = number of tiles);
// a thread takes the elements tid, tid + kBlock, ... of the tile.  Shared w: grid = (tiles, 1), the
// thread walks the workers in batches of four with all loads of a batch issued before its first
// store; replicas: grid = (tiles, P).
constexpr int kDecScalarU = 4;

template <bool EF, bool STORE, int GB = 0, bool MOM = false>
__global__ void __launch_bounds__(kBlock) k_decode_scalar(DecodeArgs a)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();

    __shared__ WorkerConst sh_c[kMaxP];
    const float m_pos = __ldg(a.global_means), m_neg = __ldg(a.global_means + 1);
    const bool shared = a.w_stride == 0;
    const uint32_t p_lo = shared ? 0 : blockIdx.y, p_hi = shared ? a.P : blockIdx.y + 1;
    const UpdateConst uc = update_const(a, shared ? (float)a.P : 1.0f);
    for (uint32_t p = p_lo + threadIdx.x; p < p_hi; p += kBlock) sh_c[p] = worker_const<EF>(a, p, m_pos, m_neg);
    __syncthreads();

    constexpr int U = kDecScalarU, PB = 4;
    constexpr uint64_t kTile = (uint64_t)kBlock * U;
    const uint64_t tiles = (a.n + kTile - 1) / kTile;
    for (uint64_t t = blockIdx.x; t < tiles; t += gridDim.x) {
        const uint64_t base = t * kTile + threadIdx.x;
        bool live[U];
        float wv[U], mv[U], sum[U];
        float *wrow = a.w + (int64_t)p_lo * a.w_stride;
        float *mrow = MOM ? a.mom + (int64_t)p_lo * a.mom_stride : nullptr;
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const uint64_t i = base + (uint64_t)k * kBlock;
            live[k] = i < a.n;
            wv[k] = live[k] ? ld_stream1(wrow + i) : 0.f;
            mv[k] = (MOM && live[k]) ? ld_stream1(mrow + i) : 0.f;
            sum[k] = 0.f;
        }
        for (uint32_t p0 = p_lo; p0 < p_hi; p0 += PB) {
            float gv[PB][U], ev[PB][U];
#pragma unroll
            for (int q = 0; q < PB; ++q) {
                const bool wq = p0 + q < p_hi;
                const GradRow<GB> g(a.grad, (int64_t)(wq ? p0 + q : p0) * a.grad_stride);
#pragma unroll
                for (int k = 0; k < U; ++k) gv[q][k] = (wq && live[k]) ? g.one(base + (uint64_t)k * kBlock) : 0.f;
            }
            if (EF) {
#pragma unroll
                for (int q = 0; q < PB; ++q) {
                    const bool wq = p0 + q < p_hi;
                    const float *e = a.err + (int64_t)(wq ? p0 + q : p0) * a.err_stride;
#pragma unroll
                    for (int k = 0; k < U; ++k) ev[q][k] = (wq && live[k]) ? ld_stream1(e + base + (uint64_t)k * kBlock) : 0.f;
                }
            }
#pragma unroll
            for (int q = 0; q < PB; ++q) {
                if (p0 + q >= p_hi) break;
                const WorkerConst c = sh_c[p0 + q];
                float *e = STORE ? a.err + (int64_t)(p0 + q) * a.err_stride : nullptr;
#pragma unroll
                for (int k = 0; k < U; ++k) {
                    if (!live[k]) continue;
                    const float v = EF ? gv[q][k] + ev[q][k] : gv[q][k];
                    float gh, rs;
                    decode1<EF>(v, c, gh, rs);
                    sum[k] += gh;
                    if (STORE) st_stream1(e + base + (uint64_t)k * kBlock, rs);
                }
            }
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            if (!live[k]) continue;
            const uint64_t i = base + (uint64_t)k * kBlock;
            float m = mv[k];
            st_stream1(wrow + i, update1<MOM>(uc, sum[k], wv[k], m));
            if (MOM) st_stream1(mrow + i, m);
        }
    }
}

// ------------------------------------------------------------------ K3', deferred-residual form
// The error buffer already holds v (written by the encode kernel) and the residual is not formed
// until the next step, so decoding needs only pos(v) — one bit per worker-element from the packed
// mask — and w: (P/8 + 8) bytes per model element instead of (12P + 8).  g_hat values are summed in
// worker order exactly as in k_decode_shared_vec, so w is bit-identical to the canonical path.
// The mask covers the full 32-element words; the last n % 32 elements are decoded from v itself.
struct DeferredDecodeArgs {
    float *w;
    int64_t w_stride; // 0 = shared
    const float *v;   // the error buffer, holding v
    int64_t v_stride;
    const uint32_t *mask; // [P][ceil(n/32)]
    uint64_t n;
    uint32_t P;
    const float *global_means; // [2], this step's
    float *prev_means;         // [2], out: copy of this step's means for the next encode
    float lr;
};

template <int PT, bool REPL>
__global__ void __launch_bounds__(kBlock) k_decode_deferred(DeferredDecodeArgs a)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    const uint32_t P = PT > 0 ? PT : a.P;
    const float m_pos = __ldg(a.global_means), m_neg = __ldg(a.global_means + 1);
    const float g_pos = m_pos, g_neg = -m_neg;
    const float scale = REPL ? -a.lr : -a.lr / (float)P;
    const uint64_t words = (a.n + 31) >> 5, full_words = a.n >> 5;
    const uint64_t nv = full_words * 4; // 8-element vectors covered by full mask words
    const uint64_t stride = (uint64_t)gridDim.x * kBlock;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        a.prev_means[0] = m_pos;
        a.prev_means[1] = m_neg;
    }
    for (uint64_t j = (uint64_t)blockIdx.x * kBlock + threadIdx.x; j < nv; j += stride) {
        const unsigned shift = 8u * (unsigned)(j & 3);
        if (REPL) {
            for (uint32_t p = 0; p < P; ++p) {
                const unsigned bits = (__ldg(a.mask + (uint64_t)p * words + (j >> 2)) >> shift) & 0xffu;
                float *wp = a.w + (int64_t)p * a.w_stride + 8 * j;
                Vec<8> wv = ld_vec<8>(wp);
#pragma unroll
                for (int k = 0; k < 8; ++k) wv.v[k] = fmaf(scale, ((bits >> k) & 1u) ? g_pos : g_neg, wv.v[k]);
                st_vec<8>(wp, wv);
            }
        } else {
            const Vec<8> wv = ld_vec<8>(a.w + 8 * j);
            Vec<8> sum = zero_vec<8>();
            if (PT > 0) {
                unsigned bits[PT > 0 ? PT : 1];
#pragma unroll
                for (int p = 0; p < PT; ++p) bits[p] = (__ldg(a.mask + (uint64_t)p * words + (j >> 2)) >> shift) & 0xffu;
#pragma unroll
                for (int p = 0; p < PT; ++p) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) sum.v[k] += ((bits[p] >> k) & 1u) ? g_pos : g_neg;
                }
            } else {
                for (uint32_t p = 0; p < P; ++p) {
                    const unsigned bits = (__ldg(a.mask + (uint64_t)p * words + (j >> 2)) >> shift) & 0xffu;
#pragma unroll
                    for (int k = 0; k < 8; ++k) sum.v[k] += ((bits >> k) & 1u) ? g_pos : g_neg;
                }
            }
            st_vec<8>(a.w + 8 * j, axpy_vec<8>(scale, sum, wv));
        }
    }
    // the last n % 32 elements: pos(v) read from v itself
    if (blockIdx.x == 0 && threadIdx.x < 32) {
        const uint64_t i = (full_words << 5) + threadIdx.x;
        if (i < a.n) {
            float sum = 0.f;
            for (uint32_t p = 0; p < P; ++p) {
                const float gh = (ld1(a.v + (int64_t)p * a.v_stride + i) >= 0.0f) ? g_pos : g_neg;
                if (REPL) {
                    float *wp = a.w + (int64_t)p * a.w_stride + i;
                    st1(wp, fmaf(scale, gh, ld1(wp)));
                } else {
                    sum += gh;
                }
            }
            if (!REPL) st1(a.w + i, fmaf(scale, sum, ld1(a.w + i)));
        }
    }
}

// Turns a buffer that holds v back into the true residual e' = v - g_hat(v) with the means of the
// step that produced it (checkpointing, or leaving the deferred form).  grid.y = worker.
static __global__ void __launch_bounds__(kBlock) k_materialize_err(float *v, int64_t v_stride, uint64_t n,
                                                                   const float *means)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    float *row = v + (int64_t)blockIdx.y * v_stride;
    const float g_pos = __ldg(means), g_neg = -__ldg(means + 1);
    const uint64_t nv = n / 8, stride = (uint64_t)gridDim.x * kBlock;
    for (uint64_t j = (uint64_t)blockIdx.x * kBlock + threadIdx.x; j < nv; j += stride) {
        Vec<8> x = ld_vec<8>(row + 8 * j);
#pragma unroll
        for (int k = 0; k < 8; ++k) x.v[k] = x.v[k] - (x.v[k] >= 0.0f ? g_pos : g_neg);
        st_vec<8>(row + 8 * j, x);
    }
    if (blockIdx.x == 0 && threadIdx.x < 8) {
        const uint64_t i = nv * 8 + threadIdx.x;
        if (i < n) {
            const float x = ld1(row + i);
            st1(row + i, x - (x >= 0.0f ? g_pos : g_neg));
        }
    }
}

// ------------------------------------------------------------------ K5: dense synchronisation step
// Algorithm 1 lines 9-10 (Eq. 1 for one step): w <- w - lr * (1/P) sum_p g^p.
// One streaming pass: P gradient vectors in, summed in worker order, w updated.
// Shared w: (4P + 8) B per model element; replicas (REPL): every replica gets
// the same averaged update, (4P + 8P) B.  One vector per thread.
struct DenseArgs {
    float *w;
    int64_t w_stride; // 0 = shared
    const float *grad;
    int64_t grad_stride;
    uint64_t n;
    uint32_t P;       // gradient rows summed here
    float lr;
    float divisor;    // workers the mean is taken over: P, or more when the rows are already sums over ranks
};

template <int PT, int VW, bool REPL>
__global__ void __launch_bounds__(kBlock) k_dense_sync_vec(DenseArgs a)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    const uint32_t P = PT > 0 ? PT : a.P;
    const float scale = -a.lr / a.divisor;
    const uint64_t nv = a.n / VW;
    const uint64_t stride = (uint64_t)gridDim.x * kBlock;
    for (uint64_t j = (uint64_t)blockIdx.x * kBlock + threadIdx.x; j < nv; j += stride) {
        Vec<VW> sum = zero_vec<VW>();
        if (PT > 0) {
            constexpr int PP = PT > 0 ? PT : 1;
            Vec<VW> gv[PP];
#pragma unroll
            for (int p = 0; p < PP; ++p) gv[p] = ld_vec<VW>(a.grad + (int64_t)p * a.grad_stride + VW * j);
#pragma unroll
            for (int p = 0; p < PP; ++p) sum = add_vec<VW>(sum, gv[p]);
        } else {
            for (uint32_t p = 0; p < P; ++p) sum = add_vec<VW>(sum, ld_vec<VW>(a.grad + (int64_t)p * a.grad_stride + VW * j));
        }
        if (REPL) {
            for (uint32_t p = 0; p < P; ++p) {
                float *wp = a.w + (int64_t)p * a.w_stride + VW * j;
                st_vec<VW>(wp, axpy_vec<VW>(scale, sum, ld_vec<VW>(wp)));
            }
        } else {
            st_vec<VW>(a.w + VW * j, axpy_vec<VW>(scale, sum, ld_vec<VW>(a.w + VW * j)));
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < VW) {
        const uint64_t i = nv * VW + threadIdx.x;
        if (i < a.n) {
            float sum = 0.f;
            for (uint32_t p = 0; p < P; ++p) sum += ld_stream1(a.grad + (int64_t)p * a.grad_stride + i);
            const uint32_t reps = REPL ? P : 1;
            for (uint32_t r = 0; r < reps; ++r) {
                float *wp = a.w + (int64_t)r * a.w_stride + i;
                st1(wp, fmaf(scale, sum, ld1(wp)));
            }
        }
    }
}

// Any 4-byte alignment.
__global__ void __launch_bounds__(kBlock) static k_dense_sync_scalar(DenseArgs a)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    const float scale = -a.lr / a.divisor;
    const uint64_t stride = (uint64_t)gridDim.x * kBlock;
    const uint32_t reps = a.w_stride == 0 ? 1 : a.P;
    for (uint64_t i = (uint64_t)blockIdx.x * kBlock + threadIdx.x; i < a.n; i += stride) {
        float sum = 0.f;
        for (uint32_t p = 0; p < a.P; ++p) sum += ld_stream1(a.grad + (int64_t)p * a.grad_stride + i);
        for (uint32_t r = 0; r < reps; ++r) {
            float *wp = a.w + (int64_t)r * a.w_stride + i;
            st1(wp, fmaf(scale, sum, ld1(wp)));
        }
    }
}

// ------------------------------------------------------------------ K4: single cooperative launch
// For n*P small enough that every thread can keep its share of v in
// registers: phase 1 loads g (and e) once and reduces, a grid-wide barrier
// publishes the means, phase 2 decodes from the registers.  HBM traffic is
// 20 B per worker-element instead of 28, and one launch instead of two.
// Must be launched cooperatively (all CTAs co-resident).  The barrier wait is
// bounded: a CTA that gives up latches kDevTimeout and returns without
// writing any output.
struct CoopArgs {
    EncodeArgs enc;            // pos_mask unused; global_means required
    DecodeArgs dec;
    unsigned int *barrier;     // [0] arrival counter (zero between launches), [1] generation counter
    unsigned int expected;     // arrivals that open the barrier (= gridDim.x in normal use)
    unsigned int spin_limit;   // polls before giving up
};

constexpr int kCoopVecPerThread = 8; // 128-bit vectors of v a thread may hold, summed over its workers

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int *p)
{
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u32(unsigned int *p, unsigned int v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Shared memory of the single-launch kernels' reduction and barrier.
template <int PT>
struct CoopShared {
    double part[PT][2][kWarps];
    unsigned long long cnt[PT][kWarps];
    float mu[PT][2];
    unsigned int generation;
    int flag;
};

__device__ __forceinline__ void warp_reduce3(double &s_pos, double &s_neg, unsigned long long &n_pos, int width)
{
    for (int off = width / 2; off > 0; off >>= 1) {
        s_pos += shfl_down_f64(s_pos, off);
        s_neg += shfl_down_f64(s_neg, off);
        n_pos += __shfl_down_sync(0xffffffffu, n_pos, off);
    }
}

// Block reduction of all PT workers at once (warp w finishes worker w), partial sums to scratch,
// grid barrier.  The last CTA to arrive folds the partials — all workers at the same time, each by
// its own group of warps in a fixed order — publishes the local and global means and opens the
// barrier; the others poll a release word a bounded number of times.  Returns false in a CTA that
// gave up.  PT <= kWarps.
template <int PT>
__device__ __forceinline__ bool coop_reduce_and_barrier(const CoopArgs &a, Acc (&acc)[PT], CoopShared<PT> &sh)
{
    static_assert(PT <= kWarps, "one warp per worker");
    const EncodeArgs &ea = a.enc;
    const uint32_t G = gridDim.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int p = 0; p < PT; ++p) {
        double s_pos = acc[p].s_pos, s_neg = acc[p].s_neg;
        unsigned long long n_pos = acc[p].n_pos;
        warp_reduce3(s_pos, s_neg, n_pos, 32);
        if (lane == 0) {
            sh.part[p][0][warp] = s_pos;
            sh.part[p][1][warp] = s_neg;
            sh.cnt[p][warp] = n_pos;
        }
    }
    __syncthreads();
    if (warp < PT) {
        double s_pos = lane < kWarps ? sh.part[warp][0][lane] : 0.0;
        double s_neg = lane < kWarps ? sh.part[warp][1][lane] : 0.0;
        unsigned long long n_pos = lane < kWarps ? sh.cnt[warp][lane] : 0ull;
        warp_reduce3(s_pos, s_neg, n_pos, kWarps);
        if (lane == 0) {
            Partial *mine = ea.partials + (uint64_t)warp * G;
            mine[blockIdx.x].s_pos = s_pos;
            mine[blockIdx.x].s_neg = s_neg;
            mine[blockIdx.x].n_pos = n_pos;
        }
    }
    __syncthreads();
    // ---- grid barrier (one fence per CTA: fences are the expensive part of this path)
    // The release word is a generation counter that lives on the device: every CTA notes its value
    // before arriving and waits for it to change; the last arriver increments it.  It cannot change
    // before all CTAs have arrived, hence after all have read it.  Nothing depends on a value passed
    // from the host, so a captured launch can be replayed any number of times.
    if (threadIdx.x == 0) {
        sh.generation = ld_acquire_u32(&a.barrier[1]);
        __threadfence();
        const unsigned int t = atomicAdd(&a.barrier[0], 1u);
        int role = (t == a.expected - 1) ? 1 : 0;
        // A CTA that gave up has written nothing.  If one already did, the last arriver leaves the
        // barrier shut, so the remaining CTAs run out too and the step is abandoned as a whole
        // (best effort: a CTA may still give up just after this check).
        if (role == 1 && ld_acquire_u32(reinterpret_cast<const unsigned int *>(ea.status)) == (unsigned int)kDevTimeout)
            role = -1;
        sh.flag = role;
    }
    __syncthreads();
    // every thread takes its own copy before the word is reused for the outcome of the wait below
    const int role = sh.flag;
    __syncthreads();
    if (role < 0) return false;
    if (role == 1) {
        __threadfence();
        // kWarps / PT warps fold each worker's G partials: thread tg of the group takes partials
        // tg, tg + group size, ... (index order), then a fixed tree inside the group
        constexpr int WPW = kWarps / PT;
        const int worker = warp / WPW, warp_in_group = warp % WPW;
        if (worker < PT) {
            const Partial *part = ea.partials + (uint64_t)worker * G;
            double fp = 0.0, fn = 0.0;
            unsigned long long fc = 0;
#pragma unroll 4
            for (uint32_t i = warp_in_group * 32 + lane; i < G; i += WPW * 32) {
                fp += __ldcg(&part[i].s_pos);
                fn += __ldcg(&part[i].s_neg);
                fc += __ldcg(&part[i].n_pos);
            }
            warp_reduce3(fp, fn, fc, 32);
            if (lane == 0) {
                sh.part[worker][0][warp_in_group] = fp;
                sh.part[worker][1][warp_in_group] = fn;
                sh.cnt[worker][warp_in_group] = fc;
            }
        }
        __syncthreads();
        if (warp < PT) {
            double fp = lane < WPW ? sh.part[warp][0][lane] : 0.0;
            double fn = lane < WPW ? sh.part[warp][1][lane] : 0.0;
            unsigned long long fc = lane < WPW ? sh.cnt[warp][lane] : 0ull;
            warp_reduce3(fp, fn, fc, kWarps);
            if (lane == 0) {
                const unsigned long long n_neg = ea.n - fc;
                const float mu_pos = fc ? (float)(fp / (double)fc) : 0.0f;
                const float mu_neg = n_neg ? (float)(fn / (double)n_neg) : 0.0f;
                sh.mu[warp][0] = mu_pos;
                sh.mu[warp][1] = mu_neg;
                ea.local_means[2 * warp + 0] = mu_pos;
                ea.local_means[2 * warp + 1] = mu_neg;
                if (ea.pos_counts) ea.pos_counts[warp] = fc;
                if (!isfinite(fp) || !isfinite(fn)) atomicCAS(ea.status, kDevOk, kDevNonFinite);
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            double gp = 0.0, gn = 0.0;
            for (uint32_t q = 0; q < PT; ++q) { // worker order
                gp += (double)sh.mu[q][0];
                gn += (double)sh.mu[q][1];
            }
            ea.global_means[0] = (float)(gp / (double)PT);
            ea.global_means[1] = (float)(gn / (double)PT);
            a.barrier[0] = 0;
            __threadfence();
            st_release_u32(&a.barrier[1], sh.generation + 1u);
        }
        __syncthreads();
    } else {
        if (threadIdx.x == 0) {
            unsigned int polls = 0;
            int ok = 1;
            while (ld_acquire_u32(&a.barrier[1]) == sh.generation) {
                if (++polls > a.spin_limit) {
                    ok = 0;
                    break;
                }
                __nanosleep(40);
            }
            if (!ok) atomicCAS(ea.status, kDevOk, kDevTimeout);
            sh.flag = ok ? 2 : -1;
        }
        __syncthreads();
        if (sh.flag < 0) return false; // gave up: no output is written by this CTA
    }
    return true;
}

// Constants of the reconstruction for every worker, read after the barrier.
template <bool EF, int PT>
__device__ __forceinline__ void coop_worker_consts(const EncodeArgs &ea, WorkerConst (&c)[PT])
{
    const float m_pos = __ldcg(ea.global_means), m_neg = __ldcg(ea.global_means + 1);
#pragma unroll
    for (int p = 0; p < PT; ++p) {
        if (EF) {
            c[p].a_pos = m_pos;
            c[p].a_neg = -m_neg;
            c[p].b_pos = c[p].b_neg = 0.f;
        } else {
            const float mu_pos = __ldcg(ea.local_means + 2 * p), mu_neg = __ldcg(ea.local_means + 2 * p + 1);
            c[p].a_pos = m_pos - mu_pos;
            c[p].a_neg = mu_neg - m_neg;
            c[p].b_pos = mu_pos;
            c[p].b_neg = -mu_neg;
        }
    }
}

template <bool EF, bool STORE, int PT, bool SHARED>
__global__ void __launch_bounds__(kBlock) k_step_coop(CoopArgs a)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    constexpr int K = kCoopVecPerThread / PT;
    __shared__ CoopShared<PT> sh;

    const EncodeArgs &ea = a.enc;
    const DecodeArgs &da = a.dec;
    const uint64_t n4 = ea.n >> 2;
    const uint64_t T = (uint64_t)gridDim.x * kBlock;
    const uint64_t tid = (uint64_t)blockIdx.x * kBlock + threadIdx.x;
    const bool has_tail = blockIdx.x == 0 && threadIdx.x < 4 && (n4 << 2) + threadIdx.x < ea.n;
    const uint64_t i_tail = (n4 << 2) + threadIdx.x;

    // ---- phase 1: load, form v, reduce per worker
    Vec<4> v[PT][K];
    float v_tail[PT];
    Acc acc[PT];
#pragma unroll
    for (int p = 0; p < PT; ++p) {
        const float *g = ea.grad + (int64_t)p * ea.grad_stride;
        const float *e = EF ? ea.err + (int64_t)p * ea.err_stride : nullptr;
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const uint64_t j = tid + (uint64_t)k * T;
            v[p][k] = zero_vec<4>();
            if (j < n4) {
                v[p][k] = ld_vec<4>(g + 4 * j);
                if (EF) v[p][k] = add_vec<4>(v[p][k], ld_vec<4>(e + 4 * j));
            }
        }
        v_tail[p] = 0.f;
        if (has_tail) {
            v_tail[p] = ld_stream1(g + i_tail);
            if (EF) v_tail[p] += ld_stream1(e + i_tail);
        }
    }
#pragma unroll
    for (int p = 0; p < PT; ++p) {
        float sp[K], sn[K];
#pragma unroll
        for (int k = 0; k < K; ++k) {
            sp[k] = sn[k] = 0.f;
            unsigned bits;
            if (tid + (uint64_t)k * T < n4) split_vec<4>(v[p][k], sp[k], sn[k], acc[p].n_pos, bits);
        }
        acc[p].s_pos = (double)tree_sum<K>(sp);
        acc[p].s_neg = (double)tree_sum<K>(sn);
        if (has_tail) {
            float tp, tn;
            unsigned bit;
            split1(v_tail[p], tp, tn, acc[p].n_pos, bit);
            acc[p].s_pos += (double)tp;
            acc[p].s_neg += (double)tn;
        }
    }
    if (!coop_reduce_and_barrier<PT>(a, acc, sh)) return;
    // ---- phase 2: decode from registers
    WorkerConst c[PT];
    coop_worker_consts<EF, PT>(ea, c);
    const float scale = SHARED ? -da.lr / (float)PT : -da.lr;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const uint64_t j = tid + (uint64_t)k * T;
        if (j >= n4) continue;
        if (SHARED) {
            const Vec<4> wv = ld_vec<4>(da.w + 4 * j);
            Vec<4> sum = zero_vec<4>();
#pragma unroll
            for (int p = 0; p < PT; ++p) {
                Vec<4> gh, rs;
                decode_vec<EF, 4>(v[p][k], c[p], gh, rs);
                sum = add_vec<4>(sum, gh);
                if (STORE) st_vec<4>(da.err + (int64_t)p * da.err_stride + 4 * j, rs);
            }
            st_vec<4>(da.w + 4 * j, axpy_vec<4>(scale, sum, wv));
        } else {
            Vec<4> wv[PT];
#pragma unroll
            for (int p = 0; p < PT; ++p) wv[p] = ld_vec<4>(da.w + (int64_t)p * da.w_stride + 4 * j);
#pragma unroll
            for (int p = 0; p < PT; ++p) {
                Vec<4> gh, rs;
                decode_vec<EF, 4>(v[p][k], c[p], gh, rs);
                if (STORE) st_vec<4>(da.err + (int64_t)p * da.err_stride + 4 * j, rs);
                st_vec<4>(da.w + (int64_t)p * da.w_stride + 4 * j, axpy_vec<4>(scale, gh, wv[p]));
            }
        }
    }
    if (has_tail) {
        float sum = 0.f;
#pragma unroll
        for (int p = 0; p < PT; ++p) {
            float gh, rs;
            decode1<EF>(v_tail[p], c[p], gh, rs);
            if (STORE) st_stream1(da.err + (int64_t)p * da.err_stride + i_tail, rs);
            if (SHARED) {
                sum += gh;
            } else {
                float *wp = da.w + (int64_t)p * da.w_stride + i_tail;
                st1(wp, fmaf(scale, gh, ld1(wp)));
            }
        }
        if (SHARED) st1(da.w + i_tail, fmaf(scale, sum, ld1(da.w + i_tail)));
    }
}

// L2-resident form of the single launch: for sizes whose g, e and w together fit in L2 but not in
// registers.  Phase 1 streams g and e (they stay in L2: 128-bit loads without an eviction hint),
// phase 2 reads them again from L2 after the barrier, so HBM still sees each byte once.
template <bool EF, bool STORE, int PT, bool SHARED>
__global__ void __launch_bounds__(kBlock) k_step_coop_l2(CoopArgs a)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    __shared__ CoopShared<PT> sh;
    const EncodeArgs &ea = a.enc;
    const DecodeArgs &da = a.dec;
    const uint64_t n4 = ea.n >> 2;
    const uint64_t T = (uint64_t)gridDim.x * kBlock;
    const uint64_t tid = (uint64_t)blockIdx.x * kBlock + threadIdx.x;
    const bool has_tail = blockIdx.x == 0 && threadIdx.x < 4 && (n4 << 2) + threadIdx.x < ea.n;
    const uint64_t i_tail = (n4 << 2) + threadIdx.x;

    Acc acc[PT];
    for (uint64_t j = tid; j < n4; j += T) {
        Vec<4> gv[PT], ev[PT];
#pragma unroll
        for (int p = 0; p < PT; ++p) gv[p] = ld_vec<4>(ea.grad + (int64_t)p * ea.grad_stride + 4 * j);
        if (EF) {
#pragma unroll
            for (int p = 0; p < PT; ++p) ev[p] = ld_vec<4>(ea.err + (int64_t)p * ea.err_stride + 4 * j);
        }
#pragma unroll
        for (int p = 0; p < PT; ++p) {
            const Vec<4> v = EF ? add_vec<4>(gv[p], ev[p]) : gv[p];
            float sp, sn;
            unsigned bits;
            split_vec<4>(v, sp, sn, acc[p].n_pos, bits);
            acc[p].s_pos += (double)sp;
            acc[p].s_neg += (double)sn;
        }
    }
    if (has_tail) {
#pragma unroll
        for (int p = 0; p < PT; ++p) {
            float v = ld_stream1(ea.grad + (int64_t)p * ea.grad_stride + i_tail);
            if (EF) v += ld_stream1(ea.err + (int64_t)p * ea.err_stride + i_tail);
            float tp, tn;
            unsigned bit;
            split1(v, tp, tn, acc[p].n_pos, bit);
            acc[p].s_pos += (double)tp;
            acc[p].s_neg += (double)tn;
        }
    }
    if (!coop_reduce_and_barrier<PT>(a, acc, sh)) return;
    WorkerConst c[PT];
    coop_worker_consts<EF, PT>(ea, c);
    const float scale = SHARED ? -da.lr / (float)PT : -da.lr;
    for (uint64_t j = tid; j < n4; j += T) {
        Vec<4> gv[PT], ev[PT], wv[SHARED ? 1 : PT];
#pragma unroll
        for (int p = 0; p < PT; ++p) gv[p] = ld_vec<4>(da.grad + (int64_t)p * da.grad_stride + 4 * j);
        if (EF) {
#pragma unroll
            for (int p = 0; p < PT; ++p) ev[p] = ld_vec<4>(da.err + (int64_t)p * da.err_stride + 4 * j);
        }
        if (SHARED) {
            wv[0] = ld_vec<4>(da.w + 4 * j);
        } else {
#pragma unroll
            for (int p = 0; p < PT; ++p) wv[SHARED ? 0 : p] = ld_vec<4>(da.w + (int64_t)p * da.w_stride + 4 * j);
        }
        Vec<4> sum = zero_vec<4>();
#pragma unroll
        for (int p = 0; p < PT; ++p) {
            const Vec<4> v = EF ? add_vec<4>(gv[p], ev[p]) : gv[p];
            Vec<4> gh, rs;
            decode_vec<EF, 4>(v, c[p], gh, rs);
            if (STORE) st_vec<4>(da.err + (int64_t)p * da.err_stride + 4 * j, rs);
            if (SHARED) sum = add_vec<4>(sum, gh);
            else st_vec<4>(da.w + (int64_t)p * da.w_stride + 4 * j, axpy_vec<4>(scale, gh, wv[SHARED ? 0 : p]));
        }
        if (SHARED) st_vec<4>(da.w + 4 * j, axpy_vec<4>(scale, sum, wv[0]));
    }
    if (has_tail) {
        float sum = 0.f;
#pragma unroll
        for (int p = 0; p < PT; ++p) {
            float v = ld_stream1(da.grad + (int64_t)p * da.grad_stride + i_tail);
            if (EF) v += ld_stream1(da.err + (int64_t)p * da.err_stride + i_tail);
            float gh, rs;
            decode1<EF>(v, c[p], gh, rs);
            if (STORE) st_stream1(da.err + (int64_t)p * da.err_stride + i_tail, rs);
            if (SHARED) {
                sum += gh;
            } else {
                float *wp = da.w + (int64_t)p * da.w_stride + i_tail;
                st1(wp, fmaf(scale, gh, ld1(wp)));
            }
        }
        if (SHARED) st1(da.w + i_tail, fmaf(scale, sum, ld1(da.w + i_tail)));
    }
}

} // namespace A2SGD_NS
