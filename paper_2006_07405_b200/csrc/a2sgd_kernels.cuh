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
// 128-bit coalesced accesses with many independent loads in flight per
// thread, persistent grids sized to the SM count, streaming cache policy, and
// no tensor cores (nothing on this path is a contraction).
//
// Summation.  Within one unrolled batch a thread adds non-negative fp32
// values pairwise (depth <= 4, relative error <= 4 * 2^-24 of the batch sum);
// everything above that level — the thread's running sum, the warp and block
// trees, the cross-CTA combine — is fp64 in a fixed order.  Counts are
// integers.  No floating-point atomics: each CTA stores one partial, and the
// CTA that draws the last ticket folds all partials in index order, so the
// result depends only on (n, P, grid), never on scheduling.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace a2sgd {

constexpr int kBlock = 256;
constexpr int kWarps = kBlock / 32;
constexpr int kMaxP = 1024;

// status word values (mirrors the public enum; kept separate so that this
// header depends on nothing outside the CUDA toolkit)
constexpr int kDevOk = 0;
constexpr int kDevTimeout = -4;
constexpr int kDevNonFinite = -5;

struct __align__(8) Partial {
    double s_pos;
    double s_neg;
    unsigned long long n_pos;
};

// ------------------------------------------------------------------ memory access helpers
// Streaming 128-bit accesses.  Every byte on this path is touched at most
// twice per step (once by K1, once by K3) with gigabytes in between, so L1
// allocation is pointless and L2 lines should be first in line for eviction.
__device__ __forceinline__ float4 ld_stream(const float *p)
{
    float4 r;
    asm volatile("ld.global.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w)
                 : "l"(p));
    return r;
}
__device__ __forceinline__ float ld_stream1(const float *p)
{
    float r;
    asm volatile("ld.global.L1::no_allocate.f32 %0, [%1];" : "=f"(r) : "l"(p));
    return r;
}
__device__ __forceinline__ void st_stream(float *p, float4 v)
{
    asm volatile("st.global.L1::no_allocate.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(p),
                 "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
                 : "memory");
}
__device__ __forceinline__ void st_stream1(float *p, float v)
{
    asm volatile("st.global.L1::no_allocate.f32 [%0], %1;" ::"l"(p), "f"(v) : "memory");
}

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

// One 4-vector: pairwise fp32 sums of the two groups, count, 4-bit pos nibble.
__device__ __forceinline__ void split4(float4 v, float &sp, float &sn, unsigned &c, unsigned &nib)
{
    float p0, p1, p2, p3, n0, n1, n2, n3;
    unsigned b0, b1, b2, b3;
    split1(v.x, p0, n0, c, b0);
    split1(v.y, p1, n1, c, b1);
    split1(v.z, p2, n2, c, b2);
    split1(v.w, p3, n3, c, b3);
    sp = (p0 + p1) + (p2 + p3);
    sn = (n0 + n1) + (n2 + n3);
    nib = b0 | (b1 << 1) | (b2 << 2) | (b3 << 3);
}

__device__ __forceinline__ float4 add4(float4 a, float4 b)
{
    return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
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
    // last CTA of this worker: fold the G partials, thread t takes t, t+kBlock, ... in order
    double fp = 0.0, fn = 0.0;
    unsigned long long fc = 0;
    for (uint32_t i = threadIdx.x; i < G; i += kBlock) {
        fp += __ldcg(&mine[i].s_pos);
        fn += __ldcg(&mine[i].s_neg);
        fc += __ldcg(&mine[i].n_pos);
    }
    __syncthreads();
    block_reduce(fp, fn, fc, sh_d, sh_n);
    if (threadIdx.x != 0) return;
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
    if (a.global_means) {
        __threadfence();
        const unsigned int t = atomicAdd(&a.tickets[a.P], 1u);
        if (t == a.P - 1) {
            __threadfence();
            double gp = 0.0, gn = 0.0;
            for (uint32_t q = 0; q < a.P; ++q) { // worker order
                gp += (double)__ldcg(&a.local_means[2 * q + 0]);
                gn += (double)__ldcg(&a.local_means[2 * q + 1]);
            }
            a.global_means[0] = (float)(gp / (double)a.P);
            a.global_means[1] = (float)(gn / (double)a.P);
            a.tickets[a.P] = 0;
        }
    }
}

// Fast path: 16-byte aligned bases, strides multiple of 4.  grid = (G, P).
// Lanes are handled in groups of 8 (= one 32-element mask word) whose loop
// bounds are uniform across the group, so the sub-warp shuffles that assemble
// a mask word always see all eight lanes.
template <bool EF, bool MASK>
__global__ void __launch_bounds__(kBlock) k_encode_vec(EncodeArgs a)
{
    __shared__ double sh_d[2][kWarps];
    __shared__ unsigned long long sh_n[kWarps];
    __shared__ int sh_flag;

    const uint32_t p = blockIdx.y;
    const float *__restrict__ g = a.grad + (int64_t)p * a.grad_stride;
    const float *__restrict__ e = EF ? a.err + (int64_t)p * a.err_stride : nullptr;
    const uint64_t n4 = a.n >> 2;
    const uint64_t full_words = a.n >> 5;
    uint32_t *mask = MASK ? a.pos_mask + (uint64_t)p * ((a.n + 31) >> 5) : nullptr;

    const unsigned lane = threadIdx.x & 31u;
    const unsigned sub = lane & 7u;
    const unsigned group_mask = 0xffu << (lane & ~7u);
    const uint64_t stride = (uint64_t)gridDim.x * kBlock;
    uint64_t j = (uint64_t)blockIdx.x * kBlock + threadIdx.x;

    Acc acc;

    auto emit_word = [&](unsigned nib, uint64_t jv) {
        if (MASK) {
            unsigned w = nib << (4u * sub);
            w |= __shfl_xor_sync(group_mask, w, 1);
            w |= __shfl_xor_sync(group_mask, w, 2);
            w |= __shfl_xor_sync(group_mask, w, 4);
            const uint64_t word = jv >> 3;
            if (sub == 0 && word < full_words) mask[word] = w;
        }
    };

    // main loop: 4 vectors per thread per trip, all loads issued before use
    for (; (j - sub + 7) + 3 * stride < n4; j += 4 * stride) {
        float4 gv[4], ev[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) gv[u] = ld_stream(g + 4 * (j + u * stride));
        if (EF) {
#pragma unroll
            for (int u = 0; u < 4; ++u) ev[u] = ld_stream(e + 4 * (j + u * stride));
        }
        float sp[4], sn[4];
        unsigned nib[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float4 v = EF ? add4(gv[u], ev[u]) : gv[u];
            split4(v, sp[u], sn[u], acc.n_pos, nib[u]);
        }
        acc.s_pos += (double)((sp[0] + sp[1]) + (sp[2] + sp[3]));
        acc.s_neg += (double)((sn[0] + sn[1]) + (sn[2] + sn[3]));
#pragma unroll
        for (int u = 0; u < 4; ++u) emit_word(nib[u], j + u * stride);
    }
    // remainder: one vector per trip, bounds uniform per group of 8 lanes
    for (; (j - sub) < n4; j += stride) {
        float sp = 0.f, sn = 0.f;
        unsigned nib = 0;
        if (j < n4) {
            float4 v = ld_stream(g + 4 * j);
            if (EF) v = add4(v, ld_stream(e + 4 * j));
            split4(v, sp, sn, acc.n_pos, nib);
        }
        acc.s_pos += (double)sp;
        acc.s_neg += (double)sn;
        emit_word(nib, j);
    }
    if (blockIdx.x == 0) {
        // the n % 4 trailing elements
        const uint64_t i = (n4 << 2) + threadIdx.x;
        if (threadIdx.x < 4 && i < a.n) {
            float v = ld_stream1(g + i);
            if (EF) v += ld_stream1(e + i);
            float sp, sn;
            unsigned bit;
            split1(v, sp, sn, acc.n_pos, bit);
            acc.s_pos += (double)sp;
            acc.s_neg += (double)sn;
        }
        // the last, partial mask word (n % 32 elements): one warp re-reads them
        if (MASK && threadIdx.x < 32 && (a.n & 31u)) {
            const uint64_t i2 = (full_words << 5) + lane;
            bool pos = false;
            if (i2 < a.n) {
                float v = ld_stream1(g + i2);
                if (EF) v += ld_stream1(e + i2);
                pos = v >= 0.0f;
            }
            const unsigned w = __ballot_sync(0xffffffffu, pos);
            if (lane == 0) mask[full_words] = w;
        }
    }
    double s_pos = acc.s_pos, s_neg = acc.s_neg;
    unsigned long long n_pos = acc.n_pos;
    block_reduce(s_pos, s_neg, n_pos, sh_d, sh_n);
    finish_worker(a, p, s_pos, s_neg, n_pos, sh_d, sh_n, &sh_flag);
}

// General path: any 4-byte alignment, scalar coalesced accesses.  grid = (G, P).
template <bool EF, bool MASK>
__global__ void __launch_bounds__(kBlock) k_encode_scalar(EncodeArgs a)
{
    __shared__ double sh_d[2][kWarps];
    __shared__ unsigned long long sh_n[kWarps];
    __shared__ int sh_flag;

    const uint32_t p = blockIdx.y;
    const float *__restrict__ g = a.grad + (int64_t)p * a.grad_stride;
    const float *__restrict__ e = EF ? a.err + (int64_t)p * a.err_stride : nullptr;
    uint32_t *mask = MASK ? a.pos_mask + (uint64_t)p * ((a.n + 31) >> 5) : nullptr;
    const unsigned lane = threadIdx.x & 31u;
    const uint64_t stride = (uint64_t)gridDim.x * kBlock;
    Acc acc;
    for (uint64_t i = (uint64_t)blockIdx.x * kBlock + threadIdx.x; (i - lane) < a.n; i += stride) {
        float sp = 0.f, sn = 0.f;
        unsigned bit = 0;
        if (i < a.n) {
            float v = ld_stream1(g + i);
            if (EF) v += ld_stream1(e + i);
            split1(v, sp, sn, acc.n_pos, bit);
        }
        acc.s_pos += (double)sp;
        acc.s_neg += (double)sn;
        if (MASK) {
            const unsigned w = __ballot_sync(0xffffffffu, bit != 0);
            if (lane == 0) mask[i >> 5] = w;
        }
    }
    double s_pos = acc.s_pos, s_neg = acc.s_neg;
    unsigned long long n_pos = acc.n_pos;
    block_reduce(s_pos, s_neg, n_pos, sh_d, sh_n);
    finish_worker(a, p, s_pos, s_neg, n_pos, sh_d, sh_n, &sh_flag);
}

// ------------------------------------------------------------------ K2: global average (stand-alone form)
__global__ void k_global_average(const float *__restrict__ local_means, uint32_t P, float *global_means,
                                 float *ctx_global_means)
{
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
};

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

template <bool EF>
__device__ __forceinline__ void decode4(float4 v, const WorkerConst &c, float4 &g_hat, float4 &resid)
{
    decode1<EF>(v.x, c, g_hat.x, resid.x);
    decode1<EF>(v.y, c, g_hat.y, resid.y);
    decode1<EF>(v.z, c, g_hat.z, resid.z);
    decode1<EF>(v.w, c, g_hat.w, resid.w);
}

// One shared w: each thread owns a 4-vector of the model and walks the P
// workers in order (fixed summation order), so w is read and written once
// per model element.  PT > 0: P known at compile time (all 2P+1 loads of a
// vector are issued before any is used); PT == 0: run-time P.
template <bool EF, bool STORE, int PT>
__global__ void __launch_bounds__(kBlock) k_decode_shared_vec(DecodeArgs a)
{
    __shared__ WorkerConst sh_c[PT > 0 ? 1 : kMaxP];
    const uint32_t P = PT > 0 ? PT : a.P;
    const float m_pos = __ldg(a.global_means), m_neg = __ldg(a.global_means + 1);
    const float scale = -a.lr / (float)P;
    const uint64_t n4 = a.n >> 2;
    const uint64_t stride = (uint64_t)gridDim.x * kBlock;

    if (PT > 0) {
        WorkerConst c[PT > 0 ? PT : 1];
#pragma unroll
        for (int p = 0; p < PT; ++p) c[p] = worker_const<EF>(a, p, m_pos, m_neg);
        for (uint64_t j = (uint64_t)blockIdx.x * kBlock + threadIdx.x; j < n4; j += stride) {
            float4 gv[PT > 0 ? PT : 1], ev[PT > 0 ? PT : 1];
            const float4 wv = ld_stream(a.w + 4 * j);
#pragma unroll
            for (int p = 0; p < PT; ++p) gv[p] = ld_stream(a.grad + (int64_t)p * a.grad_stride + 4 * j);
            if (EF) {
#pragma unroll
                for (int p = 0; p < PT; ++p) ev[p] = ld_stream(a.err + (int64_t)p * a.err_stride + 4 * j);
            }
            float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int p = 0; p < PT; ++p) {
                const float4 v = EF ? add4(gv[p], ev[p]) : gv[p];
                float4 gh, rs;
                decode4<EF>(v, c[p], gh, rs);
                sum = add4(sum, gh);
                if (STORE) st_stream(a.err + (int64_t)p * a.err_stride + 4 * j, rs);
            }
            st_stream(a.w + 4 * j, make_float4(fmaf(scale, sum.x, wv.x), fmaf(scale, sum.y, wv.y),
                                               fmaf(scale, sum.z, wv.z), fmaf(scale, sum.w, wv.w)));
        }
    } else {
        for (uint32_t p = threadIdx.x; p < P; p += kBlock) sh_c[p] = worker_const<EF>(a, p, m_pos, m_neg);
        __syncthreads();
        for (uint64_t j = (uint64_t)blockIdx.x * kBlock + threadIdx.x; j < n4; j += stride) {
            const float4 wv = ld_stream(a.w + 4 * j);
            float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
            for (uint32_t p = 0; p < P; ++p) {
                float4 v = ld_stream(a.grad + (int64_t)p * a.grad_stride + 4 * j);
                if (EF) v = add4(v, ld_stream(a.err + (int64_t)p * a.err_stride + 4 * j));
                float4 gh, rs;
                decode4<EF>(v, sh_c[p], gh, rs);
                sum = add4(sum, gh);
                if (STORE) st_stream(a.err + (int64_t)p * a.err_stride + 4 * j, rs);
            }
            st_stream(a.w + 4 * j, make_float4(fmaf(scale, sum.x, wv.x), fmaf(scale, sum.y, wv.y),
                                               fmaf(scale, sum.z, wv.z), fmaf(scale, sum.w, wv.w)));
        }
    }
    // the n % 4 trailing elements
    if (blockIdx.x == 0 && threadIdx.x < 4) {
        const uint64_t i = (n4 << 2) + threadIdx.x;
        if (i < a.n) {
            float sum = 0.f;
            for (uint32_t p = 0; p < P; ++p) {
                const WorkerConst c = worker_const<EF>(a, p, m_pos, m_neg);
                float v = ld_stream1(a.grad + (int64_t)p * a.grad_stride + i);
                if (EF) v += ld_stream1(a.err + (int64_t)p * a.err_stride + i);
                float gh, rs;
                decode1<EF>(v, c, gh, rs);
                sum += gh;
                if (STORE) st_stream1(a.err + (int64_t)p * a.err_stride + i, rs);
            }
            a.w[i] = fmaf(scale, sum, a.w[i]);
        }
    }
}

// One w replica per worker (Algorithm 1's layout).  grid = (G, P).
template <bool EF, bool STORE>
__global__ void __launch_bounds__(kBlock) k_decode_repl_vec(DecodeArgs a)
{
    const uint32_t p = blockIdx.y;
    const float m_pos = __ldg(a.global_means), m_neg = __ldg(a.global_means + 1);
    const WorkerConst c = worker_const<EF>(a, p, m_pos, m_neg);
    const float *__restrict__ g = a.grad + (int64_t)p * a.grad_stride;
    float *e = (EF || STORE) ? a.err + (int64_t)p * a.err_stride : nullptr;
    float *w = a.w + (int64_t)p * a.w_stride;
    const float neg_lr = -a.lr;
    const uint64_t n4 = a.n >> 2;
    const uint64_t stride = (uint64_t)gridDim.x * kBlock;
    uint64_t j = (uint64_t)blockIdx.x * kBlock + threadIdx.x;
    constexpr int U = 2;
    for (; j + (U - 1) * stride < n4; j += U * stride) {
        float4 gv[U], ev[U], wv[U];
#pragma unroll
        for (int u = 0; u < U; ++u) gv[u] = ld_stream(g + 4 * (j + u * stride));
        if (EF) {
#pragma unroll
            for (int u = 0; u < U; ++u) ev[u] = ld_stream(e + 4 * (j + u * stride));
        }
#pragma unroll
        for (int u = 0; u < U; ++u) wv[u] = ld_stream(w + 4 * (j + u * stride));
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const float4 v = EF ? add4(gv[u], ev[u]) : gv[u];
            float4 gh, rs;
            decode4<EF>(v, c, gh, rs);
            if (STORE) st_stream(e + 4 * (j + u * stride), rs);
            st_stream(w + 4 * (j + u * stride),
                      make_float4(fmaf(neg_lr, gh.x, wv[u].x), fmaf(neg_lr, gh.y, wv[u].y),
                                  fmaf(neg_lr, gh.z, wv[u].z), fmaf(neg_lr, gh.w, wv[u].w)));
        }
    }
    for (; j < n4; j += stride) {
        float4 v = ld_stream(g + 4 * j);
        if (EF) v = add4(v, ld_stream(e + 4 * j));
        const float4 wv = ld_stream(w + 4 * j);
        float4 gh, rs;
        decode4<EF>(v, c, gh, rs);
        if (STORE) st_stream(e + 4 * j, rs);
        st_stream(w + 4 * j, make_float4(fmaf(neg_lr, gh.x, wv.x), fmaf(neg_lr, gh.y, wv.y),
                                         fmaf(neg_lr, gh.z, wv.z), fmaf(neg_lr, gh.w, wv.w)));
    }
    if (blockIdx.x == 0 && threadIdx.x < 4) {
        const uint64_t i = (n4 << 2) + threadIdx.x;
        if (i < a.n) {
            float v = ld_stream1(g + i);
            if (EF) v += ld_stream1(e + i);
            float gh, rs;
            decode1<EF>(v, c, gh, rs);
            if (STORE) st_stream1(e + i, rs);
            w[i] = fmaf(neg_lr, gh, w[i]);
        }
    }
}

// General path: any 4-byte alignment, both weight layouts, scalar accesses.
// Shared w: grid = (G, 1), the thread walks the workers; replicas: grid = (G, P).
template <bool EF, bool STORE>
__global__ void __launch_bounds__(kBlock) k_decode_scalar(DecodeArgs a)
{
    const float m_pos = __ldg(a.global_means), m_neg = __ldg(a.global_means + 1);
    const uint64_t stride = (uint64_t)gridDim.x * kBlock;
    const bool shared = a.w_stride == 0;
    const uint32_t p_lo = shared ? 0 : blockIdx.y, p_hi = shared ? a.P : blockIdx.y + 1;
    const float scale = shared ? -a.lr / (float)a.P : -a.lr;
    for (uint64_t i = (uint64_t)blockIdx.x * kBlock + threadIdx.x; i < a.n; i += stride) {
        float sum = 0.f;
        for (uint32_t p = p_lo; p < p_hi; ++p) {
            const WorkerConst c = worker_const<EF>(a, p, m_pos, m_neg);
            float v = ld_stream1(a.grad + (int64_t)p * a.grad_stride + i);
            if (EF) v += ld_stream1(a.err + (int64_t)p * a.err_stride + i);
            float gh, rs;
            decode1<EF>(v, c, gh, rs);
            sum += gh;
            if (STORE) st_stream1(a.err + (int64_t)p * a.err_stride + i, rs);
        }
        float *wp = a.w + (int64_t)p_lo * a.w_stride + i;
        *wp = fmaf(scale, sum, *wp);
    }
}

} // namespace a2sgd
