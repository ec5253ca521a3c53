// Segment-list (multi-tensor) forms of K1 and K3: the model is a list of
// tensors living in separate allocations, as a training framework holds them,
// and is reduced to the same two whole-model means per worker (Section 4.3:
// the two averages are taken over all gradients of the model) without first
// being copied into one flat vector.
//
// The flat index space of each tensor is cut into tiles of kSegTile elements;
// a table built once per plan maps tile -> (tensor, offset).  A tile never
// crosses a tensor boundary, so all addressing inside a tile is one base
// pointer plus a contiguous range.  Tensors whose pointers are all 32-byte
// aligned take 256-bit accesses; any other 4-byte alignment takes coalesced
// scalar accesses (decided per tensor on the host, uniform per CTA).
// Like a2sgd_kernels.cuh this header has no include guard: it is compiled once per kernel variant,
// after a2sgd_kernels.cuh, into the namespace A2SGD_NS.
namespace A2SGD_NS {

constexpr int kSegVW = 8;
constexpr uint32_t kSegTile = kBlock * kSegVW; // 2048 elements per tile
constexpr uint32_t kSegFlagVec = 1u;

struct __align__(16) SegTile {
    uint32_t seg;    // tensor index
    uint32_t flags;  // kSegFlagVec: every pointer of this tensor is 32-byte aligned
    uint64_t offset; // first element of the tile inside the tensor
};

// First tile and access flags of a tensor; one entry per tensor plus an end marker.  The decode
// kernel finds its tensor by scanning this small table (L1-resident: every CTA reads the same
// entries) instead of reading a per-tile descriptor, which would be a fresh L2 access in front of
// every CTA's data loads.
struct __align__(16) SegStart {
    uint64_t first_tile;
    uint64_t numel;
    uint32_t flags;
    uint32_t first_job; // per-tensor-means variant: this tensor's fold jobs are [first_job, next entry's first_job)
    uint32_t pad[2];
};

// Per-tensor-means variant: the per-tile partial sums of a tensor are added in two levels so that a
// tensor of tens of thousands of tiles is not folded by a single CTA.  A job is a run of at most
// kFoldJobTiles consecutive tiles of one tensor.
constexpr uint32_t kFoldJobTiles = 1024;
struct __align__(16) FoldJob {
    uint64_t first_tile;
    uint32_t count;
    uint32_t seg;
};
constexpr uint32_t kSegScanMax = 4096; // tensors up to which the decode kernel scans SegStart (else: tile table)

struct SegTables {
    const SegTile *tiles;
    const SegStart *starts; // [S + 1] or nullptr (S > kSegScanMax)
    uint64_t n_tiles;
    const uint64_t *numel;      // [S]
    const float *const *grad;   // [P][S] device pointers, worker-major
    float *const *err;          // [P][S] or nullptr
    float *const *w;            // [S] (shared) or [P][S] (replicas)
    uint32_t S;
    uint32_t w_replicated;
    const float *lr_per_segment; // [S] device, or nullptr: one learning rate for the whole model
    // per-tensor-means variant only (plan-owned scratch)
    const SegStart *all_starts;        // [S + 1], always present
    const FoldJob *fold_jobs;          // [n_jobs]
    uint32_t n_jobs;
    Partial *tile_partials;            // [P][n_tiles]
    Partial *job_partials;             // [P][n_jobs]
    float *seg_local_means;            // [S][P][2]
    unsigned long long *seg_counts;    // [S][P]
    float *seg_global_means;           // [S][2]
};

// An entry of a pointer table through the read-only (L1-cached) path: the tables are small and every
// CTA of a tensor reads the same entries, while the data streams bypass L1.
template <typename T>
__device__ __forceinline__ T *ld_ptr(T *const *slot)
{
    return reinterpret_cast<T *>(__ldg(reinterpret_cast<const unsigned long long *>(slot)));
}

// K1 over a segment list.  grid = (G, P); CTA x walks tiles x, x + G, ...
// PER_TENSOR: every tensor keeps its own pair of means, so the sums are not carried across tiles:
// each tile's (S+, S-, n+) goes to its own slot of t.tile_partials and k_fold_segments adds the
// slots of a tensor in tile order afterwards.
template <bool EF, bool PER_TENSOR = false>
__global__ void __launch_bounds__(kBlock) k_encode_segments(EncodeArgs a, SegTables t)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    __shared__ double sh_d[2][kWarps];
    __shared__ unsigned long long sh_n[kWarps];
    __shared__ int sh_flag;
    const uint32_t p = blockIdx.y;
    Acc acc;
    for (uint64_t tile = blockIdx.x; tile < t.n_tiles; tile += gridDim.x) {
        if (PER_TENSOR) acc = Acc();
        const SegTile d = t.tiles[tile];
        if (d.seg >= t.S) {                     // only reachable with a corrupt table
            span_ok(d.seg, 1, t.S);
            continue;
        }
        const uint64_t n_s = t.numel[d.seg];
        if (!span_ok(d.offset, 1, n_s)) continue;
        const float *__restrict__ g = t.grad[(uint64_t)p * t.S + d.seg];
        const float *__restrict__ e = EF ? t.err[(uint64_t)p * t.S + d.seg] : nullptr;
        float sp = 0.f, sn = 0.f;
        unsigned bits;
        const uint64_t i = d.offset + (uint64_t)threadIdx.x * kSegVW;
        if ((d.flags & kSegFlagVec) && i + kSegVW <= n_s) {
            Vec<kSegVW> v = ld_vec<kSegVW>(g + i);
            if (EF) v = add_vec<kSegVW>(v, ld_vec<kSegVW>(e + i));
            split_vec<kSegVW>(v, sp, sn, acc.n_pos, bits);
        } else if (d.flags & kSegFlagVec) {
            // the tensor's last, partial vector
            float ps[kSegVW], ns[kSegVW];
#pragma unroll
            for (int k = 0; k < kSegVW; ++k) {
                ps[k] = ns[k] = 0.f;
                if (i + k < n_s) {
                    float v = ld_stream1(g + i + k);
                    if (EF) v += ld_stream1(e + i + k);
                    unsigned b;
                    split1(v, ps[k], ns[k], acc.n_pos, b);
                }
            }
            sp = tree_sum<kSegVW>(ps);
            sn = tree_sum<kSegVW>(ns);
        } else {
            float ps[kSegVW], ns[kSegVW];
#pragma unroll
            for (int k = 0; k < kSegVW; ++k) {
                const uint64_t idx = d.offset + (uint64_t)k * kBlock + threadIdx.x;
                ps[k] = ns[k] = 0.f;
                if (idx < n_s) {
                    float v = ld_stream1(g + idx);
                    if (EF) v += ld_stream1(e + idx);
                    unsigned b;
                    split1(v, ps[k], ns[k], acc.n_pos, b);
                }
            }
            sp = tree_sum<kSegVW>(ps);
            sn = tree_sum<kSegVW>(ns);
        }
        acc.s_pos += (double)sp;
        acc.s_neg += (double)sn;
        if (PER_TENSOR) {
            double s_pos = acc.s_pos, s_neg = acc.s_neg;
            unsigned long long n_pos = acc.n_pos;
            block_reduce(s_pos, s_neg, n_pos, sh_d, sh_n);
            if (threadIdx.x == 0) {
                Partial &slot = t.tile_partials[(uint64_t)p * t.n_tiles + tile];
                slot.s_pos = s_pos;
                slot.s_neg = s_neg;
                slot.n_pos = n_pos;
            }
        }
    }
    if (PER_TENSOR) return;
    double s_pos = acc.s_pos, s_neg = acc.s_neg;
    unsigned long long n_pos = acc.n_pos;
    block_reduce(s_pos, s_neg, n_pos, sh_d, sh_n);
    finish_worker(a, p, s_pos, s_neg, n_pos, sh_d, sh_n, &sh_flag);
}

// Per-tensor-means variant, between K1 and K3, first level: block (j, p) adds the tile slots of job j
// of worker p in tile order (thread t takes slots t, t + 256, ...; fixed tree above).  grid = (jobs, P).
static __global__ void __launch_bounds__(kBlock) k_fold_jobs(SegTables t)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    __shared__ double sh_d[2][kWarps];
    __shared__ unsigned long long sh_n[kWarps];
    const FoldJob job = t.fold_jobs[blockIdx.x];
    const uint32_t p = blockIdx.y;
    const Partial *slot = t.tile_partials + (uint64_t)p * t.n_tiles + job.first_tile;
    double s_pos = 0.0, s_neg = 0.0;
    unsigned long long n_pos = 0;
    for (uint32_t i = threadIdx.x; i < job.count; i += kBlock) {
        s_pos += __ldcg(&slot[i].s_pos);
        s_neg += __ldcg(&slot[i].s_neg);
        n_pos += __ldcg(&slot[i].n_pos);
    }
    block_reduce(s_pos, s_neg, n_pos, sh_d, sh_n);
    if (threadIdx.x == 0) {
        Partial &out = t.job_partials[(uint64_t)p * t.n_jobs + blockIdx.x];
        out.s_pos = s_pos;
        out.s_neg = s_neg;
        out.n_pos = n_pos;
    }
}

// Second level: block s adds the job sums of tensor s in job order, one worker after the other,
// writes that tensor's local means and counts, and averages them over the workers in worker order
// (Algorithm 1 line 5, once per tensor).  grid = S.
static __global__ void __launch_bounds__(kBlock) k_fold_segments(SegTables t, uint32_t P, int *status)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    __shared__ double sh_d[2][kWarps];
    __shared__ unsigned long long sh_n[kWarps];
    const uint32_t sg = blockIdx.x;
    const uint32_t first = t.all_starts[sg].first_job, last = t.all_starts[sg + 1].first_job;
    const uint64_t numel = t.all_starts[sg].numel;
    double g_pos = 0.0, g_neg = 0.0; // thread 0: sums of the workers' means
    for (uint32_t p = 0; p < P; ++p) {
        const Partial *slot = t.job_partials + (uint64_t)p * t.n_jobs;
        double s_pos = 0.0, s_neg = 0.0;
        unsigned long long n_pos = 0;
        for (uint32_t i = first + threadIdx.x; i < last; i += kBlock) {
            s_pos += __ldcg(&slot[i].s_pos);
            s_neg += __ldcg(&slot[i].s_neg);
            n_pos += __ldcg(&slot[i].n_pos);
        }
        block_reduce(s_pos, s_neg, n_pos, sh_d, sh_n);
        if (threadIdx.x == 0) {
            const unsigned long long n_neg = numel - n_pos;
            const float mu_pos = n_pos ? (float)(s_pos / (double)n_pos) : 0.0f;
            const float mu_neg = n_neg ? (float)(s_neg / (double)n_neg) : 0.0f;
            if (!isfinite(s_pos) || !isfinite(s_neg)) atomicCAS(status, kDevOk, kDevNonFinite);
            t.seg_local_means[((uint64_t)sg * P + p) * 2 + 0] = mu_pos;
            t.seg_local_means[((uint64_t)sg * P + p) * 2 + 1] = mu_neg;
            t.seg_counts[(uint64_t)sg * P + p] = n_pos;
            g_pos += (double)mu_pos;
            g_neg += (double)mu_neg;
        }
    }
    if (threadIdx.x == 0) {
        t.seg_global_means[2 * sg + 0] = (float)(g_pos / (double)P);
        t.seg_global_means[2 * sg + 1] = (float)(g_neg / (double)P);
    }
}

// K3 over a segment list: one tile per CTA.  PT > 0: compile-time worker count.  PER_TENSOR: the
// means of the tile's own tensor (written by k_fold_segments) instead of the whole-model means.
template <bool EF, bool STORE, int PT, bool PER_TENSOR = false>
__global__ void __launch_bounds__(kBlock) k_decode_segments(DecodeArgs a, SegTables t)
{
    pdl_wait_prior_grid();
    pdl_release_next_grid();
    __shared__ WorkerConst sh_c[PT > 0 ? 1 : kMaxP];
    const uint32_t P = PT > 0 ? PT : a.P;
    float m_pos = 0.f, m_neg = 0.f;
    if (!PER_TENSOR) {
        m_pos = __ldg(a.global_means);
        m_neg = __ldg(a.global_means + 1);
    }
    const bool repl = t.w_replicated != 0;
    if (PT == 0 && !PER_TENSOR) {
        for (uint32_t p = threadIdx.x; p < P; p += kBlock) sh_c[p] = worker_const<EF>(a, p, m_pos, m_neg);
        __syncthreads();
    }
    __shared__ SegTile sh_tile;
    __shared__ uint64_t sh_numel;
    for (uint64_t tile = blockIdx.x; tile < t.n_tiles; tile += gridDim.x) {
        SegTile d;
        uint64_t n_s;
        if (t.starts) {
            for (uint32_t sg = threadIdx.x; sg < t.S; sg += kBlock) {
                const uint64_t lo = __ldg(&t.starts[sg].first_tile), hi = __ldg(&t.starts[sg + 1].first_tile);
                if (tile >= lo && tile < hi) {
                    sh_tile = SegTile{sg, __ldg(&t.starts[sg].flags), (tile - lo) * kSegTile};
                    sh_numel = __ldg(&t.starts[sg].numel);
                }
            }
            __syncthreads();
            d = sh_tile;
            n_s = sh_numel;
            if (tile + gridDim.x < t.n_tiles) __syncthreads(); // the slots are rewritten in the next trip
        } else {
            d = t.tiles[tile];
            n_s = __ldg(t.numel + d.seg);
        }
        if (!span_ok(d.offset, 1, n_s)) continue; // the tile starts inside its tensor
        if (PER_TENSOR) {
            m_pos = __ldcg(t.seg_global_means + 2 * d.seg);
            m_neg = __ldcg(t.seg_global_means + 2 * d.seg + 1);
            a.local_means = t.seg_local_means + (uint64_t)d.seg * P * 2; // this tensor's P pairs
            if (PT == 0) {
                __syncthreads();
                for (uint32_t p = threadIdx.x; p < P; p += kBlock) sh_c[p] = worker_const<EF>(a, p, m_pos, m_neg);
                __syncthreads();
            }
        }
        const uint64_t i = d.offset + (uint64_t)threadIdx.x * kSegVW;
        // layer-wise learning rates (e.g. LARS, which the paper uses for VGG-16): one per tensor
        const float lr = t.lr_per_segment ? __ldg(t.lr_per_segment + d.seg) : a.lr;
        const float scale = repl ? -lr : -lr / (float)P;
        if ((d.flags & kSegFlagVec) && i + kSegVW <= n_s) {
            if (PT > 0 && !repl) {
                // workers in batches of four, as in the flat kernel: all loads of a batch are issued
                // before its first store, and the register count stays low enough for two CTAs per SM
                constexpr int PP = PT > 0 ? PT : 1;
                constexpr int PB = PP < 4 ? PP : 4;
                // every pointer of the tile is fetched before the first data access: a pointer load
                // placed after a store could not be moved above it
                const float *gp[PP];
                float *ep[PP];
                float *wp = ld_ptr(t.w + d.seg) + i;
#pragma unroll
                for (int p = 0; p < PP; ++p) gp[p] = ld_ptr(t.grad + (uint64_t)p * t.S + d.seg) + i;
                if (EF || STORE) {
#pragma unroll
                    for (int p = 0; p < PP; ++p) ep[p] = ld_ptr(t.err + (uint64_t)p * t.S + d.seg) + i;
                }
                const Vec<kSegVW> wv = ld_vec<kSegVW>(wp);
                Vec<kSegVW> sum = zero_vec<kSegVW>();
#pragma unroll
                for (int p0 = 0; p0 < PP; p0 += PB) {
                    Vec<kSegVW> gv[PB], ev[PB];
#pragma unroll
                    for (int q = 0; q < PB; ++q) gv[q] = ld_vec<kSegVW>(gp[p0 + q]);
                    if (EF) {
#pragma unroll
                        for (int q = 0; q < PB; ++q) ev[q] = ld_vec<kSegVW>(ep[p0 + q]);
                    }
#pragma unroll
                    for (int q = 0; q < PB; ++q) {
                        const Vec<kSegVW> v = EF ? add_vec<kSegVW>(gv[q], ev[q]) : gv[q];
                        Vec<kSegVW> gh, rs;
                        decode_vec<EF, kSegVW>(v, worker_const<EF>(a, p0 + q, m_pos, m_neg), gh, rs);
                        sum = add_vec<kSegVW>(sum, gh);
                        if (STORE) st_vec<kSegVW>(ep[p0 + q], rs);
                    }
                }
                st_vec<kSegVW>(wp, axpy_vec<kSegVW>(scale, sum, wv));
            } else {
                Vec<kSegVW> sum = zero_vec<kSegVW>();
                for (uint32_t p = 0; p < P; ++p) {
                    const WorkerConst c = PT > 0 ? worker_const<EF>(a, p, m_pos, m_neg) : sh_c[p];
                    Vec<kSegVW> v = ld_vec<kSegVW>(t.grad[(uint64_t)p * t.S + d.seg] + i);
                    if (EF) v = add_vec<kSegVW>(v, ld_vec<kSegVW>(t.err[(uint64_t)p * t.S + d.seg] + i));
                    Vec<kSegVW> gh, rs;
                    decode_vec<EF, kSegVW>(v, c, gh, rs);
                    if (STORE) st_vec<kSegVW>(t.err[(uint64_t)p * t.S + d.seg] + i, rs);
                    if (repl) {
                        float *wp = t.w[(uint64_t)p * t.S + d.seg] + i;
                        st_vec<kSegVW>(wp, axpy_vec<kSegVW>(scale, gh, ld_vec<kSegVW>(wp)));
                    } else {
                        sum = add_vec<kSegVW>(sum, gh);
                    }
                }
                if (!repl) {
                    float *wp = t.w[d.seg] + i;
                    st_vec<kSegVW>(wp, axpy_vec<kSegVW>(scale, sum, ld_vec<kSegVW>(wp)));
                }
            }
        } else {
            // scalar elements: a misaligned tensor (coalesced, stride kBlock) or a tensor's last partial vector
            const bool vec_tail = (d.flags & kSegFlagVec) != 0;
#pragma unroll 1
            for (int k = 0; k < kSegVW; ++k) {
                const uint64_t idx = vec_tail ? i + k : d.offset + (uint64_t)k * kBlock + threadIdx.x;
                if (idx >= n_s) continue;
                float sum = 0.f;
                for (uint32_t p = 0; p < P; ++p) {
                    const WorkerConst c = PT > 0 ? worker_const<EF>(a, p, m_pos, m_neg) : sh_c[p];
                    float v = ld_stream1(t.grad[(uint64_t)p * t.S + d.seg] + idx);
                    if (EF) v += ld_stream1(t.err[(uint64_t)p * t.S + d.seg] + idx);
                    float gh, rs;
                    decode1<EF>(v, c, gh, rs);
                    if (STORE) st_stream1(t.err[(uint64_t)p * t.S + d.seg] + idx, rs);
                    if (repl) {
                        float *wp = t.w[(uint64_t)p * t.S + d.seg] + idx;
                        st1(wp, fmaf(scale, gh, ld1(wp)));
                    } else {
                        sum += gh;
                    }
                }
                if (!repl) {
                    float *wp = t.w[d.seg] + idx;
                    st1(wp, fmaf(scale, sum, ld1(wp)));
                }
            }
        }
    }
}

} // namespace A2SGD_NS
