/*
 * liba2sgd — the per-worker gradient path of A2SGD (two-level gradient
 * averaging) as CUDA kernels for sm_100a behind a plain C ABI.
 *
 * What the path computes (Section 3.1, Eq. 2 and Algorithm 1 of the paper).
 * For every one of P data-parallel workers holding an n-element fp32 vector v:
 *   pos(v)_i = 1 if v_i >= 0 else 0,  neg(v) = 1 - pos(v)
 *   mu_pos(v) = mean of the entries v_i >= 0      (0 for an empty group)
 *   mu_neg(v) = mean of |v_i| over entries v_i < 0 (0 for an empty group)
 * The P pairs (mu_pos, mu_neg) — 64 bits per worker — are averaged, unweighted,
 * into the global pair (m_pos, m_neg) (Algorithm 1 line 5).  Each worker then
 * rebuilds a dense gradient from the two global means, updates its local
 * error vector and applies w <- w - lr * g_hat (Algorithm 1 lines 4, 6, 7).
 *
 * Two modes, chosen at a2sgd_create:
 *   A2SGD_MODE_EF    error feedback carried between iterations:
 *                    v = g + e,  g_hat = pos(v)*m_pos - neg(v)*m_neg,
 *                    e <- v - g_hat        (so e_new + g_hat == g + e_old).
 *   A2SGD_MODE_ALG1  Algorithm 1 as printed (same-iteration add-back, Eq. 13):
 *                    v = g,  eps = g - (pos*mu_pos^p - neg*mu_neg^p),
 *                    g_hat = eps + pos*m_pos - neg*m_neg; eps is stored to
 *                    `err` only when the caller passes a non-NULL err.
 *
 * The P workers are simulated as P buffers on one GPU: worker p's vector is
 * at `base + p*stride` (stride in ELEMENTS, 64-bit).  Weights are either one
 * replica per worker (w_stride >= n, the layout of Algorithm 1) or one shared
 * vector (w_stride == 0), which receives the worker-mean of the reconstructed
 * gradients, w <- w - (lr/P) * sum_p g_hat^p — the mean of the P replicas.
 *
 * Pointers.  Unless an argument is marked HOST it is DEVICE memory on the
 * context's device, owned by the caller, at least 4-byte aligned.  The
 * library never allocates, frees or retains these buffers (a segment plan
 * retains the pointers it was given, see a2sgd_segments_create).  Any
 * alignment that is a multiple of 4 bytes is computed correctly: rows that
 * are 32-byte aligned with strides that are multiples of 8 elements take the
 * 256-bit kernels, 16-byte / 4 elements the 128-bit ones, anything else the
 * scalar kernels.  For full speed start every row on a 128-byte boundary
 * (stride = n rounded up to 32 elements).  `grad` is never written.
 *
 * Execution.  Every call enqueues its kernels on `stream` (a cudaStream_t
 * passed as void*, NULL = default stream) and returns without waiting, except
 * a2sgd_read_stats and a2sgd_step_host, which synchronise `stream`.
 * Conditions seen by the host (bad arguments) return a negative status and
 * launch nothing.  Conditions seen on the device (non-finite sums, a bounded
 * wait that ran out) are latched in a status word read by a2sgd_read_stats.
 * Results are bitwise reproducible for a fixed (n, P, strides' alignment,
 * device, build): no floating-point atomics, fixed-order combines.
 * A context owns only small scratch (per-CTA partial sums, 2P+2 means, P
 * counts, tickets, barrier words, status); use one context per stream; a
 * context is not thread-safe.  Kernels are launched with programmatic stream
 * serialisation and wait for the preceding grid before their first memory
 * access, so ordinary stream order is what the caller observes.
 * Limits: 1 <= n < 2^40, 1 <= P <= 1024.
 */
#ifndef A2SGD_H_
#define A2SGD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct a2sgd_ctx a2sgd_ctx;

enum a2sgd_status {
    A2SGD_OK = 0,
    A2SGD_ERR_ARG = -1,       /* NULL pointer, n or P out of range, stride < n, bad flag */
    A2SGD_ERR_ALIGN = -2,     /* a float pointer that is not 4-byte aligned */
    A2SGD_ERR_CUDA = -3,      /* a CUDA runtime call failed */
    A2SGD_ERR_TIMEOUT = -4,   /* a bounded device-side wait ran out (latched in the status word).  A CTA that
                                 gives up writes nothing, and the barrier is left shut once one has, but a CTA
                                 may still give up after the others went on: after this status w and err of
                                 that step are undefined — restore them from a copy */
    A2SGD_ERR_NONFINITE = -5, /* a group sum was NaN or Inf (latched in the status word) */
    A2SGD_ERR_NOMEM = -6,     /* scratch allocation failed */
    A2SGD_ERR_TOO_LARGE = -7, /* n*P exceeds what the single-launch path can hold on chip (A2SGD_FORCE_COOPERATIVE),
                                 or P > A2SGD_NOALLOC_MAX_P in a2sgd_encode_noalloc (its fixed scratch) */
    A2SGD_ERR_BOUNDS = -8     /* A2SGD_DEBUG_CHECKS: a kernel computed an access outside the live elements of
                                 the buffers it was given; the access was skipped (latched in the status word) */
};

enum a2sgd_flags {
    A2SGD_MODE_EF = 0,                /* default */
    A2SGD_MODE_ALG1 = 1,
    A2SGD_FORCE_TWO_PASS = 1 << 4,    /* a2sgd_step never takes the single-launch path */
    A2SGD_FORCE_COOPERATIVE = 1 << 5, /* a2sgd_step takes the single-launch path whenever (n, P) fits it — v in
                                         registers, or g, e, w within 70 % of L2 — and returns
                                         A2SGD_ERR_TOO_LARGE otherwise.  Without this flag the single launch is
                                         used only where it measured faster: v in registers with one CTA per SM
                                         (n*P up to about 1.2 M elements), or one worker with v in registers. */
    A2SGD_DEFERRED_RESIDUAL = 1 << 7, /* EF mode only, opt-in: between steps the caller's error buffer holds the
                                         compensated vector v of the last step instead of the residual
                                         e = v - g_hat(v); the subtraction is done one step later, with the
                                         means the context kept.  Same fp32 operations, so w and (after
                                         a2sgd_materialize_err) err are bit-identical to the default, but a
                                         step moves (12P + 8 + P/4) bytes per model element instead of
                                         (20P + 8).  Needs 32-byte aligned rows with strides that are multiples
                                         of 8 (A2SGD_ERR_ALIGN otherwise), the same error buffer at every
                                         step, and only a2sgd_step / a2sgd_step_host / a2sgd_dense_sync /
                                         a2sgd_materialize_err on this context.  The context also owns a sign
                                         mask of P*n/8 bytes.  Which kernel a step launches depends on
                                         host-side state (does the buffer hold v yet?), so a captured step
                                         must not be replayed across the first step or a materialise call. */
    A2SGD_CHECK_POINTERS = 1 << 8,    /* every call that takes device buffers first asks the runtime whether each
                                         one is device (or managed) memory usable from the context's device and
                                         returns A2SGD_ERR_ARG otherwise, before anything is launched: a host
                                         pointer handed to a kernel would fault the GPU.  A segment plan checks
                                         every tensor pointer once, in a2sgd_segments_create.  Costs about a
                                         microsecond per pointer per call; off by default. */
    A2SGD_DEBUG_CHECKS = 1 << 10,     /* the stand-in for a memory checker where none can be run: while a call
                                         of this context is in flight, every access its kernels make to grad, err,
                                         w, the momentum buffer and the packed mask is first checked, on the
                                         device, against the extents the call was given (inside the n live
                                         elements of one row); an access that is not is skipped — loads return 0 —
                                         and A2SGD_ERR_BOUNDS is latched for a2sgd_read_stats.  Nothing traps or
                                         faults.  For segment lists the check is on tile and tensor indices
                                         instead of addresses.  The extents live in one descriptor per device, so
                                         calls of a checking context must not overlap other calls of the library
                                         on the same device (different streams or threads), and they cannot be
                                         captured into a CUDA graph (A2SGD_ERR_CUDA during capture).  Several
                                         times slower; off by default. */
    A2SGD_TEST_SHRINK_EXTENTS = 1 << 11, /* test hook for A2SGD_DEBUG_CHECKS: the extents recorded for a call are
                                            one element per row short, so the checked kernels skip every access
                                            that touches a row's last element and latch A2SGD_ERR_BOUNDS — the
                                            check is seen to fire without any access ever leaving a buffer */
    A2SGD_TEST_BARRIER_NEVER_OPENS = 1 << 9 /* test hook: the single-launch path waits for one arrival more
                                               than its grid has, with a ~0.2 ms limit, so every CTA gives up,
                                               writes nothing and A2SGD_ERR_TIMEOUT is latched */
};

/* Creates a context for vectors of n elements and P workers on `device`
 * (made current for the duration of each call, then restored).  Allocates
 * the scratch listed above with cudaMalloc.  *out is NULL on failure. */
int a2sgd_create(a2sgd_ctx **out, uint64_t n, uint32_t P, int device, uint32_t flags);

/* Frees the scratch.  NULL is accepted. */
int a2sgd_destroy(a2sgd_ctx *ctx);

/* Algorithm 1 line 3 (Section 3.1): the two local means of every worker.
 *   grad        [P] vectors of n floats, worker stride grad_stride (>= n)
 *   err         EF: the retained error, same layout (required).  ALG1: ignored, may be NULL
 *   local_means out, [P][2] floats = {mu_pos, mu_neg}: exactly 8 bytes per worker
 *   pos_counts  out, [P] uint64 = #{i : v_i >= 0}, may be NULL
 *   pos_mask    out, [P][ceil(n/32)] uint32, bit b of word j = pos of element 32*j+b,
 *               unused high bits of the last word 0; may be NULL */
int a2sgd_encode(a2sgd_ctx *ctx, const float *grad, int64_t grad_stride,
                 const float *err, int64_t err_stride, float *local_means,
                 uint64_t *pos_counts, uint32_t *pos_mask, void *stream);

/* Algorithm 1 line 5, with the P workers on one device: the unweighted mean
 * of the P pairs, summed in worker order in fp64, rounded once to fp32.
 *   local_means  in,  [P][2]      global_means  out, [2] = {m_pos, m_neg} */
int a2sgd_global_average(a2sgd_ctx *ctx, const float *local_means,
                         float *global_means, void *stream);

/* Algorithm 1 line 5 with one worker per GPU, for an exchange done as the paper does it, by
 * Allreduce: a collective between the GPUs has formed the SUMS of the two local means over all
 * workers (in fp64, so that the order in which the collective adds cannot matter at fp32
 * precision); this call divides by the worker count in fp64 and rounds once — the "average" of
 * Allreduce(average), inside the library.
 *   sums  in, DEVICE, [2] doubles = {sum_p mu_pos^p, sum_p mu_neg^p};  workers >= 1
 *   global_means  out, [2] */
int a2sgd_global_average_from_sums(a2sgd_ctx *ctx, const double *sums, uint32_t workers,
                                   float *global_means, void *stream);

/* Algorithm 1 lines 4, 6 and 7 fused: reconstruct, update the residual,
 * apply the SGD step.  Reads grad, err (EF) and w once, writes err and w once.
 *   w            in/out; w_stride == 0: one shared vector, else >= n: one per worker
 *   err          EF: in/out (required).  ALG1: out (eps), may be NULL
 *   local_means  in, [P][2]; read in ALG1 mode only (may be NULL in EF)
 *   global_means in, [2]
 *   lr           learning rate of this step */
int a2sgd_decode_update(a2sgd_ctx *ctx, float *w, int64_t w_stride,
                        const float *grad, int64_t grad_stride,
                        float *err, int64_t err_stride,
                        const float *local_means, const float *global_means,
                        float lr, void *stream);

/* One whole loop body of Algorithm 1 (lines 3-7) for all P workers: encode,
 * average the 2P scalars, decode/update.  The means stay in the context and
 * can be read back with a2sgd_read_stats.  Two launches in general; a single
 * cooperative launch (v kept in registers between the two phases, or, with
 * A2SGD_FORCE_COOPERATIVE, re-read from L2) for small n*P, see a2sgd_flags. */
int a2sgd_step(a2sgd_ctx *ctx, float *w, int64_t w_stride,
               const float *grad, int64_t grad_stride,
               float *err, int64_t err_stride, float lr, void *stream);

/* Algorithm 1 lines 4, 6 and 7 with the optimiser the paper's experiments put on top of line 7:
 * SGD with momentum and weight decay (Section 4.1 and Table 1 list the training policies;
 * Algorithm 1 line 7 itself prints the plain step and has no counterpart for the two terms).  The
 * method compresses the gradient only (lines 3-6), so both terms act on the reconstructed gradient:
 *     u = g_hat + weight_decay * w;   mom <- beta * mom + u;   w <- w - lr * mom
 * (heavy ball, no dampening, no Nesterov look-ahead, decay folded into the gradient).
 *   mom          in/out, DEVICE, same layout as w: one vector when w is shared (mom_stride == 0,
 *                it sees the worker-mean of g_hat), one per worker otherwise (mom_stride >= n);
 *                zero it before the first step
 *   beta         0 <= beta < 1;  weight_decay >= 0 (A2SGD_ERR_ARG otherwise)
 * Everything else as a2sgd_decode_update.  beta = weight_decay = 0 gives the same w as
 * a2sgd_decode_update and leaves g_hat in mom.  One streaming pass: (12P + 16) bytes per model
 * element for a shared w, 28P for replicas. */
int a2sgd_decode_update_momentum(a2sgd_ctx *ctx, float *w, int64_t w_stride, float *mom, int64_t mom_stride,
                                 const float *grad, int64_t grad_stride, float *err, int64_t err_stride,
                                 const float *local_means, const float *global_means, float lr,
                                 float beta, float weight_decay, void *stream);

/* a2sgd_step (Algorithm 1 lines 3-7 for all P workers) with the momentum / weight-decay update
 * above in place of the plain SGD step.  Always two launches.  Not available on contexts
 * created with A2SGD_DEFERRED_RESIDUAL. */
int a2sgd_step_momentum(a2sgd_ctx *ctx, float *w, int64_t w_stride, float *mom, int64_t mom_stride,
                        const float *grad, int64_t grad_stride, float *err, int64_t err_stride,
                        float lr, float beta, float weight_decay, void *stream);

/* a2sgd_step with the fresh gradients stored as bfloat16 (Section 1 of the paper names the
 * combination with quantisation as a natural extension; a bfloat16 gradient is the common case
 * of a mixed-precision backward pass).  grad: [P] vectors of n bfloat16 values (raw uint16 bit
 * patterns), worker stride grad_stride in ELEMENTS.  Widening bfloat16 to fp32 is exact, so the
 * result equals a2sgd_step on the widened gradients; err and w stay fp32.  Traffic drops from
 * (20P + 8) to (16P + 8) bytes per model element.  Always two launches.  The fast path needs
 * 16-byte aligned gradient rows with strides that are multiples of 8 elements and 32-byte
 * aligned err / w rows; anything else takes the scalar kernels. */
int a2sgd_step_bf16(a2sgd_ctx *ctx, float *w, int64_t w_stride,
                    const uint16_t *grad, int64_t grad_stride,
                    float *err, int64_t err_stride, float lr, void *stream);

/* The same with IEEE half-precision (fp16) gradients; widening is exact here too. */
int a2sgd_step_f16(a2sgd_ctx *ctx, float *w, int64_t w_stride,
                   const uint16_t *grad, int64_t grad_stride,
                   float *err, int64_t err_stride, float lr, void *stream);

/* For contexts created with A2SGD_DEFERRED_RESIDUAL: rewrites the error buffer in place from the
 * compensated vector v it holds after a step to the true residual e = v - g_hat(v) of that step
 * (one pass, 8 bytes per worker-element), e.g. before a checkpoint or before handing the buffer
 * to other code.  The next a2sgd_step then treats it as a residual again.  No-op when the buffer
 * already holds a residual (before the first step, or right after this call). */
int a2sgd_materialize_err(a2sgd_ctx *ctx, float *err, int64_t err_stride, void *stream);

/* Algorithm 1 lines 9-10: the dense synchronisation that follows the last compressed iteration
 * (Eq. 1 for one step).  The workers' gradients are averaged element-wise, summed in worker
 * order, and applied: w <- w - lr * (1/P) * sum_p grad^p.  With w_stride == 0 the one shared w is
 * updated; with w_stride >= n every replica receives the same averaged update (which is what
 * brings drifted replicas back in step).  No error buffer is involved.  One streaming pass:
 * (4P + 8) bytes per model element for a shared w. */
int a2sgd_dense_sync(a2sgd_ctx *ctx, float *w, int64_t w_stride,
                     const float *grad, int64_t grad_stride, float lr, void *stream);

/* Algorithm 1 lines 9-10 with one worker per GPU: the dense Allreduce between the GPUs has
 * already formed grad_sum, the element-wise SUM of all workers' gradients; this call applies
 * w <- w - lr * grad_sum / workers (the division that makes the all-reduce an average is done
 * here, not by the caller).  Contexts with P == 1 only (this rank's one worker).
 *   grad_sum  in, DEVICE, [n];  workers >= 1 */
int a2sgd_dense_sync_reduced(a2sgd_ctx *ctx, float *w, const float *grad_sum, uint32_t workers, float lr,
                             void *stream);

/* Segment lists: the model as S separate tensors (the way a training framework holds its
 * parameters and gradients) instead of one flat vector.  The S tensors are treated as the
 * concatenation they would form: ONE pair of means per worker over the whole model (Section 4.3:
 * the two averages are taken over all gradients of the model), the same
 * results as a2sgd_step on the flattened copy, without making that copy.
 *
 * a2sgd_segments_create records the layout once (device tables owned by the plan):
 *   S           number of tensors; sum of numel[] must equal the context's n
 *   numel       HOST, [S] element counts (each >= 1)
 *   grad        HOST array of [P][S] DEVICE pointers, worker-major: grad[p*S + s]
 *   err         HOST array of [P][S] DEVICE pointers; required in EF mode; in ALG1 mode NULL
 *               (eps is not stored) or the buffers that receive eps
 *   w           HOST array of DEVICE pointers: [S] (one shared model) or, when w_replicated
 *               is non-zero, [P][S] (one replica per worker)
 * Tensors may have any 4-byte alignment; a tensor all of whose pointers are 32-byte aligned
 * takes the 256-bit path.  The plan keeps the pointers: the tensors must stay where they are
 * while the plan is used.  Destroy the plan before its context. */
typedef struct a2sgd_segments a2sgd_segments;
int a2sgd_segments_create(a2sgd_ctx *ctx, uint32_t S, const uint64_t *numel,
                          const float *const *grad, float *const *err, float *const *w,
                          int w_replicated, a2sgd_segments **out);
int a2sgd_segments_destroy(a2sgd_segments *plan);

/* One whole loop body of Algorithm 1 (lines 3-7) over a segment list; two launches.  Means and
 * counts are left in the context for a2sgd_read_stats, as with a2sgd_step. */
int a2sgd_step_segments(a2sgd_ctx *ctx, a2sgd_segments *plan, float lr, void *stream);

/* a2sgd_step_segments with one learning rate per tensor: lr_per_segment is a DEVICE array of S
 * floats.  This is the hook for layer-wise learning-rate policies such as LARS (listed in the
 * paper's experimental setup for VGG-16); computing those rates is the caller's business. */
int a2sgd_step_segments_lr(a2sgd_ctx *ctx, a2sgd_segments *plan, const float *lr_per_segment, void *stream);

/* The per-tensor variant of a2sgd_step_segments: every tensor of the list is compressed on its own,
 * as if Algorithm 1 (lines 3-7) were run once per tensor — tensor s has its own pair of local means
 * per worker, its own pair of global means (the unweighted average over the workers), and is
 * reconstructed from those.  The payload a worker would exchange grows from 2 to 2S floats: this is
 * NOT the method's whole-model reading (Section 4.3 takes the two averages over all gradients of the
 * model) but the granularity a per-tensor communication layer works at; results equal a2sgd_step
 * called separately on every tensor.  Four launches (encode per tile, two-level fold per tensor,
 * decode/update).  The first call on a plan allocates the variant's scratch (24 bytes per worker
 * and 2048-element tile, plus the per-tensor means).  lr_per_segment: DEVICE [S] or NULL.
 * a2sgd_read_segment_stats synchronises `stream` and copies the per-tensor results to HOST memory:
 *   local_means_host [S][P][2], global_means_host [S][2], pos_counts_host [S][P]; any may be NULL. */
int a2sgd_step_segments_per_tensor(a2sgd_ctx *ctx, a2sgd_segments *plan, float lr, const float *lr_per_segment,
                                   void *stream);
int a2sgd_read_segment_stats(a2sgd_ctx *ctx, a2sgd_segments *plan, float *local_means_host,
                             float *global_means_host, uint64_t *pos_counts_host, void *stream);

/* The two stages of a2sgd_step_segments as separate calls, mirroring a2sgd_encode and
 * a2sgd_decode_update (Algorithm 1 line 3, and lines 4, 6, 7) for a segment list; the 2P scalars
 * are averaged in between with a2sgd_global_average (line 5).
 *   local_means   DEVICE [P][2] (out of the first call, in of the second: read in ALG1 mode only)
 *   pos_counts    DEVICE [P], may be NULL;   global_means  DEVICE [2]
 *   lr_per_segment  DEVICE [S] or NULL (then `lr` applies to every tensor) */
int a2sgd_encode_segments(a2sgd_ctx *ctx, a2sgd_segments *plan, float *local_means, uint64_t *pos_counts,
                          void *stream);
int a2sgd_decode_update_segments(a2sgd_ctx *ctx, a2sgd_segments *plan, const float *local_means,
                                 const float *global_means, float lr, const float *lr_per_segment, void *stream);

/* a2sgd_step for a caller whose fresh gradients sit in HOST memory (pinned
 * memory makes the copies asynchronous): copies grad_host -> grad_staging
 * worker by worker, runs the step, copies the 2P local and 2 global means
 * to means_host and synchronises `stream`.
 *   grad_host     HOST, [P] vectors of n floats, stride grad_host_stride
 *   grad_staging  device, caller-owned, [P] vectors with stride grad_stride
 *   means_host    HOST, out, [2P + 2] floats: local pairs then the global pair */
int a2sgd_step_host(a2sgd_ctx *ctx, float *w, int64_t w_stride,
                    const float *grad_host, int64_t grad_host_stride,
                    float *grad_staging, int64_t grad_stride,
                    float *err, int64_t err_stride, float lr,
                    float *means_host, void *stream);

/* Synchronises `stream`, then copies the context's latest means and counts
 * (written by a2sgd_step / a2sgd_encode) to HOST memory and returns the
 * latched device status (A2SGD_OK, A2SGD_ERR_TIMEOUT or A2SGD_ERR_NONFINITE)
 * in *device_status, clearing the latch.  Any out pointer may be NULL.
 *   local_means_host [P][2], global_means_host [2], pos_counts_host [P] */
int a2sgd_read_stats(a2sgd_ctx *ctx, float *local_means_host,
                     float *global_means_host, uint64_t *pos_counts_host,
                     int *device_status, void *stream);

/* Launch geometry of the context's kernels, for benchmarks and reports:
 * out[0] = CTAs of the encode launch, out[1] = CTAs of the decode launch,
 * out[2] = threads per CTA, out[3] = 1 if a2sgd_step takes the single-launch
 * path for this (n, P), out[4] = SM count.  HOST pointer. */
int a2sgd_launch_info(a2sgd_ctx *ctx, int64_t w_stride, uint32_t out[5]);

/* The encode step (two local means per worker, see a2sgd_encode) for callers that must not
 * allocate device memory.  The paper has no counterpart to this entry point: it exists for
 * integration reasons only.  Typical callers: code running inside a framework that has given
 * the whole GPU to its own caching allocator (a raw cudaMalloc there fails or fragments the
 * pool), loops that cannot afford the device-wide synchronisation a cudaMalloc implies, and
 * plug-ins bound by a "nothing is allocated after start-up" rule.  It takes no context: the
 * reduction scratch is a fixed 64 KiB array inside the library image (every GPU that loads the
 * library holds it until the process exits), and the call itself performs no cudaMalloc,
 * cudaFree or other allocating call.
 *   n, P         as in a2sgd_create; P <= A2SGD_NOALLOC_MAX_P, else A2SGD_ERR_TOO_LARGE
 *                (the fixed scratch has ticket slots for that many workers; n is not limited
 *                beyond n < 2^40 because the grid, not n, sizes the partial sums)
 *   mode         A2SGD_MODE_EF or A2SGD_MODE_ALG1
 *   grad, err    device, as in a2sgd_encode (err required in EF mode)
 *   local_means  device, out, [P][2];  pos_counts  device, out, [P], may be NULL
 * Runs on the CURRENT device.  The first call on each device also looks up the device address of
 * the scratch array; make that first call before any stream capture begins.  All calls on a
 * device share the one scratch array: the tickets are cleared at the start of every call, but two
 * calls whose kernels overlap on the GPU (different streams, different threads) race on it and
 * give wrong means — serialise them.  No packed mask output and no latched device status here;
 * results are identical to a2sgd_encode up to the summation order of a differently sized grid. */
#define A2SGD_NOALLOC_MAX_P 64
int a2sgd_encode_noalloc(uint64_t n, uint32_t P, uint32_t mode, const float *grad, int64_t grad_stride,
                         const float *err, int64_t err_stride, float *local_means, uint64_t *pos_counts,
                         void *stream);

/* Static, never NULL. */
const char *a2sgd_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* A2SGD_H_ */
