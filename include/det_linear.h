/*
 * det_linear.h -- C ABI of the deterministic fused-upcast linear layer for NVIDIA B200 (sm_100a).
 *
 *     y = x * up(W_bf16)^T (+ b)                                            (paper Eq. 2)
 *
 * FP32 activations, BF16 weights read once from HBM and widened to FP32 in registers, IEEE-754
 * FP32 fused multiply-add accumulation on the CUDA cores (design rule R1: never tensor cores), in
 * a reduction order that is a pure function of the problem shape (M, N, K) (rules R2-R4): the bits
 * of y do not depend on the SM count, the grid, the stream, co-scheduled work or, inside the
 * decode bucket (M <= 64), on M.
 *
 * Reduction order, version 2 (what "the same bits" means):
 *   bucket   = decode if M <= 64, else prefill                                  (R2, R4)
 *   decode : V = 4, L = 32, P = 1        prefill: V = 1, L = 1, P = 1 (strictly ascending k)
 *   K is cut into S contiguous segments of seg_len elements (a multiple of 256; only the last
 *   may be short); S is shape-pure and, for decode, independent of M: 2 segments for weight
 *   matrices below 16384 rows (1 if K <= 256), no split above                      (R3, R4)
 *   inside a segment, chunks of V*L elements are walked in ascending k; "lane" l owns the V
 *   consecutive elements c + l*V + j; element j is accumulated with one fmaf into the lane's
 *   sub-chain j mod P, starting from +0.0f; elements beyond the segment end are skipped;
 *   the L*P leaves are summed by a balanced tree, adjacent leaves first;
 *   segment sums are added in ascending segment order (R3, no atomics);
 *   the bias, when given, is added last with a single rounding                    (Eq. 2).
 *
 * All functions return a status or NULL and never throw, abort or synchronise the device unless
 * stated.  Pointers named "device" must be device memory of the current CUDA device; "host" means
 * ordinary (preferably pinned) host memory.  The library requires compute capability 10.x; on any
 * other device plan creation fails with DET_ERR_ARCH (there is no fallback path).
 */
#ifndef DET_LINEAR_H
#define DET_LINEAR_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define DET_API __attribute__((visibility("default")))
#else
#define DET_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct det_linear_plan det_linear_plan_t;   /* opaque, owned by the library */

typedef enum {
    DET_OK = 0,
    DET_ERR_INVALID_ARG = 1,        /* NULL pointer, non-positive size, buffer too small          */
    DET_ERR_UNSUPPORTED_SHAPE = 2,  /* a dimension exceeds what the kernels index (see below)     */
    DET_ERR_ALIGNMENT = 3,          /* a buffer misses the alignment an entry point without a generic path needs */
    DET_ERR_ALLOC = 4,              /* device or host allocation failed                           */
    DET_ERR_CUDA = 5,               /* a CUDA call failed; det_last_error() has the message       */
    DET_ERR_DEVICE_TIMEOUT = 6,     /* a kernel gave up a bounded wait (see det_linear_plan_check)*/
    DET_ERR_ARCH = 7                /* current device is not sm_100                               */
} det_status_t;

/* Storage format of the weight matrix.  Every format widens exactly to FP32 in registers (Eq. 2's
 * up()); the reduction order does not depend on it.  The paper's kernels take 16-bit weights and
 * its seeded probe covers BF16 and FP32 weights. */
typedef enum {
    DET_WEIGHT_BF16 = 0,            /* bfloat16 bit patterns, 2 bytes per element (default)        */
    DET_WEIGHT_FP16 = 1,            /* IEEE binary16 bit patterns, 2 bytes per element             */
    DET_WEIGHT_FP32 = 2             /* IEEE binary32, 4 bytes per element (no widening needed)     */
} det_weight_format_t;

/* Order parameters of a shape; filled by det_linear_plan_params / det_linear_plan_get_params. */
typedef struct {
    int64_t M, N, K;
    int32_t bucket;          /* 0 = decode (M <= 64), 1 = prefill                                   */
    int32_t V, L, P;         /* order family parameters (see the header comment)                    */
    int64_t seg_len;         /* K elements per segment                                              */
    int32_t S;               /* number of segments, = ceil(K / seg_len)                             */
    int32_t order_version;   /* version of the order definition, 2                                  */
    int32_t kernel;          /* 0 generic, 1 decode (TMA pipeline), 2 prefill tile kernel           */
    int32_t weight_format;   /* det_weight_format_t of the plan (0 = BF16 for det_linear_plan_params)    */
    uint64_t workspace_bytes;/* split-K partials of the prefill bucket: 4*S*M*N bytes when S > 1; decode: 0 */
} det_linear_params_t;

/*
 * Shape -> order parameters (rule R2: the configuration is a constant chosen by the shape alone;
 * R3: the split is shape-pure; R4: decode parameters never read M).  Pure host
 * function: touches no device, allocates nothing.  M, N, K >= 1 and each < 2^31, M*N < 2^40.
 * The `kernel` field reports the kernel for 16-byte aligned buffers.
 */
DET_API det_status_t det_linear_plan_params(int64_t M, int64_t N, int64_t K, det_linear_params_t* out);

/*
 * Create a plan for y[M,N] = x[M,K] * up(W[N,K])^T (+ b[N]) on the current device.  Allocates a
 * status word and, in the prefill bucket when S > 1, the split-K partials workspace (device); the
 * decode bucket folds its segments inside the kernel and needs none.  Returns NULL on failure
 * (det_last_error(), det_last_status()).
 * A prefill plan also asks for 4 * K * roundup(M, 4) bytes in which every run
 * writes x transposed for its TMA-fed kernel (schedule only; reported as "activation_workspace_bytes"
 * by det_linear_plan_describe, not in workspace_bytes).  If that allocation fails the plan is still
 * created and runs the register-staged kernel, which computes the same bits.
 * A plan may be used from one stream at a time: its workspace is not re-entrant; make one plan
 * per stream for concurrent use.  Destroy with det_linear_plan_destroy.
 */
DET_API det_linear_plan_t* det_linear_plan(int64_t M, int64_t N, int64_t K);

/* The same for a weight matrix stored as FP16 or FP32 (wfmt: det_weight_format_t).  The order
 * parameters are those of det_linear_plan_params: they depend on the shape only. */
DET_API det_linear_plan_t* det_linear_plan_w(int64_t M, int64_t N, int64_t K, int32_t wfmt);

/*
 * Plan for ONE COLUMN SHARD of a layer: outputs n_begin .. n_begin + n_count - 1 of y[M,N] (tensor
 * parallelism over the output dimension).  Every output depends on one weight row only, and the
 * order parameters are those of the whole layer (M, N, K) -- the split factor is evaluated on the
 * global N -- so a shard's outputs carry the same bits as the same columns computed by
 * det_linear_plan(M, N, K) on one GPU, whatever the number of shards.  The paper runs on a single
 * GPU; this is the column-parallel extension its reduction order allows without any change.
 * With such a plan det_linear_run_w takes
 *   W : the shard's rows, [n_count, K] row-major (element (0,0) = weight row n_begin of the layer)
 *   b : the shard's n_count bias values, or NULL
 *   y : address of the shard's first column inside a row-major matrix with row pitch `ldy` floats
 *       (ldy = N writes in place into the full [M,N] output, ldy = n_count gives a compact block)
 * The fast kernels need y 16-byte aligned (and ldy % 4 == 0 in the prefill bucket); otherwise the
 * generic kernels run.  Requires 0 <= n_begin, 1 <= n_count, n_begin + n_count <= N, ldy >= n_count.
 * det_linear_plan_params / get_params report the layer's N; workspace_bytes is the shard's.
 * det_linear_run_host* reject shard plans.  The all-gather of the shards is the caller's.
 */
DET_API det_linear_plan_t* det_linear_plan_shard(int64_t M, int64_t N, int64_t K, int64_t n_begin, int64_t n_count,
                                                 int64_t ldy, int32_t wfmt);

/*
 * Enqueue the computation on `stream` (a cudaStream_t; NULL = the legacy default stream) and
 * return without synchronising.  Eq. 2 with the order above; the segment sums are folded in
 * ascending order (R3) -- inside the kernel in the decode bucket, by a second fixed-order pass in the
 * prefill bucket -- never by atomics.
 *   x : device, FP32, [M,K] row-major (row pitch K)
 *   W : device, BF16 bit patterns, [N,K] row-major (row pitch K): one weight row per output column
 *   b : device, FP32, [N], or NULL for no bias (then no final add happens at all)
 *   y : device, FP32, [M,N] row-major; overwritten; must not overlap the inputs
 * Buffers stay owned by the caller and must stay valid until the stream reaches the end of the
 * work.  W and b are parameters: they must be complete before the kernel that precedes this call in
 * the stream STARTS (the decode kernel is launched with programmatic dependent launch and requests
 * its first weight tiles, and reads b, before it waits for that kernel to finish; only x and y are
 * touched after the wait).  If W or b were just written on the same stream -- a dequantise or copy
 * kernel, a device-side random fill -- put another kernel or a synchronisation in between.  The fast kernels need K % 8 == 0 and 16-byte aligned x, W, y; anything else runs a
 * slower generic kernel that produces the same bits.  Errors: DET_ERR_INVALID_ARG for NULL
 * arguments, DET_ERR_CUDA if a launch fails.  Nothing is launched when an error is returned.
 */
DET_API det_status_t det_linear_run(const det_linear_plan_t* plan, const float* x, const uint16_t* W,
                            const float* b, float* y, void* stream);

/* det_linear_run for any weight format: W points to [N,K] row-major elements of the plan's format
 * (det_linear_run itself accepts BF16 and FP16 plans; an FP32 plan needs this entry point).  The fast
 * kernels need 16-byte aligned buffers and a 16-byte row pitch (K % 8 == 0 for 16-bit weights,
 * K % 4 == 0 for FP32 weights). */
DET_API det_status_t det_linear_run_w(const det_linear_plan_t* plan, const float* x, const void* W,
                              const float* b, float* y, void* stream);

/*
 * End-to-end variant with HOST activations: copies x (host, [M,K]) to a plan-owned device buffer,
 * runs the same kernels, copies y back to y_host (host, [M,N]) and waits for the stream.  W (in the
 * plan's weight format) and b stay device-resident (they are the model's parameters).  The staging buffers are allocated on
 * first use.  Synchronises `stream` before returning.
 */
DET_API det_status_t det_linear_run_host(det_linear_plan_t* plan, const float* x_host, const void* W,
                                 const float* b, float* y_host, void* stream);

/*
 * The same without the final wait: the copies and kernels are only enqueued; y_host is valid once
 * the caller has synchronised `stream`.  x_host must stay unchanged and y_host untouched until then;
 * pinned host memory is needed for the copies to be asynchronous.  One call in flight per plan.
 */
DET_API det_status_t det_linear_run_host_async(det_linear_plan_t* plan, const float* x_host, const void* W,
                                       const float* b, float* y_host, void* stream);

/*
 * Optional: time the plan's candidate thread-block tilings on the caller's buffers and pin the
 * fastest one in the plan.  Only the schedule is chosen: tile sizes, warp counts and ring depth
 * do not enter the reduction order (supplement C on rule R2 calls them numerically inert), every
 * candidate produces the same bits, and the order parameters (V, L, P, S) remain the pure function
 * of the shape that rule R2 asks for -- this is not the numeric autotuning the rule forbids.
 * Without this call a cost model picks the tiling from the shape and the SM count.
 * Plans of the decode bucket only; for other plans the call does nothing and reports variant 0.
 * Runs every candidate six times on `stream` (CUDA events; a 192 MiB scratch buffer, allocated
 * and freed inside the call, is read through L2 before each timed run so that the weights come
 * from HBM) and synchronises; y holds the layer's result afterwards.  Do not call during stream capture.
 * *variant_out (may be NULL): the pinned candidate's number; *best_us_out (may be NULL): its time.
 */
DET_API det_status_t det_linear_plan_tune(det_linear_plan_t* plan, const float* x, const void* W, const float* b,
                                          float* y, void* stream, int32_t* variant_out, float* best_us_out);

/*
 * Synchronise `stream` and report whether any kernel launched through this plan gave up a bounded
 * device-side wait (every wait on a TMA completion barrier is limited; on expiry the kernel
 * records the fact and returns instead of spinning).  DET_OK, DET_ERR_DEVICE_TIMEOUT or
 * DET_ERR_CUDA.  The record is cleared by the call.  After a kernel gave up, the outputs of that run are
 * undefined and the plan must pass through this call (which also resets the plan's split-K bookkeeping)
 * before it is used again.
 */
DET_API det_status_t det_linear_plan_check(det_linear_plan_t* plan, void* stream);

/* Copy the plan's order parameters to *out. */
DET_API det_status_t det_linear_plan_get_params(const det_linear_plan_t* plan, det_linear_params_t* out);

/* Write a JSON description (bucket, V, L, P, S, seg_len, order_version, kernel, workspace_bytes, the shard
 * and, schedule only: for the decode kernel the tiling in use on the current device with its resident
 * blocks per SM, for the prefill kernel the tile, how it is fed ("tma" or "registers") and the bytes of
 * the activation workspace)
 * to buf (at most n bytes including the terminator).  DET_ERR_INVALID_ARG if it does not fit. */
DET_API det_status_t det_linear_plan_describe(const det_linear_plan_t* plan, char* buf, size_t n);

/* Free the plan and everything it owns.  NULL is ignored.  The caller must make sure no work
 * using the plan is still running. */
DET_API void det_linear_plan_destroy(det_linear_plan_t* plan);

/*
 * Greedy argmax per row with the LOWER index winning a tie (the tie rule the paper states for
 * greedy decoding): idx[m] = min{ n : y[m,n] = max_n y[m,n] }.  -0.0 and +0.0 compare equal; a
 * row containing NaN returns the index of its first NaN.
 *   y : device FP32 [M,N] row-major;  idx : device int32 [M].  1 <= N < 2^31, M >= 1.
 * Enqueued on `stream`, no synchronisation.  Exact (comparisons only), so it is order-free.
 */
DET_API det_status_t det_argmax_rows(const float* y, int64_t M, int64_t N, int32_t* idx, void* stream);

/*
 * Fixed-order RMSNorm per row: y[m,h] = (x[m,h] * r[m]) * g[h] with r = 1 / sqrt(ss / H + eps).
 * An extension, not one of the paper's kernels: the paper keeps vendor FP32 RMSNorm and names the
 * reductions outside the linear layers as the residual channel of cross-run divergence.  The row's
 * sum of squares ss is reduced in the decode order of this header (chunks of 128 ascending, lane l
 * owns 4 consecutive elements, one fmaf(x, x, acc) per element from +0.0f, elements beyond H
 * skipped, 32 lane sums added by the adjacent-first tree); then one IEEE binary32 operation per step:
 * mean = ss / float(H), t = mean + eps, root = sqrt(t), r = 1 / root, y = (x * r) * g.  The bits do
 * not depend on M, the grid, the stream or the SM count.
 *   x : device FP32 [M,H] row-major;  g : device FP32 [H];  y : device FP32 [M,H], must not overlap x
 *   eps >= 0;  1 <= M, H < 2^31.  16-byte aligned buffers with H % 4 == 0 take vector loads.
 * Enqueued on `stream`, no synchronisation, no allocation.
 */
DET_API det_status_t det_rmsnorm(const float* x, const float* g, float eps, int64_t M, int64_t H, float* y,
                                 void* stream);

/*
 * Fixed-order decode attention: o[b,h,:] = softmax_j(q[b,h,:] . k[b,h',j,:] * scale) . v[b,h',:,:] for one
 * query row per (batch, head) against T cached keys and values, h' = h / (Hq / Hkv) (grouped-query heads).
 * An extension, not one of the paper's kernels: the paper keeps vendor attention and names fixed-order
 * attention as the outstanding source of residual divergence between GPU architectures.  Every step is
 * one IEEE binary32 operation in an order fixed by (T, D) alone:
 *   s_j = dot(q, k_j) * scale, the dot product in the decode lane order of this header over D (chunks of
 *         128 ascending, lane l owns 4 consecutive elements, one fmaf per element from +0.0f, elements
 *         beyond D skipped, adjacent-first 32-lane tree), then one multiply;
 *   m   = max_j s_j;   e_j = exp_det(s_j - m), exp_det a fixed sequence of binary32 operations (range
 *         reduction by ln 2 in two pieces, degree-7 Taylor polynomial by Horner's rule with fmaf, exact
 *         scaling by 2^n; within 2 ulp of the real exponential; +0 below -104);
 *   l   = sum_j e_j in the lane order over j (chunks of 128 keys, lane l owns 4 consecutive keys, one add
 *         per key from +0.0f, adjacent-first tree);
 *   o_d = (sum over 256-key segments, ascending, of the chain a = fmaf(e_j, v_j[d], a) from +0.0f) / l.
 * The bits do not depend on B, the grid, the stream or the SM count.
 *   q : device FP32 [B, Hq, D];  k, v : device FP32 [B, Hkv, T, D];  o : device FP32 [B, Hq, D]; all
 *   row-major, contiguous and 16-byte aligned (DET_ERR_ALIGNMENT otherwise).
 *   Hq / Hkv in {1, 2, 4, 8}; D a multiple of 4, at most 256; the scores and segment sums of a (batch,
 *   KV head) live in shared memory, which limits T (about 9000 keys at Hq / Hkv = 4, D = 128):
 *   DET_ERR_UNSUPPORTED_SHAPE with a message beyond that.
 * Enqueued on `stream`, no synchronisation, no allocation.
 */
DET_API det_status_t det_attention_decode(const float* q, const float* k, const float* v, float scale, int64_t B,
                                          int64_t Hq, int64_t Hkv, int64_t T, int64_t D, float* o, void* stream);

/*
 * The same computation for callers that cannot allocate (the paper has no counterpart for this
 * entry point).  A host that owns all device memory through its own pool or arena, a plugin that
 * may not allocate after initialisation, or a latency-critical loop that cannot afford the
 * implicit synchronisation of an allocation can use this call instead of det_linear_plan +
 * det_linear_run: it calls no cudaMalloc / cudaFree and no allocating library routine, and keeps no
 * plan.  Inputs and output are passed as for det_linear_run (device pointers, same layouts, b may
 * be NULL); the result has the same bits.
 *
 * The split-K partials (needed only in the prefill bucket, M > 64, when the shape splits K, i.e.
 * S > 1: 4*S*M*N bytes) live in a 4 MiB array built into the library image, present on every GPU that loads the library until the
 * process exits.  A shape that needs more is rejected with DET_ERR_UNSUPPORTED_SHAPE and a message
 * that names both sizes; nothing is launched then.  All calls share that one array and it keeps the
 * last call's contents (nothing in it needs clearing: each call overwrites what it reads), so two
 * calls whose GPU work overlaps -- different streams, or different host threads -- race on it:
 * issue them on one stream or order them yourself.
 *
 * The first call on each device looks up the array's device address (with that device current);
 * make that first call before starting any stream capture.  The address is kept for the life of the
 * process: after a cudaDeviceReset the library must be reloaded before this entry point is used again.  The kernels are the library's generic
 * ones (any shape and alignment, not tuned for speed).  Enqueues on `stream`, no synchronisation.
 */
DET_API det_status_t det_linear_run_noalloc(int64_t M, int64_t N, int64_t K, const float* x, const uint16_t* W,
                                            const float* b, float* y, void* stream);

/* Message of the last error on the calling thread ("" if none).  Never NULL. */
DET_API const char* det_last_error(void);

/* Status behind the last det_linear_plan* call of the calling thread: DET_OK if it returned a plan,
 * otherwise why it returned NULL (DET_ERR_INVALID_ARG, DET_ERR_UNSUPPORTED_SHAPE, DET_ERR_ARCH,
 * DET_ERR_ALLOC, DET_ERR_CUDA). */
DET_API det_status_t det_last_status(void);

/* Version of the reduction-order definition implemented by this library (currently 2). */
DET_API int det_order_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DET_LINEAR_H */
