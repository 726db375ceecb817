/*
 * det_linear_test.h -- test-only exports of the det_linear library.  Nothing here changes the
 * arithmetic: the hooks select among kernels and launch geometries that must all produce the same
 * bits (tile sizes, warp counts, pipeline depth and grid size are numerically inert: supplement C
 * on rule R2), and create streams restricted to a subset of the SMs so that tests can check that
 * the output does not depend on the SM count (rule R3: the result may depend on neither the device,
 * the number of SMs nor the way the grid is scheduled).  The paper has no counterpart for these functions.
 */
#ifndef DET_LINEAR_TEST_H
#define DET_LINEAR_TEST_H

#include "det_linear.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Force the kernel a plan uses: 0 generic, 1 decode pipeline, 2 prefill tile kernel, -1 automatic.
 * DET_ERR_INVALID_ARG when the kernel cannot serve the plan's bucket. */
DET_API det_status_t det_test_plan_force_kernel(det_linear_plan_t* plan, int kernel);

/* Limit the number of thread blocks the plan's persistent kernels launch (0 = automatic, i.e.
 * derived from the SM count).  Only the schedule changes. */
DET_API det_status_t det_test_plan_set_max_blocks(det_linear_plan_t* plan, int max_blocks);

/* Select a tile configuration variant of the plan's kernel (0 = automatic). Only the schedule
 * changes. DET_ERR_INVALID_ARG if the variant does not exist for this plan. */
DET_API det_status_t det_test_plan_set_variant(det_linear_plan_t* plan, int variant);

/*
 * Host-side fault injection: make the nth device allocation the library attempts from now on (1 = the
 * next one) fail once with an out-of-memory error, without touching the device; 0 switches the hook
 * off.  det_linear_plan* must then return NULL with det_last_status() == DET_ERR_ALLOC and free
 * whatever it had already allocated.  Process-wide, not thread-safe: tests only.
 */
DET_API void det_test_fail_next_alloc(int nth);

/*
 * det_attention_decode spreads the keys of one (batch, KV head) row over a cluster of 1, 2, 4, 8 or 16 thread
 * blocks, chosen from the shape and the SM count (schedule only: every choice gives the same bits).  This
 * forces the choice for the calls that follow (capped by the number of 256-key segments of the row);
 * 0 = automatic again.  Process-wide: tests only.
 */
DET_API void det_test_attention_set_split(int blocks_per_row);
/* The cluster size det_attention_decode would use for this shape on a device with sm_count SMs, and the dynamic
 * shared memory of one block for it (*smem_bytes_out, may be NULL; above 232448 the call would be refused).
 * Host arithmetic only: touches no device.  0 on bad arguments. */
DET_API int det_test_attention_schedule(int64_t B, int64_t Hq, int64_t Hkv, int64_t T, int64_t D, int sm_count,
                                        uint64_t* smem_bytes_out);

/*
 * Bound of one device-side wait for the kernels launched through this plan (default 2 s), and flags:
 * bit 0 (value 1) is a deliberate stall: thread block 0 of the decode kernel (of the TMA-fed prefill
 * kernel likewise) never requests the activations of its first stage, so the wait for that stage runs
 * into the bound.  The
 * kernel then records the timeout in the plan's status word, drains and returns (no trap, no endless
 * loop; the other blocks finish normally), and det_linear_plan_check reports DET_ERR_DEVICE_TIMEOUT.
 * The output of such a run is undefined.  Bit 1 (value 2) makes a prefill plan with several K segments fold them
 * with the second (combine) launch instead of inside the kernel: same bits, another schedule.
 * Reset with (2000000000, 0).
 */
DET_API det_status_t det_test_plan_set_wait(det_linear_plan_t* plan, uint64_t wait_limit_ns, int flags);

/*
 * Create a CUDA green context holding (at least) `sm_count` SMs of the current device and a
 * stream on it.  *stream_out receives a cudaStream_t usable with det_linear_run; *handle_out an
 * opaque handle for det_test_green_stream_destroy; *sm_granted the number of SMs in the
 * partition.  DET_ERR_CUDA if the driver refuses (the caller should then fall back to other
 * invariance checks).
 */
DET_API det_status_t det_test_green_stream_create(int sm_count, void** stream_out, void** handle_out,
                                          int* sm_granted);
DET_API void det_test_green_stream_destroy(void* handle);

/*
 * Calibration for the benchmark's rooflines (these compute nothing of the method).
 * det_test_measure_fma_peak: FP32 multiply-add issue peak of the CUDA cores in TFLOP/s, measured
 * with a register-only loop of scalar fma.rn.f32 (packed = 0) or fma.rn.f32x2 (packed = 1); packed = 2
 * times the prefill kernel's multiply loop alone (8 x 8 outputs per thread from resident shared-memory tiles,
 * no staging, no barriers): the ceiling of that loop.
 * det_test_measure_read_bandwidth: read-only streaming rate in GB/s over `bytes` of device memory
 * at `buf` (16-byte aligned, at least 1 MiB; use a buffer much larger than L2).
 * Both run on the default stream and synchronise.
 */
DET_API det_status_t det_test_measure_fma_peak(int packed, double* tflops_out);
DET_API det_status_t det_test_measure_read_bandwidth(const void* buf, size_t bytes, double* gbs_out);

/*
 * Negative control for rule R3 (the paper's split-K ablation in supplement C: no split, ordered combine, atomic combine): the decode
 * order's segment partials for a requested split S_req (segments of whole 256-element blocks, as in
 * the library), combined with atomicAdd onto y (pre-set to the bias, or zero) in arrival order --
 * the scheme the rule forbids.  The output is close to det_linear_run's but its bits depend on grid
 * scheduling and may change from run to run.  BF16 weights, device pointers, layouts as for
 * det_linear_run; enqueued on `stream`.  Nothing in the library uses it.
 */
DET_API det_status_t det_test_linear_atomic_splitk(int64_t M, int64_t N, int64_t K, int32_t S_req, const float* x,
                                                   const uint16_t* W, const float* b, float* y, void* stream);

/*
 * Glue for the multi-layer test harness (no part of the method): dst[m, j] = src[m, j] * c for the first
 * `cols` columns of a row-major device matrix with row pitch ld_src; dst is [M, cols], contiguous.
 * One IEEE multiplication per element.  Enqueued on `stream` with programmatic dependent launch, so a
 * chain det_linear_run -> glue -> det_linear_run keeps overlapping kernel prologues.
 */
DET_API det_status_t det_test_scale_cols(const float* src, int64_t ld_src, float* dst, int64_t M, int64_t cols, float c,
                                         void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DET_LINEAR_TEST_H */
