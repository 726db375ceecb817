// C ABI of libdet_linear: argument checks, plan life cycle, kernel dispatch.  Host code only.
#include "internal.h"
#include "det_linear_test.h"
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

namespace detlin {

static thread_local char g_err[512] = "";
static thread_local int g_last_status = DET_OK;   // status behind a NULL plan (det_last_status)

void set_error(const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
}

static det_status_t cuda_fail(const char* what, cudaError_t e)
{
    set_error("%s: %s", what, cudaGetErrorString(e));
    return DET_ERR_CUDA;
}

// Driver entry points are looked up at run time so that the library loads on machines without
// a driver (the build check and the symbol test run on CPU-only hosts).
template <typename Fn>
static Fn driver_fn(const char* name)
{
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint(name, &fn, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
        return nullptr;
    return reinterpret_cast<Fn>(fn);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D row-major tensor [rows, cols] of `elem_bytes`-wide elements, box [box_rows, box_cols].
static bool encode_2d(CUtensorMap* map, CUtensorMapDataType dt, int elem_bytes, const void* base, uint64_t rows,
                      uint64_t cols, uint32_t box_rows, uint32_t box_cols, CUtensorMapL2promotion promo,
                      CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_NONE)
{
    static EncodeTiledFn encode = driver_fn<EncodeTiledFn>("cuTensorMapEncodeTiled");
    if (!encode) { set_error("cuTensorMapEncodeTiled is not available from the driver"); return false; }
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * (uint64_t)elem_bytes};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        swizzle, promo, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled failed with CUresult %d", (int)r); return false; }
    return true;
}

// Device allocation with the test hook of det_test_fail_next_alloc: the next `skip`-th call fails once
// with cudaErrorMemoryAllocation without touching the device.
static int g_fail_alloc_countdown = 0;          // 0 = off; n = the n-th allocation from now fails
static cudaError_t device_alloc(void** p, size_t bytes)
{
    if (g_fail_alloc_countdown > 0 && --g_fail_alloc_countdown == 0) { *p = nullptr; return cudaErrorMemoryAllocation; }
    return cudaMalloc(p, bytes);
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static det_status_t run_device(det_linear_plan_t* plan, const float* x, const void* W, const float* b, float* y,
                               cudaStream_t stream)
{
    const det_linear_params_t& p = plan->prm;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != plan->device) {
        set_error("run: the plan belongs to device %d but device %d is current", plan->device, dev);
        return DET_ERR_INVALID_ARG;
    }
    LaunchArgs a{};
    a.x = x; a.W = W; a.b = b; a.y = y;
    a.wfmt = p.weight_format;
    a.partials = plan->partials;
    // Prefill with 2 .. 4 segments: the block that completes a tile folds it (measured 0.5 - 3 % faster than the second
    // launch); with more segments the fold of a tile by one block is a longer serial tail than the combine launch
    // (1 - 5 % slower), so that keeps the second pass.  Test flag 2 forces the second pass.  Same bits either way.
    a.tile_counters = ((plan->test_flags & 2) || p.S > 4) ? nullptr : plan->tile_counters;
    a.M = p.M; a.N = plan->n_count; a.K = p.K;            // the kernels see the shard; the order is the layer's
    a.ldy = plan->ldy;
    a.seg_len = p.seg_len; a.S = p.S;
    a.stream = stream;
    a.status = plan->status;
    a.sm_count = plan->sm_count;
    a.max_blocks = plan->max_blocks;
    a.variant = plan->variant;

    int kernel = plan->forced_kernel >= 0 ? plan->forced_kernel : p.kernel;
    const int64_t k_align = p.weight_format == DET_WEIGHT_FP32 ? 4 : 8;     // 16-byte row pitch of W (x: K % 4)
    const bool fast_ok = (p.K % k_align == 0) && (p.K % 4 == 0) && p.K <= (1 << 30) && p.N <= (1 << 30) && aligned16(x) && aligned16(W) && aligned16(y);
    if (!fast_ok) kernel = kKernelGeneric;

    a.wait_limit_ns = plan->wait_limit_ns;
    a.test_flags = plan->test_flags;

    cudaError_t e = cudaSuccess;
    if (kernel == kKernelDecode) {
        // the tiling is a function of the plan and the device: chosen once, then cached
        if (plan->decode_cfg_variant != plan->variant) {
            if (!decode_config_for(p.M, plan->n_count, p.K, p.S, p.weight_format, plan->variant, &plan->decode_cfg)) {
                set_error("run: no decode configuration for this shape/variant");
                return DET_ERR_INVALID_ARG;
            }
            plan->decode_cfg_variant = plan->variant;
        }
        const DecodeConfig& cfg = plan->decode_cfg;
        if (plan->map_w_ptr != W || plan->map_x_ptr != x || plan->map_cfg_id != cfg.id + 1024 * p.weight_format) {
            const CUtensorMapDataType wdt = p.weight_format == DET_WEIGHT_FP32   ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                            : p.weight_format == DET_WEIGHT_FP16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                                                                 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
            if (!encode_2d(&plan->map_w, wdt, p.weight_format == DET_WEIGHT_FP32 ? 4 : 2, W, (uint64_t)plan->n_count, (uint64_t)p.K,
                           (uint32_t)(cfg.rt * cfg.wr), (uint32_t)(cfg.kc < 256 ? cfg.kc : 256), CU_TENSOR_MAP_L2_PROMOTION_L2_256B))
                return DET_ERR_CUDA;
            if (!encode_2d(&plan->map_x, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, x, (uint64_t)p.M, (uint64_t)p.K,
                           (uint32_t)(cfg.mt * cfg.wm), (uint32_t)(cfg.kc < 256 ? cfg.kc : 256), CU_TENSOR_MAP_L2_PROMOTION_L2_256B))
                return DET_ERR_CUDA;
            plan->map_w_ptr = W; plan->map_x_ptr = x; plan->map_cfg_id = cfg.id + 1024 * p.weight_format;
        }
        e = launch_decode(a, cfg, &plan->map_w, &plan->map_x);
    } else if (kernel == kKernelPrefill) {
        // the TMA-fed kernel (variant 5 .. 8 forces its rows per thread); without the activation workspace, or with
        // variant 15 .. 18, the register-staged kernel
        const int v = plan->variant;
        if (!plan->x_t || (v >= 15 && v <= 18)) {
            e = launch_prefill(a);
        } else {
            const int tr = (v >= 5 && v <= 8) ? v : prefill_rows_per_thread(p.M);
            const int cfg_id = 4096 + tr + 1024 * p.weight_format;
            const int64_t ldt = (p.M + 3) / 4 * 4;
            e = launch_transpose_x(x, plan->x_t, p.M, p.K, ldt, stream);
            if (e != cudaSuccess) return cuda_fail("kernel launch", e);
            if (plan->map_w_ptr != W || plan->map_cfg_id != cfg_id) {
                const CUtensorMapDataType wdt = p.weight_format == DET_WEIGHT_FP32   ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                                : p.weight_format == DET_WEIGHT_FP16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                                                                     : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
                if (!encode_2d(&plan->map_w, wdt, p.weight_format == DET_WEIGHT_FP32 ? 4 : 2, W, (uint64_t)plan->n_count, (uint64_t)p.K,
                               128u, 32u, CU_TENSOR_MAP_L2_PROMOTION_L2_256B))
                    return DET_ERR_CUDA;
                if (!encode_2d(&plan->map_x, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, plan->x_t, (uint64_t)p.K, (uint64_t)ldt, 32u,
                               (uint32_t)(16 * tr), CU_TENSOR_MAP_L2_PROMOTION_L2_256B))
                    return DET_ERR_CUDA;
                plan->map_w_ptr = W; plan->map_x_ptr = plan->x_t; plan->map_cfg_id = cfg_id;
            }
            e = launch_prefill_tma(a, tr, &plan->map_w, &plan->map_x);
        }
    } else {
        e = launch_generic(a, p.bucket);
    }
    if (e != cudaSuccess) return cuda_fail("kernel launch", e);
    return DET_OK;
}

}  // namespace detlin

using namespace detlin;

extern "C" {

det_status_t det_linear_plan_params(int64_t M, int64_t N, int64_t K, det_linear_params_t* out)
{
    return fill_params(M, N, K, out);
}

det_linear_plan_t* det_linear_plan(int64_t M, int64_t N, int64_t K) { return det_linear_plan_w(M, N, K, DET_WEIGHT_BF16); }

det_linear_plan_t* det_linear_plan_w(int64_t M, int64_t N, int64_t K, int32_t wfmt)
{
    return det_linear_plan_shard(M, N, K, 0, N, N, wfmt);
}

det_linear_plan_t* det_linear_plan_shard(int64_t M, int64_t N, int64_t K, int64_t n_begin, int64_t n_count, int64_t ldy,
                                         int32_t wfmt)
{
    det_linear_params_t prm;
    g_last_status = fill_params(M, N, K, &prm);
    if (g_last_status != DET_OK) return nullptr;
    g_last_status = DET_ERR_INVALID_ARG;
    if (wfmt < DET_WEIGHT_BF16 || wfmt > DET_WEIGHT_FP32) { set_error("plan: unknown weight format %d", wfmt); return nullptr; }
    if (n_begin < 0 || n_count < 1 || n_begin > N - n_count || ldy < n_count) {
        set_error("plan: shard [%lld, %lld) with row pitch %lld does not fit a layer with N = %lld", (long long)n_begin,
                  (long long)(n_begin + n_count), (long long)ldy, (long long)N);
        return nullptr;
    }
    prm.workspace_bytes = (prm.bucket == 1 && prm.S > 1) ? 4ull * (uint64_t)prm.S * (uint64_t)M * (uint64_t)n_count : 0;
    prm.weight_format = wfmt;
    if (wfmt == DET_WEIGHT_FP32) prm.kernel = (K % 4 == 0) ? (prm.bucket == 0 ? kKernelDecode : kKernelPrefill) : kKernelGeneric;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { g_last_status = cuda_fail("cudaGetDevice", e); return nullptr; }
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, dev);
    if (e != cudaSuccess) { g_last_status = cuda_fail("cudaGetDeviceProperties", e); return nullptr; }
    if (prop.major != 10) {
        g_last_status = DET_ERR_ARCH;
        set_error("plan: device %d is sm_%d%d; this library is built for sm_100a only (no fallback)", dev, prop.major,
                  prop.minor);
        return nullptr;
    }
    det_linear_plan_t* plan = new (std::nothrow) det_linear_plan_t();
    if (!plan) { g_last_status = DET_ERR_ALLOC; set_error("plan: host allocation failed"); return nullptr; }
    memset(plan, 0, sizeof *plan);
    plan->prm = prm;
    plan->n_begin = n_begin;
    plan->n_count = n_count;
    plan->ldy = ldy;
    plan->device = dev;
    plan->sm_count = prop.multiProcessorCount;
    plan->forced_kernel = -1;
    plan->map_cfg_id = -1;
    plan->decode_cfg_variant = -1;
    plan->wait_limit_ns = kDefaultWaitLimitNs;
    g_last_status = DET_OK;
    e = device_alloc(reinterpret_cast<void**>(&plan->status), sizeof(DeviceStatus));
    if (e == cudaSuccess) e = cudaMemset(plan->status, 0, sizeof(DeviceStatus));
    // the partials are followed by one counter per output tile of the prefill kernel (at most ceil(M/80) ceil(N/128))
    const uint64_t counters_at = (prm.workspace_bytes + 255) / 256 * 256;
    const uint64_t n_counters = (uint64_t)((M + 79) / 80) * (uint64_t)((n_count + 127) / 128);
    if (e == cudaSuccess && prm.workspace_bytes) {
        e = device_alloc(reinterpret_cast<void**>(&plan->partials), counters_at + 4 * n_counters);
        if (e == cudaSuccess) {
            plan->tile_counters = reinterpret_cast<unsigned*>(reinterpret_cast<char*>(plan->partials) + counters_at);
            plan->n_tile_counters = n_counters;
            e = cudaMemset(plan->tile_counters, 0, 4 * n_counters);
        }
    }
    if (e != cudaSuccess) {
        g_last_status = DET_ERR_ALLOC;
        set_error("plan: device allocation (status word, %llu bytes of split-K workspace) failed: %s",
                  (unsigned long long)prm.workspace_bytes, cudaGetErrorString(e));
        cudaGetLastError();
        det_linear_plan_destroy(plan);              // frees whatever was allocated before the failure
        return nullptr;
    }
    // Activation workspace of the TMA-fed prefill kernel: x transposed, 4 K roundup(M, 4) bytes.
    // Without it the plan still works: it uses the register-staged kernel, which computes the same bits.
    if (prm.kernel == kKernelPrefill) {
        e = device_alloc(reinterpret_cast<void**>(&plan->x_t), 4ull * (uint64_t)((M + 3) / 4 * 4) * (uint64_t)K);
        if (e != cudaSuccess) { plan->x_t = nullptr; cudaGetLastError(); }
    }
    return plan;
}

det_status_t det_linear_run(const det_linear_plan_t* plan, const float* x, const uint16_t* W, const float* b, float* y,
                            void* stream)
{
    if (plan && plan->prm.weight_format == DET_WEIGHT_FP32) {
        set_error("run: the plan stores FP32 weights; use det_linear_run_w");
        return DET_ERR_INVALID_ARG;
    }
    return det_linear_run_w(plan, x, W, b, y, stream);
}

det_status_t det_linear_run_w(const det_linear_plan_t* plan, const float* x, const void* W, const float* b, float* y,
                              void* stream)
{
    if (!plan || !x || !W || !y) { set_error("run: plan, x, W and y must not be NULL"); return DET_ERR_INVALID_ARG; }
    // the plan's tensor-map cache is the only state a run touches
    return run_device(const_cast<det_linear_plan_t*>(plan), x, W, b, y, static_cast<cudaStream_t>(stream));
}

static det_status_t run_host_impl(det_linear_plan_t* plan, const float* x_host, const void* W, const float* b,
                                  float* y_host, void* stream, bool sync)
{
    if (!plan || !x_host || !W || !y_host) {
        set_error("run_host: plan, x_host, W and y_host must not be NULL");
        return DET_ERR_INVALID_ARG;
    }
    const det_linear_params_t& p = plan->prm;
    if (plan->n_count != p.N || plan->ldy != p.N) {
        set_error("run_host: the plan is a column shard; use det_linear_run_w with device buffers");
        return DET_ERR_INVALID_ARG;
    }
    const size_t xb = (size_t)p.M * p.K * 4, yb = (size_t)p.M * p.N * 4;
    cudaError_t e;
    if (!plan->x_stage) {
        e = device_alloc(reinterpret_cast<void**>(&plan->x_stage), xb);
        if (e == cudaSuccess) e = device_alloc(reinterpret_cast<void**>(&plan->y_stage), yb);
        if (e != cudaSuccess) {
            set_error("run_host: staging allocation failed: %s", cudaGetErrorString(e));
            cudaGetLastError();
            if (plan->x_stage) { cudaFree(plan->x_stage); plan->x_stage = nullptr; }     // all or nothing: a later call retries both
            return DET_ERR_ALLOC;
        }
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    e = cudaMemcpyAsync(plan->x_stage, x_host, xb, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail("run_host: copy of x", e);
    det_status_t s = run_device(plan, plan->x_stage, W, b, plan->y_stage, st);
    if (s != DET_OK) return s;
    e = cudaMemcpyAsync(y_host, plan->y_stage, yb, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail("run_host: copy of y", e);
    if (sync) {
        e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) return cuda_fail("run_host: synchronise", e);
    }
    return DET_OK;
}

det_status_t det_linear_run_host(det_linear_plan_t* plan, const float* x_host, const void* W, const float* b,
                                 float* y_host, void* stream)
{
    return run_host_impl(plan, x_host, W, b, y_host, stream, true);
}

det_status_t det_linear_run_host_async(det_linear_plan_t* plan, const float* x_host, const void* W, const float* b,
                                       float* y_host, void* stream)
{
    return run_host_impl(plan, x_host, W, b, y_host, stream, false);
}

det_status_t det_rmsnorm(const float* x, const float* g, float eps, int64_t M, int64_t H, float* y, void* stream)
{
    if (!x || !g || !y || M < 1 || H < 1 || H >= (1ll << 31) || M >= (1ll << 31)) {
        set_error("rmsnorm: NULL pointer or size out of range (1 <= M, H < 2^31)");
        return DET_ERR_INVALID_ARG;
    }
    if (!(eps >= 0.0f)) { set_error("rmsnorm: eps must be a non-negative number"); return DET_ERR_INVALID_ARG; }
    int dev = 0, major = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);   // cheap, per call
    if (e != cudaSuccess) return cuda_fail("rmsnorm: device query", e);
    if (major != 10) { set_error("rmsnorm: device %d is sm_%dx; this library is built for sm_100a only", dev, major); return DET_ERR_ARCH; }
    e = launch_rmsnorm(x, g, eps, M, H, y, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail("rmsnorm: launch", e);
    return DET_OK;
}

det_status_t det_attention_decode(const float* q, const float* k, const float* v, float scale, int64_t B, int64_t Hq, int64_t Hkv,
                                  int64_t T, int64_t D, float* o, void* stream)
{
    if (!q || !k || !v || !o) { set_error("attention: q, k, v and o must not be NULL"); return DET_ERR_INVALID_ARG; }
    if (B < 1 || Hq < 1 || Hkv < 1 || T < 1 || D < 1 || Hq % Hkv != 0 || B * Hkv >= (1ll << 31) || T >= (1ll << 24)) {
        set_error("attention: need B, Hq, Hkv, T, D >= 1, Hq a multiple of Hkv, B * Hkv < 2^31, T < 2^24");
        return DET_ERR_INVALID_ARG;
    }
    const int64_t G = Hq / Hkv;
    if ((G != 1 && G != 2 && G != 4 && G != 8) || D % 4 != 0 || D > 256) {
        set_error("attention: this kernel serves 1, 2, 4 or 8 query heads per KV head and head dimensions that are multiples of 4 up to 256 "
                  "(got Hq / Hkv = %lld, D = %lld)", (long long)G, (long long)D);
        return DET_ERR_UNSUPPORTED_SHAPE;
    }
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) {
        set_error("attention: q, k, v and o must be 16-byte aligned");
        return DET_ERR_ALIGNMENT;
    }
    const size_t smem = attention_smem_bytes((int)G, (int)T, (int)D);
    if (smem > 227u * 1024u) {
        set_error("attention: T = %lld keys with %lld query heads per KV head need %zu bytes of shared memory for the scores and the "
                  "segment sums; a thread block has %u", (long long)T, (long long)G, smem, 227u * 1024u);
        return DET_ERR_UNSUPPORTED_SHAPE;
    }
    int dev = 0, major = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail("attention: device query", e);
    if (major != 10) { set_error("attention: device %d is sm_%dx; this library is built for sm_100a only", dev, major); return DET_ERR_ARCH; }
    e = launch_attention_decode(q, k, v, scale, (int)B, (int)Hq, (int)Hkv, (int)T, (int)D, o, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail("attention: launch", e);
    return DET_OK;
}

det_status_t det_linear_plan_tune(det_linear_plan_t* plan, const float* x, const void* W, const float* b, float* y,
                                  void* stream, int32_t* variant_out, float* best_us_out)
{
    if (!plan || !x || !W || !y) { set_error("tune: plan, x, W and y must not be NULL"); return DET_ERR_INVALID_ARG; }
    if (variant_out) *variant_out = 0;
    if (best_us_out) *best_us_out = -1.0f;
    const det_linear_params_t& p = plan->prm;
    const int kernel = plan->forced_kernel >= 0 ? plan->forced_kernel : p.kernel;
    if (kernel != kKernelDecode) return DET_OK;                     // one schedule only: nothing to choose
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // cold weights: a buffer larger than L2 is rewritten before every timed run (skipped if it cannot be had)
    const size_t flush_bytes = 192u << 20;
    void* flush = nullptr;
    if (cudaMalloc(&flush, flush_bytes + 256) != cudaSuccess) { flush = nullptr; cudaGetLastError(); }
    else if (cudaMemsetAsync(flush, 0, flush_bytes + 256, st) != cudaSuccess) { cudaGetLastError(); }
    unsigned* sink = flush ? reinterpret_cast<unsigned*>(static_cast<char*>(flush) + flush_bytes) : nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaError_t e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    const int saved = plan->variant;
    det_status_t status = DET_OK;
    int best_variant = 0;
    float best_ms = 0.0f;
    if (e != cudaSuccess) status = cuda_fail("tune: event creation", e);
    for (int v = 1; status == DET_OK; ++v) {
        DecodeConfig cfg;
        if (!decode_config_for(p.M, plan->n_count, p.K, p.S, p.weight_format, v, &cfg)) break;
        plan->variant = v;
        status = run_device(plan, x, W, b, y, st);                  // loads the kernel, builds the tensor maps
        float v_ms = 0.0f;
        for (int rep = 0; rep < 5 && status == DET_OK; ++rep) {
            if (flush) e = launch_l2_evict(flush, flush_bytes, sink, plan->sm_count, st);
            if (e == cudaSuccess) e = cudaEventRecord(e0, st);
            if (e != cudaSuccess) { status = cuda_fail("tune: timing", e); break; }
            status = run_device(plan, x, W, b, y, st);
            if (status != DET_OK) break;
            e = cudaEventRecord(e1, st);
            if (e == cudaSuccess) e = cudaEventSynchronize(e1);
            float ms = 0.0f;
            if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
            if (e != cudaSuccess) { status = cuda_fail("tune: timing", e); break; }
            if (rep == 0 || ms < v_ms) v_ms = ms;
        }
        if (status == DET_OK && (best_variant == 0 || v_ms < best_ms)) { best_variant = v; best_ms = v_ms; }
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (flush) cudaFree(flush);
    if (status != DET_OK || best_variant == 0) { plan->variant = saved; return status; }
    plan->variant = best_variant;
    if (variant_out) *variant_out = best_variant;
    if (best_us_out) *best_us_out = best_ms * 1e3f;
    return DET_OK;
}

det_status_t det_linear_plan_check(det_linear_plan_t* plan, void* stream)
{
    if (!plan) { set_error("check: plan is NULL"); return DET_ERR_INVALID_ARG; }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DeviceStatus h{};
    cudaError_t e = cudaMemcpyAsync(&h, plan->status, sizeof h, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(plan->status, 0, sizeof h, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail("check", e);
    if (h.timeout_flag) {
        // a block that gave up did not count itself in: bring the tile counters of the in-kernel fold back to zero
        if (plan->tile_counters) {
            e = cudaMemsetAsync(plan->tile_counters, 0, 4 * plan->n_tile_counters, st);
            if (e == cudaSuccess) e = cudaStreamSynchronize(st);
            if (e != cudaSuccess) return cuda_fail("check", e);
        }
        set_error("check: a kernel gave up a bounded wait (site %u)", h.where);
        return DET_ERR_DEVICE_TIMEOUT;
    }
    return DET_OK;
}

det_status_t det_linear_plan_get_params(const det_linear_plan_t* plan, det_linear_params_t* out)
{
    if (!plan || !out) { set_error("get_params: NULL argument"); return DET_ERR_INVALID_ARG; }
    *out = plan->prm;
    return DET_OK;
}

det_status_t det_linear_plan_describe(const det_linear_plan_t* plan, char* buf, size_t n)
{
    if (!plan || !buf || n == 0) { set_error("describe: NULL argument"); return DET_ERR_INVALID_ARG; }
    const det_linear_params_t& p = plan->prm;
    static const char* kn[] = {"generic", "decode", "prefill"};
    char tiling[160] = "null";
    if (p.kernel == kKernelDecode) {
        DecodeConfig c;
        if (decode_config_for(p.M, plan->n_count, p.K, p.S, p.weight_format, plan->variant, &c))
            snprintf(tiling, sizeof tiling,
                     "{\"mt\": %d, \"wm\": %d, \"rt\": %d, \"wr\": %d, \"sk\": %d, \"kc\": %d, \"stages\": %d, \"blocks_per_sm\": %d}",
                     c.mt, c.wm, c.rt, c.wr, c.sk, c.kc, c.stages, decode_config_occupancy(p.weight_format, c, p.S));
    }
    char ptile[160] = "null";
    if (p.kernel == kKernelPrefill) {
        const int v = plan->variant;
        const bool staged = !plan->x_t || (v >= 15 && v <= 18);
        const int tr = (v >= 5 && v <= 8) ? v : (v >= 15 && v <= 18) ? v - 10 : prefill_rows_per_thread(p.M);
        snprintf(ptile, sizeof ptile, "{\"bm\": %d, \"bn\": 128, \"bk\": 32, \"feed\": \"%s\", \"activation_workspace_bytes\": %llu}",
                 16 * tr, staged ? "registers" : "tma",
                 plan->x_t ? 4ull * (unsigned long long)((p.M + 3) / 4 * 4) * (unsigned long long)p.K : 0ull);
    }
    int w = snprintf(buf, n,
                     "{\"M\": %lld, \"N\": %lld, \"K\": %lld, \"bucket\": \"%s\", \"V\": %d, \"L\": %d, \"P\": %d, "
                     "\"seg_len\": %lld, \"S\": %d, \"order_version\": %d, \"kernel\": \"%s\", \"workspace_bytes\": %llu, "
                     "\"weight_format\": \"%s\", \"variant\": %d, \"decode_tiling\": %s, \"prefill_tile\": %s, "
                     "\"shard\": {\"n_begin\": %lld, \"n_count\": %lld, \"ldy\": %lld}}",
                     (long long)p.M, (long long)p.N, (long long)p.K, p.bucket == 0 ? "decode" : "prefill", p.V, p.L, p.P,
                     (long long)p.seg_len, p.S, p.order_version, kn[p.kernel], (unsigned long long)p.workspace_bytes,
                     p.weight_format == DET_WEIGHT_FP32 ? "fp32" : p.weight_format == DET_WEIGHT_FP16 ? "fp16" : "bf16", plan->variant, tiling, ptile,
                     (long long)plan->n_begin, (long long)plan->n_count, (long long)plan->ldy);
    if (w < 0 || (size_t)w >= n) { set_error("describe: buffer too small (%d bytes needed)", w + 1); return DET_ERR_INVALID_ARG; }
    return DET_OK;
}

void det_linear_plan_destroy(det_linear_plan_t* plan)
{
    if (!plan) return;
    if (plan->partials) cudaFree(plan->partials);
    if (plan->x_t) cudaFree(plan->x_t);
    if (plan->status) cudaFree(plan->status);
    if (plan->x_stage) cudaFree(plan->x_stage);
    if (plan->y_stage) cudaFree(plan->y_stage);
    delete plan;
}

det_status_t det_argmax_rows(const float* y, int64_t M, int64_t N, int32_t* idx, void* stream)
{
    if (!y || !idx) { set_error("argmax: NULL argument"); return DET_ERR_INVALID_ARG; }
    if (M < 1 || N < 1 || N >= ((int64_t)1 << 31)) { set_error("argmax: need M >= 1 and 1 <= N < 2^31"); return DET_ERR_INVALID_ARG; }
    cudaError_t e = launch_argmax(y, M, N, idx, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail("argmax launch", e);
    return DET_OK;
}

const char* det_last_error(void) { return g_err; }

det_status_t det_last_status(void) { return static_cast<det_status_t>(g_last_status); }

int det_order_version(void) { return kOrderVersion; }

// ---------------------------------------------------------------------------------------------
// test-only exports
// ---------------------------------------------------------------------------------------------
det_status_t det_test_plan_force_kernel(det_linear_plan_t* plan, int kernel)
{
    if (!plan) { set_error("force_kernel: plan is NULL"); return DET_ERR_INVALID_ARG; }
    if (kernel < -1 || kernel > 2 || (kernel == kKernelDecode && plan->prm.bucket != 0) ||
        (kernel == kKernelPrefill && plan->prm.bucket != 1)) {
        set_error("force_kernel: kernel %d cannot serve this plan's bucket", kernel);
        return DET_ERR_INVALID_ARG;
    }
    plan->forced_kernel = kernel;
    return DET_OK;
}

det_status_t det_test_plan_set_max_blocks(det_linear_plan_t* plan, int max_blocks)
{
    if (!plan || max_blocks < 0) { set_error("set_max_blocks: bad argument"); return DET_ERR_INVALID_ARG; }
    plan->max_blocks = max_blocks;
    return DET_OK;
}

det_status_t det_test_plan_set_variant(det_linear_plan_t* plan, int variant)
{
    if (!plan || variant < 0) { set_error("set_variant: bad argument"); return DET_ERR_INVALID_ARG; }
    if (plan->prm.bucket == 0) {
        DecodeConfig cfg;
        if (!decode_config_for(plan->prm.M, plan->n_count, plan->prm.K, plan->prm.S, plan->prm.weight_format, variant, &cfg)) {
            set_error("set_variant: the decode kernel has fewer than %d tilings for this batch size", variant);
            return DET_ERR_INVALID_ARG;
        }
    } else if (variant != 0 && (variant < 5 || variant > 8) && (variant < 15 || variant > 18)) {
        set_error("set_variant: the prefill bucket takes 0 (automatic), 5 .. 8 (rows per thread) or 15 .. 18 (the same with "
                  "the register-staged kernel)");
        return DET_ERR_INVALID_ARG;
    }
    plan->variant = variant;
    return DET_OK;
}

void det_test_attention_set_split(int blocks_per_row) { attention_test_force_split(blocks_per_row); }

int det_test_attention_schedule(int64_t B, int64_t Hq, int64_t Hkv, int64_t T, int64_t D, int sm_count, uint64_t* smem_bytes_out)
{
    if (B < 1 || Hq < 1 || Hkv < 1 || T < 1 || D < 1 || Hq % Hkv != 0 || sm_count < 1) return 0;
    const int G = (int)(Hq / Hkv);
    int C = attention_split((int)B, (int)Hkv, G, (int)T, (int)D, sm_count);
    while (C < 16 && attention_block_smem_bytes(G, (int)T, (int)D, C) > 227u * 1024u) C *= 2;
    if (smem_bytes_out) *smem_bytes_out = attention_block_smem_bytes(G, (int)T, (int)D, C);
    return C;
}

void det_test_fail_next_alloc(int nth)
{
    g_fail_alloc_countdown = nth > 0 ? nth : 0;
}

det_status_t det_test_plan_set_wait(det_linear_plan_t* plan, uint64_t wait_limit_ns, int flags)
{
    if (!plan || wait_limit_ns == 0 || flags < 0 || flags > 3) { set_error("set_wait: bad argument"); return DET_ERR_INVALID_ARG; }
    plan->wait_limit_ns = wait_limit_ns;
    plan->test_flags = flags;
    return DET_OK;
}

struct GreenHandle {
    CUgreenCtx gctx;
    CUstream stream;
};

det_status_t det_test_green_stream_create(int sm_count, void** stream_out, void** handle_out, int* sm_granted)
{
    if (!stream_out || !handle_out || sm_count < 1) { set_error("green: bad argument"); return DET_ERR_INVALID_ARG; }
    typedef CUresult (*GetResFn)(CUdevice, CUdevResource*, CUdevResourceType);
    typedef CUresult (*SplitFn)(CUdevResource*, unsigned int*, const CUdevResource*, CUdevResource*, unsigned int, unsigned int);
    typedef CUresult (*GenDescFn)(CUdevResourceDesc*, CUdevResource*, unsigned int);
    typedef CUresult (*CreateFn)(CUgreenCtx*, CUdevResourceDesc, CUdevice, unsigned int);
    typedef CUresult (*StreamFn)(CUstream*, CUgreenCtx, unsigned int, int);
    typedef CUresult (*DevGetFn)(CUdevice*, int);
    static GetResFn get_res = driver_fn<GetResFn>("cuDeviceGetDevResource");
    static SplitFn split = driver_fn<SplitFn>("cuDevSmResourceSplitByCount");
    static GenDescFn gen_desc = driver_fn<GenDescFn>("cuDevResourceGenerateDesc");
    static CreateFn create = driver_fn<CreateFn>("cuGreenCtxCreate");
    static StreamFn stream_create = driver_fn<StreamFn>("cuGreenCtxStreamCreate");
    static DevGetFn dev_get = driver_fn<DevGetFn>("cuDeviceGet");
    if (!get_res || !split || !gen_desc || !create || !stream_create || !dev_get) {
        set_error("green: the driver does not provide the green-context entry points");
        return DET_ERR_CUDA;
    }
    int dev = 0;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce != cudaSuccess) return cuda_fail("green: cudaGetDevice", ce);
    cudaFree(nullptr);   // make sure the primary context exists
    CUdevice cudev;
    CUresult r = dev_get(&cudev, dev);
    CUdevResource all{}, part{}, rest{};
    if (r == CUDA_SUCCESS) r = get_res(cudev, &all, CU_DEV_RESOURCE_TYPE_SM);
    unsigned int groups = 1;
    if (r == CUDA_SUCCESS) r = split(&part, &groups, &all, &rest, 0, (unsigned)sm_count);
    CUdevResourceDesc desc{};
    if (r == CUDA_SUCCESS) r = gen_desc(&desc, &part, 1);
    GreenHandle* h = new (std::nothrow) GreenHandle();
    if (!h) { set_error("green: host allocation failed"); return DET_ERR_ALLOC; }
    if (r == CUDA_SUCCESS) r = create(&h->gctx, desc, cudev, CU_GREEN_CTX_DEFAULT_STREAM);
    if (r == CUDA_SUCCESS) r = stream_create(&h->stream, h->gctx, CU_STREAM_NON_BLOCKING, 0);
    if (r != CUDA_SUCCESS) {
        set_error("green: driver refused (CUresult %d)", (int)r);
        delete h;
        return DET_ERR_CUDA;
    }
    if (sm_granted) *sm_granted = (int)part.sm.smCount;
    *stream_out = h->stream;
    *handle_out = h;
    return DET_OK;
}

void det_test_green_stream_destroy(void* handle)
{
    if (!handle) return;
    GreenHandle* h = static_cast<GreenHandle*>(handle);
    typedef CUresult (*StreamDestroyFn)(CUstream);
    typedef CUresult (*DestroyFn)(CUgreenCtx);
    static StreamDestroyFn sd = driver_fn<StreamDestroyFn>("cuStreamDestroy");
    static DestroyFn gd = driver_fn<DestroyFn>("cuGreenCtxDestroy");
    if (sd) sd(h->stream);
    if (gd) gd(h->gctx);
    delete h;
}

}  // extern "C"
