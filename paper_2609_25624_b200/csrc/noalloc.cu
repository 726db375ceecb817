// det_linear_run_noalloc: the linear layer for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need a linear layer:
// code running inside a memory pool or arena that owns all device memory, a plugin whose contract
// forbids allocation after initialisation, a latency-critical loop where an allocation (an implicit
// device synchronisation) is unacceptable.  The ordinary entry points allocate when a plan is
// created (status word, split-K partials).  This one allocates nothing, neither on the device nor
// on the host: the split-K partials live in a fixed array that is part of the library image.
//
// The paper has no counterpart for this entry point; it computes exactly the same thing (same
// order, same bits) as det_linear_plan + det_linear_run.
#include "internal.h"
#include <mutex>

namespace detlin {

// Scratch for the split-K partials [S, M, N] (FP32).  Every GPU that loads the library holds these
// 4 MiB until the process exits.  All calls share the array.
constexpr size_t kNoallocScratchFloats = (size_t)1 << 20;
static __device__ __align__(256) float g_noalloc_scratch[kNoallocScratchFloats];

static float* g_scratch_addr[kMaxDevices];      // device address of the array, per device
static std::mutex g_scratch_mutex;

// In host code `g_noalloc_scratch` is only a handle for the runtime, not a device address; the
// address a kernel can use has to be asked for, once per device, with that device current.
static cudaError_t scratch_address(float** out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = static_cast<float*>(p);
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace detlin

using namespace detlin;

extern "C" det_status_t det_linear_run_noalloc(int64_t M, int64_t N, int64_t K, const float* x, const uint16_t* W,
                                               const float* b, float* y, void* stream)
{
    if (!x || !W || !y) { set_error("run_noalloc: x, W and y must not be NULL"); return DET_ERR_INVALID_ARG; }
    det_linear_params_t p;
    det_status_t st = fill_params(M, N, K, &p);
    if (st != DET_OK) return st;
    const uint64_t need = p.workspace_bytes / 4;            // split-K partials of the prefill bucket, in floats
    if (need > kNoallocScratchFloats) {
        set_error("run_noalloc: this shape splits K into %d segments and needs %llu bytes of partials; the built-in "
                  "scratch holds %llu bytes (use det_linear_plan + det_linear_run for larger problems)",
                  p.S, (unsigned long long)(need * 4), (unsigned long long)(kNoallocScratchFloats * 4));
        return DET_ERR_UNSUPPORTED_SHAPE;
    }
    int dev = 0, major = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) { set_error("run_noalloc: device query: %s", cudaGetErrorString(e)); return DET_ERR_CUDA; }
    if (major != 10) {
        set_error("run_noalloc: device %d is sm_%dx; this library is built for sm_100a only (no fallback)", dev, major);
        return DET_ERR_ARCH;
    }
    float* scratch = nullptr;
    e = scratch_address(&scratch);
    if (e != cudaSuccess) {
        set_error("run_noalloc: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
        return DET_ERR_CUDA;
    }
    LaunchArgs a{};
    a.x = x; a.W = W; a.b = b; a.y = y;
    a.wfmt = DET_WEIGHT_BF16;
    a.partials = need ? scratch : nullptr;       // every partial is written by the first pass before the
    a.M = M; a.N = N; a.K = K; a.ldy = N;                   // second pass reads it: nothing has to start at zero
    a.seg_len = p.seg_len; a.S = p.S;
    a.stream = static_cast<cudaStream_t>(stream);
    e = launch_generic(a, p.bucket);
    if (e != cudaSuccess) { set_error("run_noalloc: kernel launch: %s", cudaGetErrorString(e)); return DET_ERR_CUDA; }
    return DET_OK;
}
