// Negative control for rule R3 (the paper's split-K ablation: "none / ordered / atomic", supplement C).
// The same segment partials as the library's decode order, but combined with atomicAdd in whatever
// order the warps happen to finish, which is what the rule forbids: the result depends on grid
// scheduling and changes from run to run.  Test-only; nothing in the library calls this.
#include "internal.h"
#include "device_utils.cuh"
#include "det_linear_test.h"

namespace detlin {

__global__ void __launch_bounds__(256) atomic_init_kernel(float* __restrict__ y, const float* __restrict__ b, int64_t MN, int64_t N)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < MN) y[i] = b ? b[i % N] : 0.0f;
}

// one warp per (segment, weight row); segment-major so that the S warps of one output sit in
// different blocks and finish in an order nothing fixes
__global__ void __launch_bounds__(256)
atomic_splitk_kernel(const float* __restrict__ x, const uint16_t* __restrict__ W, float* __restrict__ y, int64_t M, int64_t N,
                     int64_t K, int64_t seg_len, int S)
{
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= N * S) return;
    const int s = (int)(warp / N);
    const int64_t n = warp % N;
    const int64_t k_lo = (int64_t)s * seg_len;
    const int64_t k_hi = (k_lo + seg_len < K) ? k_lo + seg_len : K;
    const uint16_t* wrow = W + n * K;
    for (int64_t m = 0; m < M; ++m) {
        const float* xrow = x + m * K;
        float a = 0.0f;
        for (int64_t c = k_lo; c < k_hi; c += 128) {
            const int64_t k0 = c + 4 * lane;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int64_t k = k0 + j;
                if (k < k_hi) a = __fmaf_rn(xrow[k], up_elem<0>(wrow[k]), a);
            }
        }
        const float t = lane_tree_sum(a);
        if (lane == 0) atomicAdd(&y[m * N + n], t);
    }
}

// Harness glue for multi-layer tests: dst[m, j] = src[m, j] * c for the first `cols` columns of a
// row-major matrix with row pitch ld_src (one rounding per element).  Launched with programmatic
// dependent launch on both sides so that a chain linear -> glue -> linear keeps overlapping.
__global__ void __launch_bounds__(256)
scale_cols_kernel(const float* __restrict__ src, int64_t ld_src, float* __restrict__ dst, int64_t M, int64_t cols, float c)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int64_t total = M * cols;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t m = i / cols, j = i - m * cols;
        dst[i] = __fmul_rn(src[m * ld_src + j], c);
    }
}

}  // namespace detlin

using namespace detlin;

extern "C" det_status_t det_test_scale_cols(const float* src, int64_t ld_src, float* dst, int64_t M, int64_t cols, float c,
                                            void* stream)
{
    if (!src || !dst || M < 1 || cols < 1 || ld_src < cols) { set_error("scale_cols: bad argument"); return DET_ERR_INVALID_ARG; }
    const int64_t total = M * cols;
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 8) blocks = 148 * 8;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(256);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, scale_cols_kernel, src, ld_src, dst, M, cols, c);
    if (e != cudaSuccess) { set_error("scale_cols: launch failed: %s", cudaGetErrorString(e)); return DET_ERR_CUDA; }
    return DET_OK;
}

extern "C" det_status_t det_test_linear_atomic_splitk(int64_t M, int64_t N, int64_t K, int32_t S_req, const float* x,
                                                      const uint16_t* W, const float* b, float* y, void* stream)
{
    if (M < 1 || N < 1 || K < 1 || S_req < 1 || !x || !W || !y || M * N > (1ll << 31) || N * (int64_t)S_req > (1ll << 31)) {
        set_error("atomic_splitk: bad argument");
        return DET_ERR_INVALID_ARG;
    }
    // the library's segment rule for a requested split: whole 256-element blocks, no empty segment
    const int64_t n256 = (K + 255) / 256;
    const int64_t req = S_req < n256 ? S_req : n256;
    const int64_t per = (n256 + req - 1) / req;
    const int64_t seg_len = 256 * per;
    const int S = (int)((n256 + per - 1) / per);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t MN = M * N;
    atomic_init_kernel<<<(unsigned)((MN + 255) / 256), 256, 0, st>>>(y, b, MN, N);
    const int64_t warps = N * S;
    atomic_splitk_kernel<<<(unsigned)((warps + 7) / 8), 256, 0, st>>>(x, W, y, M, N, K, seg_len, S);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("atomic_splitk: launch failed: %s", cudaGetErrorString(e)); return DET_ERR_CUDA; }
    return DET_OK;
}
