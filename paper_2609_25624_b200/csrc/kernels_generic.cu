// Generic kernels: any shape, any alignment, scalar bounds-checked loads.  They execute exactly the
// frozen order and serve ragged shapes (K % 8 != 0, misaligned buffers: what the
// paper's ragged 100 x 1000 x 1000 probe exercises), the split-K second pass and the row argmax.  They are not tuned.
#include "internal.h"
#include "device_utils.cuh"
#include <cooperative_groups.h>

namespace detlin {

// Decode order (V=4, L=32, P=1, S segments): one warp per weight row n.  Lane l owns k = c + 4l + j in
// every 128-element chunk of a segment and accumulates them in ascending order into one chain; the 32
// lanes are summed adjacent-first; the warp walks the S segments in ascending order and folds their sums
// as it goes (rule R3), so this bucket needs no workspace and no second pass.
template <int WF>
__global__ void __launch_bounds__(256)
generic_decode_kernel(const float* __restrict__ x, const typename WeightElem<WF>::type* __restrict__ W, const float* __restrict__ b,
                      float* __restrict__ y, int64_t M, int64_t N, int64_t K, int64_t seg_len, int S, int64_t ldy)
{
    const int lane = threadIdx.x & 31;
    const int64_t n = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (n >= N) return;
    const typename WeightElem<WF>::type* wrow = W + n * K;
    for (int64_t m = 0; m < M; ++m) {
        const float* xrow = x + m * K;
        float t = 0.0f;
        for (int s = 0; s < S; ++s) {
            const int64_t k_lo = (int64_t)s * seg_len;
            const int64_t k_hi = (k_lo + seg_len < K) ? k_lo + seg_len : K;
            float a = 0.0f;
            for (int64_t c = k_lo; c < k_hi; c += 128) {
                const int64_t k0 = c + 4 * lane;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int64_t k = k0 + j;
                    if (k < k_hi) a = __fmaf_rn(xrow[k], up_elem<WF>(wrow[k]), a);
                }
            }
            const float p = lane_tree_sum(a);
            t = (s == 0) ? p : __fadd_rn(t, p);
        }
        if (lane == 0) y[m * ldy + n] = b ? __fadd_rn(t, b[n]) : t;
    }
}

// Prefill order (V=1, L=1, P=1): one thread per (m, n, segment), one chain, strictly ascending k.
template <int WF>
__global__ void __launch_bounds__(256)
generic_prefill_kernel(const float* __restrict__ x, const typename WeightElem<WF>::type* __restrict__ W, const float* __restrict__ b,
                       float* __restrict__ out, int64_t M, int64_t N, int64_t K, int64_t seg_len, int S, int direct, int64_t ldy)
{
    const int64_t n = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t m = blockIdx.y;
    const int s = blockIdx.z;
    if (n >= N) return;
    const int64_t k_lo = (int64_t)s * seg_len;
    const int64_t k_hi = (k_lo + seg_len < K) ? k_lo + seg_len : K;
    const float* xrow = x + m * K;
    const typename WeightElem<WF>::type* wrow = W + n * K;
    float t = 0.0f;
    for (int64_t k = k_lo; k < k_hi; ++k) t = __fmaf_rn(xrow[k], up_elem<WF>(wrow[k]), t);
    if (direct) out[m * ldy + n] = b ? __fadd_rn(t, b[n]) : t;
    else        out[((int64_t)s * M + m) * N + n] = t;
}

// Split-K second pass (rule R3): the S partials of every output are added in ascending segment
// order by one thread, then the bias; no atomics anywhere.
__global__ void __launch_bounds__(256)
combine_kernel(const float* __restrict__ partials, const float* __restrict__ b, float* __restrict__ y,
               int64_t MN, int64_t N, int S, int64_t ldy)
{
    // programmatic dependent launch: the next kernel may start its prologue; the partials are read
    // only after the kernel that wrote them has completed
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= MN) return;
    float t = partials[i];
    for (int s = 1; s < S; ++s) t = __fadd_rn(t, partials[(int64_t)s * MN + i]);
    const int64_t m = i / N, n = i % N;
    y[m * ldy + n] = b ? __fadd_rn(t, b[n]) : t;
}

template <int WF>
static cudaError_t launch_generic_t(const LaunchArgs& a, int bucket)
{
    typedef typename WeightElem<WF>::type WT;
    const WT* W = static_cast<const WT*>(a.W);
    if (bucket == 0) {
        const int64_t blocks = (a.N + 7) / 8;
        generic_decode_kernel<WF><<<(unsigned)blocks, 256, 0, a.stream>>>(a.x, W, a.b, a.y, a.M, a.N, a.K, a.seg_len, a.S, a.ldy);
        return cudaGetLastError();
    }
    const int direct = (a.S == 1);
    float* out = direct ? a.y : a.partials;
    {
        // grid.y carries M (< 65536 per launch); larger M is cut into slabs of rows
        const int64_t max_y = 32768;
        for (int64_t m0 = 0; m0 < a.M; m0 += max_y) {
            const int64_t mm = (a.M - m0 < max_y) ? a.M - m0 : max_y;
            dim3 grid((unsigned)((a.N + 255) / 256), (unsigned)mm, (unsigned)a.S);
            float* o = out + m0 * (direct ? a.ldy : a.N);   // both layouts ([M][ldy] and [s][M][N]) advance by whole rows
            generic_prefill_kernel<WF><<<grid, 256, 0, a.stream>>>(a.x + m0 * a.K, W, a.b, o, a.M, a.N, a.K, a.seg_len, a.S, direct, a.ldy);
        }
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (!direct) return launch_combine(a);
    return cudaSuccess;
}

cudaError_t launch_generic(const LaunchArgs& a, int bucket)
{
    if (a.wfmt == 1) return launch_generic_t<1>(a, bucket);
    if (a.wfmt == 2) return launch_generic_t<2>(a, bucket);
    return launch_generic_t<0>(a, bucket);
}

cudaError_t launch_combine(const LaunchArgs& a)
{
    const int64_t MN = a.M * a.N;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)((MN + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = a.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, combine_kernel, (const float*)a.partials, a.b, a.y, MN, a.N, a.S, a.ldy);
}

// Row argmax, lowest index on ties (the paper's stated tie rule for greedy decoding).  Ordering
// key: NaN beats everything (first NaN wins), otherwise larger value, then smaller index.
// Comparisons only, so the result is exact and order-free.  A cluster of kArgmaxCluster blocks
// shares one row: each block scans a contiguous slice, the partial results meet in block 0 of the
// cluster through distributed shared memory (hardware cluster barrier, no spinning).
namespace cg = cooperative_groups;
constexpr int kArgmaxCluster = 8;

__device__ __forceinline__ bool argmax_better(float v, int i, float bv, int bi)
{
    const bool vn = (v != v), bn = (bv != bv);
    if (vn || bn) return vn && (!bn || i < bi);
    return (v > bv) || (v == bv && i < bi);
}

__device__ __forceinline__ void argmax_warp(float& bv, int& bi)
{
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, d);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, d);
        if (argmax_better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
    }
}

__global__ void __cluster_dims__(kArgmaxCluster, 1, 1) __launch_bounds__(1024)
argmax_rows_kernel(const float* __restrict__ y, int64_t N, int32_t* __restrict__ idx)
{
    __shared__ float sv[32];
    __shared__ int si[32];
    __shared__ float block_v;
    __shared__ int block_i;
    // programmatic dependent launch: let the next kernel of the stream start its prologue now, and
    // wait for the kernel that produced y before reading it
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const float* row = y + (int64_t)blockIdx.y * N;
    const int64_t per = (N + kArgmaxCluster - 1) / kArgmaxCluster;
    const int64_t lo = rank * per;
    const int64_t hi = (lo + per < N) ? lo + per : N;
    // a block whose slice is empty contributes the row's first element (always a valid candidate)
    float bv = row[lo < N ? lo : 0];
    int bi = (int)(lo < N ? lo : 0);
    for (int64_t n = lo + threadIdx.x; n < hi; n += blockDim.x) {
        const float v = row[n];
        if (argmax_better(v, (int)n, bv, bi)) { bv = v; bi = (int)n; }
    }
    argmax_warp(bv, bi);
    if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = bv; si[threadIdx.x >> 5] = bi; }
    __syncthreads();
    if (threadIdx.x < 32) {
        const int nw = blockDim.x >> 5;
        bv = (threadIdx.x < nw) ? sv[threadIdx.x] : sv[0];
        bi = (threadIdx.x < nw) ? si[threadIdx.x] : si[0];
        argmax_warp(bv, bi);
        if (threadIdx.x == 0) { block_v = bv; block_i = bi; }
    }
    cluster.sync();
    if (rank == 0 && threadIdx.x == 0) {
        bv = block_v;
        bi = block_i;
        for (int r = 1; r < kArgmaxCluster; ++r) {
            const float ov = *cluster.map_shared_rank(&block_v, r);
            const int oi = *cluster.map_shared_rank(&block_i, r);
            if (argmax_better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
        }
        idx[blockIdx.y] = bi;
    }
    cluster.sync();     // keep every block's shared memory alive until block 0 has read it
}

cudaError_t launch_argmax(const float* y, int64_t M, int64_t N, int32_t* idx, cudaStream_t stream)
{
    const int64_t max_rows = 65535;
    for (int64_t m0 = 0; m0 < M; m0 += max_rows) {
        const int64_t mm = (M - m0 < max_rows) ? M - m0 : max_rows;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(kArgmaxCluster, (unsigned)mm);
        cfg.blockDim = dim3(1024);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t e = cudaLaunchKernelEx(&cfg, argmax_rows_kernel, y + m0 * N, N, idx + m0);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace detlin
