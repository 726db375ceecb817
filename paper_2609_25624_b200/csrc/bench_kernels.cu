// Two calibration kernels used by the benchmark to measure the denominators of its rooflines on
// the device it runs on: the FP32 fused-multiply-add issue peak of the CUDA cores (scalar FFMA and
// packed FP32x2 FFMA2), and the read-only streaming bandwidth of HBM.  They compute nothing of the
// method; the paper has no counterpart.
#include "internal.h"
#include "det_linear_test.h"

namespace detlin {

template <int PACKED>
__global__ void __launch_bounds__(256) fma_peak_kernel(float* out, int iters)
{
    float2 a[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) a[i] = make_float2(threadIdx.x * 1e-3f + i, 1.0f * i);
    const float2 x = make_float2(1.0f + threadIdx.x * 1e-7f, 1.0f - threadIdx.x * 1e-7f);
    const float2 w = make_float2(0.999999f, 1.000001f);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                if (PACKED) {
                    a[i] = __ffma2_rn(x, w, a[i]);
                } else {
                    a[i].x = __fmaf_rn(x.x, w.x, a[i].x);
                    a[i].y = __fmaf_rn(x.y, w.y, a[i].y);
                }
            }
        }
    }
    float r = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) r += a[i].x + a[i].y;
    if (r == 123.456f) out[0] = r;    // keeps the loop alive without a store on the normal path
}

// The prefill multiply loop alone: 8 x 8 outputs per thread, both operand tiles k-major and resident in shared
// memory, four 16-byte loads per 32 packed FMAs, no staging, no barriers: the ceiling of that loop.
__global__ void __launch_bounds__(256, 2) fma_loop_kernel(float* out, int iters, const float* __restrict__ in)
{
    __shared__ __align__(16) float tile[2 * 32 * 132];
    for (int i = threadIdx.x; i < 2 * 32 * 132; i += 256) tile[i] = in[i & 63];
    __syncthreads();
    const uint32_t base = (uint32_t)__cvta_generic_to_shared(tile);
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const uint32_t xb = base + ty * 16, xb2 = xb + 64 * 4, wb = base + 32 * 132 * 4 + tx * 16;
    float2 acc[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int p = 0; p < 4; ++p) acc[i][p] = make_float2((float)i, (float)p);
    for (int it = 0; it < iters; ++it) {
#pragma unroll 8
        for (int kk = 0; kk < 32; ++kk) {
            float4 v[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t a = (q == 0 ? xb : q == 1 ? xb2 : q == 2 ? wb : wb + 64 * 4) + kk * 132 * 4;
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v[q].x), "=f"(v[q].y), "=f"(v[q].z), "=f"(v[q].w) : "r"(a));
            }
            const float xv[8] = {v[0].x, v[0].y, v[0].z, v[0].w, v[1].x, v[1].y, v[1].z, v[1].w};
            const float2 wp[4] = {make_float2(v[2].x, v[2].y), make_float2(v[2].z, v[2].w), make_float2(v[3].x, v[3].y),
                                  make_float2(v[3].z, v[3].w)};
#pragma unroll
            for (int p = 0; p < 4; ++p)
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[i][p] = __ffma2_rn(make_float2(xv[i], xv[i]), wp[p], acc[i][p]);
        }
    }
    float r = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int p = 0; p < 4; ++p) r += acc[i][p].x + acc[i][p].y;
    if (r == 123.456f) out[0] = r;
}

__global__ void __launch_bounds__(512) read_stream_kernel(const uint4* __restrict__ p, size_t n, unsigned* out)
{
    unsigned acc = 0;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < n; i += 4 * stride) {
        uint4 v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(v[j].x), "=r"(v[j].y), "=r"(v[j].z), "=r"(v[j].w)
                         : "l"(p + i + j * stride));
#pragma unroll
        for (int j = 0; j < 4; ++j) acc ^= v[j].x ^ v[j].y ^ v[j].z ^ v[j].w;
    }
    for (; i < n; i += stride) {
        const uint4 v = p[i];
        acc ^= v.x ^ v.y ^ v.z ^ v.w;
    }
    if (acc == 0x12345678u) out[0] = acc;
}

// Stream `bytes` of device memory through L2 (read only, so nothing is left dirty): used to evict a
// weight matrix before a timed run.
cudaError_t launch_l2_evict(const void* buf, size_t bytes, unsigned* sink, int sm_count, cudaStream_t stream)
{
    read_stream_kernel<<<sm_count * 8, 512, 0, stream>>>(static_cast<const uint4*>(buf), bytes / 16, sink);
    return cudaGetLastError();
}

}  // namespace detlin

using namespace detlin;

extern "C" {

det_status_t det_test_measure_fma_peak(int packed, double* tflops_out)
{
    if (!tflops_out) { set_error("measure_fma_peak: NULL argument"); return DET_ERR_INVALID_ARG; }
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    float* out = nullptr;
    if (e == cudaSuccess) e = cudaMalloc(&out, 256);
    if (e == cudaSuccess) e = cudaMemset(out, 0, 256);
    if (e != cudaSuccess) { set_error("measure_fma_peak: %s", cudaGetErrorString(e)); return DET_ERR_CUDA; }
    const bool loop = (packed == 2);                 // the prefill multiply loop on resident shared memory
    const int iters = loop ? 2048 : 4096, blocks = loop ? sms * 2 : sms * 8;
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    float best = 1e30f;
    for (int rep = 0; rep < 6; ++rep) {
        cudaEventRecord(e0);
        if (loop) fma_loop_kernel<<<blocks, 256>>>(out, iters, out);
        else if (packed) fma_peak_kernel<1><<<blocks, 256>>>(out, iters);
        else        fma_peak_kernel<0><<<blocks, 256>>>(out, iters);
        cudaEventRecord(e1);
        e = cudaEventSynchronize(e1);
        if (e != cudaSuccess) break;
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        if (rep > 0 && ms < best) best = ms;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(out);
    if (e != cudaSuccess) { set_error("measure_fma_peak: %s", cudaGetErrorString(e)); return DET_ERR_CUDA; }
    // per thread and iteration: 4 x 16 x 2 FMAs = 256 flop (register loops); 32 k x 64 FMAs = 4096 flop (tile loop)
    *tflops_out = (loop ? 4096.0 : 256.0) * iters * 256.0 * blocks / (best * 1e-3) / 1e12;
    return DET_OK;
}

det_status_t det_test_measure_read_bandwidth(const void* buf, size_t bytes, double* gbs_out)
{
    if (!buf || !gbs_out || bytes < (1u << 20) || (reinterpret_cast<uintptr_t>(buf) & 15u)) {
        set_error("measure_read_bandwidth: need a 16-byte aligned device buffer of at least 1 MiB");
        return DET_ERR_INVALID_ARG;
    }
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    unsigned* out = nullptr;
    if (e == cudaSuccess) e = cudaMalloc(&out, 256);
    if (e != cudaSuccess) { set_error("measure_read_bandwidth: %s", cudaGetErrorString(e)); return DET_ERR_CUDA; }
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    float best = 1e30f;
    for (int rep = 0; rep < 6; ++rep) {
        cudaEventRecord(e0);
        read_stream_kernel<<<sms * 8, 512>>>(static_cast<const uint4*>(buf), bytes / 16, out);
        cudaEventRecord(e1);
        e = cudaEventSynchronize(e1);
        if (e != cudaSuccess) break;
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        if (rep > 0 && ms < best) best = ms;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(out);
    if (e != cudaSuccess) { set_error("measure_read_bandwidth: %s", cudaGetErrorString(e)); return DET_ERR_CUDA; }
    *gbs_out = (double)bytes / (best * 1e-3) / 1e9;
    return DET_OK;
}

}  // extern "C"
