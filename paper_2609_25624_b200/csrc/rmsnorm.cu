// Fixed-order RMSNorm: y[m,h] = (x[m,h] * r[m]) * g[h],  r = 1 / sqrt(ss / H + eps).
// Not one of the paper's kernels: the paper leaves RMSNorm to vendor FP32 kernels and names the
// reductions outside the linear layers as the residual channel of divergence.  This kernel applies
// the decode order family of the linear layers (V = 4, L = 32, one segment) to the row's sum of
// squares, so its bits do not depend on the grid, the SM count or the batch size either:
//   chunks of 128 elements ascending; lane l owns the 4 consecutive elements c + 4 l + j; each
//   element enters the lane's accumulator with one fma.rn(x, x, acc) from +0; elements beyond H are
//   skipped; the 32 lane sums are added by the adjacent-first tree (shuffle xor 1, 2, 4, 8, 16).
// Then one IEEE binary32 operation per step: mean = ss / float(H); t = mean + eps; root = sqrt(t);
// r = 1 / root; y = (x * r) * g.
//
// Schedule (numerically inert): one warp per row, eight rows per block.  The 32 chains of a row are
// exactly one warp's lanes, so a row cannot use more than one warp without changing the order.
// Rows of up to 4096 elements are held in registers (one read of x, all loads in flight at once);
// longer rows stream twice: pass 1 with 16-byte loads (a warp reads 512 contiguous bytes per chunk),
// pass 2 re-reads the row (L1/L2: a row is a few KB) and writes y with 16-byte stores.  HBM traffic
// is 4 M H bytes in and 4 M H out.
#include "internal.h"
#include "device_utils.cuh"

namespace detlin {

namespace {

constexpr int kRowsPerBlock = 8;

template <bool VEC>
__global__ void __launch_bounds__(kRowsPerBlock * 32)
rmsnorm_kernel(const float* __restrict__ x, const float* __restrict__ g, float eps, long long M, long long H,
               float* __restrict__ y)
{
    const int lane = threadIdx.x & 31;
    const long long m = (long long)blockIdx.x * kRowsPerBlock + (threadIdx.x >> 5);
    if (m >= M) return;
    const float* xr = x + m * H;
    float* yr = y + m * H;

    float a = 0.0f;
    if (VEC) {
        // H % 4 == 0 and 16-byte aligned rows: a lane's four elements are all inside or all outside H
        long long c = 0;
        for (; c + 512 <= H; c += 512) {               // four chunks in flight per lane
            float4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = __ldg(reinterpret_cast<const float4*>(xr + c + 128 * u + 4 * lane));
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                a = __fmaf_rn(v[u].x, v[u].x, a);
                a = __fmaf_rn(v[u].y, v[u].y, a);
                a = __fmaf_rn(v[u].z, v[u].z, a);
                a = __fmaf_rn(v[u].w, v[u].w, a);
            }
        }
        for (; c < H; c += 128) {
            const long long k = c + 4 * lane;
            if (k < H) {
                const float4 v = __ldg(reinterpret_cast<const float4*>(xr + k));
                a = __fmaf_rn(v.x, v.x, a);
                a = __fmaf_rn(v.y, v.y, a);
                a = __fmaf_rn(v.z, v.z, a);
                a = __fmaf_rn(v.w, v.w, a);
            }
        }
    } else {
        for (long long c = 0; c < H; c += 128) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const long long k = c + 4 * lane + j;
                if (k < H) {
                    const float v = __ldg(xr + k);
                    a = __fmaf_rn(v, v, a);
                }
            }
        }
    }
    const float ss = lane_tree_sum(a);                  // all lanes hold the same bits afterwards
    const float mean = __fdiv_rn(ss, (float)H);
    const float t = __fadd_rn(mean, eps);
    const float root = __fsqrt_rn(t);
    const float r = __fdiv_rn(1.0f, root);

    if (VEC) {
        for (long long k = 4 * lane; k < H; k += 128) {
            const float4 v = *reinterpret_cast<const float4*>(xr + k);
            const float4 w = __ldg(reinterpret_cast<const float4*>(g + k));
            float4 o;
            o.x = __fmul_rn(__fmul_rn(v.x, r), w.x);
            o.y = __fmul_rn(__fmul_rn(v.y, r), w.y);
            o.z = __fmul_rn(__fmul_rn(v.z, r), w.z);
            o.w = __fmul_rn(__fmul_rn(v.w, r), w.w);
            *reinterpret_cast<float4*>(yr + k) = o;
        }
    } else {
        for (long long k = lane; k < H; k += 32) yr[k] = __fmul_rn(__fmul_rn(xr[k], r), __ldg(g + k));
    }
}

// Rows of at most 128 CH elements (16-byte aligned, H % 4 == 0): the whole row stays in registers, so
// x crosses the memory system once, every load of the row is in flight at the same time, and pass 2
// needs no second read.  Same order: chunk u of the row is v[u], walked in ascending u.
template <int CH>
__global__ void __launch_bounds__(kRowsPerBlock * 32)
rmsnorm_row_in_registers_kernel(const float* __restrict__ x, const float* __restrict__ g, float eps, long long M, int H,
                                float* __restrict__ y)
{
    const int lane = threadIdx.x & 31;
    const long long m = (long long)blockIdx.x * kRowsPerBlock + (threadIdx.x >> 5);
    if (m >= M) return;
    const float* xr = x + m * H;
    float* yr = y + m * H;
    float4 v[CH];
#pragma unroll
    for (int u = 0; u < CH; ++u) {
        const int k = 128 * u + 4 * lane;
        if (k < H) asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                                : "=f"(v[u].x), "=f"(v[u].y), "=f"(v[u].z), "=f"(v[u].w) : "l"(xr + k));
    }
    float a = 0.0f;
#pragma unroll
    for (int u = 0; u < CH; ++u) {
        if (128 * u + 4 * lane < H) {
            a = __fmaf_rn(v[u].x, v[u].x, a);
            a = __fmaf_rn(v[u].y, v[u].y, a);
            a = __fmaf_rn(v[u].z, v[u].z, a);
            a = __fmaf_rn(v[u].w, v[u].w, a);
        }
    }
    const float ss = lane_tree_sum(a);
    const float mean = __fdiv_rn(ss, (float)H);
    const float t = __fadd_rn(mean, eps);
    const float root = __fsqrt_rn(t);
    const float r = __fdiv_rn(1.0f, root);
#pragma unroll
    for (int u = 0; u < CH; ++u) {
        const int k = 128 * u + 4 * lane;
        if (k < H) {
            const float4 w = __ldg(reinterpret_cast<const float4*>(g + k));
            float4 o;
            o.x = __fmul_rn(__fmul_rn(v[u].x, r), w.x);
            o.y = __fmul_rn(__fmul_rn(v[u].y, r), w.y);
            o.z = __fmul_rn(__fmul_rn(v[u].z, r), w.z);
            o.w = __fmul_rn(__fmul_rn(v[u].w, r), w.w);
            *reinterpret_cast<float4*>(yr + k) = o;
        }
    }
}

}  // namespace

cudaError_t launch_rmsnorm(const float* x, const float* g, float eps, int64_t M, int64_t H, float* y, cudaStream_t stream)
{
    const long long blocks = (M + kRowsPerBlock - 1) / kRowsPerBlock;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    const bool vec = (H % 4 == 0) && ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(g) | reinterpret_cast<uintptr_t>(y)) % 16 == 0);
    if (vec && H <= 128 * 8) {
        rmsnorm_row_in_registers_kernel<8><<<(unsigned)blocks, kRowsPerBlock * 32, 0, stream>>>(x, g, eps, M, (int)H, y);
    } else if (vec && H <= 128 * 32) {
        rmsnorm_row_in_registers_kernel<32><<<(unsigned)blocks, kRowsPerBlock * 32, 0, stream>>>(x, g, eps, M, (int)H, y);
    } else if (vec) rmsnorm_kernel<true><<<(unsigned)blocks, kRowsPerBlock * 32, 0, stream>>>(x, g, eps, M, H, y);
    else     rmsnorm_kernel<false><<<(unsigned)blocks, kRowsPerBlock * 32, 0, stream>>>(x, g, eps, M, H, y);
    return cudaGetLastError();
}

}  // namespace detlin
