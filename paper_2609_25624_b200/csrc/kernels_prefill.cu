// Prefill kernel (bucket M > 64): register-tiled FP32 GEMM on the CUDA cores (rule R1: IEEE FMA only,
// never tensor cores) in the frozen prefill order (V=2, L=1, P=2): every output keeps two
// accumulation chains per K segment, one over the even k and one over the odd k, each strictly
// ascending; they are added once at the end of the segment, segments are summed in ascending order
// and the bias comes last.  The two chains of an output are exactly the two halves of one packed
// FP32x2 accumulator, so one fma.rn.f32x2 advances both chains by one element each, with the
// operands (x[m,k], x[m,k+1]) and (up(W[n,k]), up(W[n,k+1])) taken as they lie in memory.
//
// Schedule (numerically inert): 128 x 128 output tile per block, 256 threads, 8 x 8 outputs per
// thread, K walked in slabs of 32.  BF16 weights are widened to FP32 once per block while the slab
// is staged into shared memory (so HBM and L2 only ever carry BF16 weights, Eq. 2), activations are
// staged as they are.  Global loads of slab i+1 are in flight while slab i is multiplied.
#include "internal.h"
#include "device_utils.cuh"

namespace detlin {

namespace {

constexpr int BM = 128, BN = 128, BK = 32;
constexpr int kThreads = 256;
constexpr int kPitch = 129;                        // 16-byte chunks per k-quad row (odd: conflict-free staging)
constexpr int kQuads = BK / 4;                     // k-quads per slab
constexpr int kTileChunks = kQuads * kPitch;       // 16-byte chunks per operand tile
constexpr int kSmemBytes = 2 /*buffers*/ * 2 /*operands*/ * kTileChunks * 16;

__device__ __forceinline__ float4 lds128(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, float4 v)
{
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ uint4 ldg128_nc(const void* p)
{
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__global__ void __launch_bounds__(kThreads, 1)
prefill_kernel(const float* __restrict__ x, const uint16_t* __restrict__ W, const float* __restrict__ bias,
               float* __restrict__ out, int M, int N, int K, int seg_len, int S, int direct, int tiles_m, int tiles_n)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const uint32_t smem = (uint32_t)__cvta_generic_to_shared(smem_raw);
    // buffer b: x tile at smem + b*2*T, w tile at smem + (b*2+1)*T, T = kTileChunks*16 bytes
    constexpr uint32_t T = kTileChunks * 16;

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;

    // block -> (m tile fastest, then n tile, then segment)
    long long u = blockIdx.x;
    const int tm = (int)(u % tiles_m);
    u /= tiles_m;
    const int tn = (int)(u % tiles_n);
    const int s = (int)(u / tiles_n);
    const int m0 = tm * BM, n0 = tn * BN;
    const int k_lo = s * seg_len;
    const int k_hi = min(K, k_lo + seg_len);

    // ---- staging assignment ----
    // x tile: 128 rows x 8 quads = 1024 chunks, 4 per thread: chunk p = tid + 256 j -> row p / 8, quad p % 8
    // w tile: 128 rows x 4 octets (8 BF16 = 16 bytes) = 512 pieces, 2 per thread: p = tid + 256 j -> row p / 4, octet p % 4
    const float* xg[4];
    uint32_t xs_off[4];
    bool xok[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int p = tid + 256 * j;
        const int r = p >> 3, q = p & 7;
        const int m = m0 + r;
        xok[j] = m < M;
        xg[j] = x + (long long)(xok[j] ? m : 0) * K + q * 4;
        xs_off[j] = (uint32_t)(q * kPitch + r) * 16;
    }
    const uint16_t* wg[2];
    uint32_t ws_off[2];
    bool wok[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int p = tid + 256 * j;
        const int r = p >> 2, o = p & 3;
        const int n = n0 + r;
        wok[j] = n < N;
        wg[j] = W + (long long)(wok[j] ? n : 0) * K + o * 8;
        ws_off[j] = (uint32_t)((2 * o) * kPitch + r) * 16;
    }

    float4 xr[4];
    uint4 wr[2];
    auto load_slab = [&](int k0) {
        // K % 8 == 0: an octet of weights / a quad of activations is entirely inside or outside [.., k_hi)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int q = (tid + 256 * j) & 7;
            if (xok[j] && k0 + q * 4 < k_hi) {
                const uint4 t = ldg128_nc(xg[j] + k0);
                xr[j] = make_float4(__uint_as_float(t.x), __uint_as_float(t.y), __uint_as_float(t.z), __uint_as_float(t.w));
            } else {
                xr[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int o = (tid + 256 * j) & 3;
            if (wok[j] && k0 + o * 8 < k_hi) wr[j] = ldg128_nc(wg[j] + k0);
            else wr[j] = make_uint4(0u, 0u, 0u, 0u);
        }
    };
    auto store_slab = [&](int buf) {
        const uint32_t xb = smem + (uint32_t)(buf * 2) * T, wb = xb + T;
#pragma unroll
        for (int j = 0; j < 4; ++j) sts128(xb + xs_off[j], xr[j]);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            // widen the eight BF16 weights to FP32 (exact): quad 2o holds k..k+3, quad 2o+1 holds k+4..k+7
            sts128(wb + ws_off[j], make_float4(up_lo(wr[j].x), up_hi(wr[j].x), up_lo(wr[j].y), up_hi(wr[j].y)));
            sts128(wb + ws_off[j] + kPitch * 16, make_float4(up_lo(wr[j].z), up_hi(wr[j].z), up_lo(wr[j].w), up_hi(wr[j].w)));
        }
    };

    float2 acc[8][8];        // [i][j] -> output (m0 + ty + 16 i, n0 + tx + 16 j): (even-k chain, odd-k chain)
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = make_float2(0.0f, 0.0f);

    load_slab(k_lo);
    store_slab(0);
    __syncthreads();

    int buf = 0;
    for (int k0 = k_lo; k0 < k_hi; k0 += BK) {
        const bool more = k0 + BK < k_hi;
        if (more) load_slab(k0 + BK);
        const uint32_t xb = smem + (uint32_t)(buf * 2) * T + (uint32_t)ty * 16;
        const uint32_t wb = smem + (uint32_t)(buf * 2 + 1) * T + (uint32_t)tx * 16;
        // k beyond the end of the segment is skipped, not zero-filled: only whole valid quads run
        const int nq = min(kQuads, (k_hi - k0) >> 2);
#pragma unroll 2
        for (int q = 0; q < nq; ++q) {
            float4 xf[8], wf[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) xf[i] = lds128(xb + (uint32_t)(q * kPitch + 16 * i) * 16);
#pragma unroll
            for (int j = 0; j < 8; ++j) wf[j] = lds128(wb + (uint32_t)(q * kPitch + 16 * j) * 16);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float2 xa = make_float2(xf[i].x, xf[i].y);
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = __ffma2_rn(xa, make_float2(wf[j].x, wf[j].y), acc[i][j]);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float2 xc = make_float2(xf[i].z, xf[i].w);
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = __ffma2_rn(xc, make_float2(wf[j].z, wf[j].w), acc[i][j]);
            }
        }
        if (more) store_slab(buf ^ 1);
        __syncthreads();
        buf ^= 1;
    }

    // ---- epilogue: even + odd chain, then bias (direct) or the segment's partial ----
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int m = m0 + ty + 16 * i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int n = n0 + tx + 16 * j;
            if (n >= N) continue;
            float t = __fadd_rn(acc[i][j].x, acc[i][j].y);
            if (direct) {
                if (bias) t = __fadd_rn(t, bias[n]);
                out[(long long)m * N + n] = t;
            } else {
                out[((long long)s * M + m) * N + n] = t;
            }
        }
    }
}

}  // namespace

cudaError_t launch_prefill(const LaunchArgs& a)
{
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(prefill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const int tiles_m = (int)((a.M + BM - 1) / BM), tiles_n = (int)((a.N + BN - 1) / BN);
    const long long units = (long long)tiles_m * tiles_n * a.S;
    if (units > 0x7fffffffLL) return cudaErrorInvalidValue;
    const int direct = (a.S == 1);
    prefill_kernel<<<(unsigned)units, kThreads, kSmemBytes, a.stream>>>(a.x, a.W, a.b, direct ? a.y : a.partials, (int)a.M,
                                                                        (int)a.N, (int)a.K, (int)a.seg_len, a.S, direct,
                                                                        tiles_m, tiles_n);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (!direct) return launch_combine(a);
    return cudaSuccess;
}

}  // namespace detlin
