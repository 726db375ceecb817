// Fixed-order decode attention: one query row per (batch, head) against T cached keys and values.
// Not one of the paper's kernels: the paper keeps vendor attention and names fixed-order attention as the
// outstanding source of residual divergence between GPU architectures.  Here every reduction of the
// attention runs in an order fixed by (T, D) alone, every step one IEEE-754 binary32 operation, so the
// bits do not depend on the batch size, the grid, the SM count or the stream:
//
//   1. s_j = dot(q, k_j) * scale; the dot product in the decode lane order over D (chunks of 128 ascending,
//      lane l owns the 4 consecutive elements c + 4 l + jj, one fma.rn per element from +0, elements
//      beyond D skipped, the 32 lane sums added adjacent-first: xor 1, 2, 4, 8, 16), then one multiply;
//   2. m = max_j s_j (comparisons only);
//   3. e_j = exp_det(s_j - m): one subtraction and the fixed-sequence exponential below;
//   4. l = sum_j e_j in the lane order over j (chunks of 128 keys ascending, lane l owns keys c + 4 l + jj,
//      one add.rn per key from +0, keys beyond T skipped, adjacent-first lane tree);
//   5. for every d: keys in segments of 256; inside a segment a = fma.rn(e_j, v_j[d], a) from +0 with j
//      ascending; segment sums added left to right in ascending order; o[d] = sum / l (one div.rn).
//
// Schedule (numerically inert): one thread block per (batch, KV head) serves the G = Hq / Hkv query
// heads that share the head's keys and values, so K and V cross the memory bus once per group.  Eight
// warps: in step 1 a warp takes eight keys at a time and folds the 8 G lane trees into one butterfly
// reduce-scatter (one shuffle per (key, head) instead of five); scores and weights live in shared memory;
// in step 5 a warp owns whole 256-key segments and a lane four consecutive d.
#include "internal.h"
#include "device_utils.cuh"

namespace detlin {

namespace {

constexpr int kAttnThreads = 256;
constexpr int kAttnWarps = kAttnThreads / 32;
constexpr int kKeysPerPass = 8;          // keys a warp scores together
constexpr int kSegKeys = 256;            // P.V segment length (part of the order)

// The attention's exponential for x <= 0: range reduction by ln 2 in two pieces, degree-7 Taylor polynomial
// by Horner's rule with fused multiply-adds, scaling by 2^n (through 2^(n+64) and 2^-64 below the normal
// range).  Every step is one explicitly rounded binary32 operation; the constants are given by bit pattern.
__device__ __forceinline__ float exp_det(float x)
{
    if (x < -104.0f) return 0.0f;
    const float t = __fmul_rn(x, __uint_as_float(0x3FB8AA3Bu));               // log2(e)
    const float n = rintf(t);                                                // nearest, ties to even
    float f = __fmaf_rn(n, -__uint_as_float(0x3F317200u), x);                // ln 2, high part
    f = __fmaf_rn(n, -__uint_as_float(0x35BFBE8Eu), f);                      // ln 2, low part
    float p = __uint_as_float(0x39500D01u);                                  // 1/5040
    p = __fmaf_rn(p, f, __uint_as_float(0x3AB60B61u));                       // 1/720
    p = __fmaf_rn(p, f, __uint_as_float(0x3C088889u));                       // 1/120
    p = __fmaf_rn(p, f, __uint_as_float(0x3D2AAAABu));                       // 1/24
    p = __fmaf_rn(p, f, __uint_as_float(0x3E2AAAABu));                       // 1/6
    p = __fmaf_rn(p, f, 0.5f);
    p = __fmaf_rn(p, f, 1.0f);
    p = __fmaf_rn(p, f, 1.0f);
    const int ni = (int)n;
    if (ni >= -126) return __fmul_rn(p, __uint_as_float((uint32_t)(ni + 127) << 23));
    const float u = __fmul_rn(p, __uint_as_float((uint32_t)(ni + 64 + 127) << 23));
    return __fmul_rn(u, __uint_as_float((uint32_t)(-64 + 127) << 23));
}

// Butterfly reduce-scatter that realises the adjacent-first lane tree for NV values per lane at once.  At
// step i (i = 0..4) lanes l and l ^ (1 << i) are partners.  While the number of values a lane holds is
// even, the partners exchange halves and add (the lane with bit i set keeps the upper half), so the work
// per step halves; afterwards the remaining steps add whole arrays.  kSteps = number of halving steps,
// kKeep = values a lane holds at the end (v[0 .. kKeep)); they are the sums of the values with index
// base + t, base = sum over halving steps i of bit_i(lane) * (NV >> (i + 1)); lanes whose bits
// kSteps .. 4 are zero hold distinct results.
template <int NV>
struct Scatter {
    static constexpr int steps()
    {
        int n = NV, h = 0;
        while (h < 5 && n % 2 == 0) { n /= 2; ++h; }
        return h;
    }
    static constexpr int kSteps = steps();
    static constexpr int kKeep = NV >> kSteps;
};

template <int NV>
__device__ __forceinline__ void lane_tree_scatter(float (&v)[NV], int lane)
{
    constexpr int H = Scatter<NV>::kSteps;
    int n = NV;
#pragma unroll
    for (int i = 0; i < 5; ++i) {
        const int d = 1 << i;
        if (i < H) {
            const int half = n >> 1;
            const bool hi = (lane >> i) & 1;
#pragma unroll
            for (int t = 0; t < NV / 2; ++t) {
                if (t < half) {
                    const float send = hi ? v[t] : v[t + half];
                    const float keep = hi ? v[t + half] : v[t];
                    v[t] = __fadd_rn(keep, __shfl_xor_sync(0xffffffffu, send, d));
                }
            }
            n = half;
        } else {
#pragma unroll
            for (int t = 0; t < Scatter<NV>::kKeep; ++t) v[t] = __fadd_rn(v[t], __shfl_xor_sync(0xffffffffu, v[t], d));
        }
    }
}

// G: query heads per KV head (1, 2, 4 or 8); DC: 128-element chunks of the head dimension (1 or 2).
template <int G, int DC>
__global__ void __launch_bounds__(kAttnThreads)
attention_decode_kernel(const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v, float scale,
                        int Hq, int Hkv, int T, int D, int t_pitch, float* __restrict__ o)
{
    extern __shared__ __align__(16) float smem_f[];
    float* e_s = smem_f;                                       // [G][t_pitch]: scores, then weights
    const int n_seg = (T + kSegKeys - 1) / kSegKeys;
    float* part = e_s + G * t_pitch;                           // [n_seg][G][D]
    float* l_s = part + (size_t)n_seg * G * D;                 // [G]
    float* red = l_s + 8;                                      // [kAttnWarps][G]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.x / Hkv, hk = blockIdx.x % Hkv;
    const float* qb = q + ((size_t)b * Hq + (size_t)hk * G) * D;
    const float* kb = k + ((size_t)b * Hkv + hk) * (size_t)T * D;
    const float* vb = v + ((size_t)b * Hkv + hk) * (size_t)T * D;
    float* ob = o + ((size_t)b * Hq + (size_t)hk * G) * D;

    // the lane's elements of a row of D floats: d = 128 c + 4 lane + jj (all four inside or outside D: D % 4 == 0)
    bool d_ok[DC];
#pragma unroll
    for (int c = 0; c < DC; ++c) d_ok[c] = 128 * c + 4 * lane < D;

    // ---- step 1: scores ----
    {
        float4 qv[G][DC];
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int c = 0; c < DC; ++c)
                qv[g][c] = d_ok[c] ? __ldg(reinterpret_cast<const float4*>(qb + (size_t)g * D + 128 * c + 4 * lane)) : make_float4(0.f, 0.f, 0.f, 0.f);
        for (int j0 = warp * kKeysPerPass; j0 < T; j0 += kAttnWarps * kKeysPerPass) {
            float4 kv[kKeysPerPass][DC];
#pragma unroll
            for (int p = 0; p < kKeysPerPass; ++p)
#pragma unroll
                for (int c = 0; c < DC; ++c)
                    kv[p][c] = (j0 + p < T && d_ok[c]) ? __ldg(reinterpret_cast<const float4*>(kb + (size_t)(j0 + p) * D + 128 * c + 4 * lane))
                                                       : make_float4(0.f, 0.f, 0.f, 0.f);
            float a[kKeysPerPass * G];                          // value index p * G + g
#pragma unroll
            for (int p = 0; p < kKeysPerPass; ++p)
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    float acc = 0.0f;
#pragma unroll
                    for (int c = 0; c < DC; ++c) {
                        if (d_ok[c]) {                           // elements beyond D are skipped, not zero-filled
                            acc = __fmaf_rn(qv[g][c].x, kv[p][c].x, acc);
                            acc = __fmaf_rn(qv[g][c].y, kv[p][c].y, acc);
                            acc = __fmaf_rn(qv[g][c].z, kv[p][c].z, acc);
                            acc = __fmaf_rn(qv[g][c].w, kv[p][c].w, acc);
                        }
                    }
                    a[p * G + g] = acc;
                }
            lane_tree_scatter<kKeysPerPass * G>(a, lane);
            constexpr int NV = kKeysPerPass * G;
            constexpr int kSteps = Scatter<NV>::kSteps, kKeep = Scatter<NV>::kKeep;
            int base = 0;
            {
                int n = NV;
#pragma unroll
                for (int i = 0; i < kSteps; ++i) { n >>= 1; base += ((lane >> i) & 1) * n; }
            }
            if ((lane >> kSteps) == 0) {
#pragma unroll
                for (int t = 0; t < kKeep; ++t) {
                    const int idx = base + t, p = idx / G, g = idx % G;
                    if (j0 + p < T) e_s[g * t_pitch + j0 + p] = __fmul_rn(a[t], scale);
                }
            }
        }
    }
    __syncthreads();

    // ---- step 2: row maxima (exact) ----
    {
        float mx[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float m = -INFINITY;
            for (int j = threadIdx.x; j < T; j += kAttnThreads) m = fmaxf(m, e_s[g * t_pitch + j]);
#pragma unroll
            for (int dlt = 16; dlt > 0; dlt >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, dlt));
            mx[g] = m;
        }
        if (lane == 0) {
#pragma unroll
            for (int g = 0; g < G; ++g) red[warp * G + g] = mx[g];
        }
        __syncthreads();
        // ---- step 3: weights ----
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float m = red[g];
#pragma unroll
            for (int w = 1; w < kAttnWarps; ++w) m = fmaxf(m, red[w * G + g]);
            for (int j = threadIdx.x; j < T; j += kAttnThreads) {
                const float s = e_s[g * t_pitch + j];
                e_s[g * t_pitch + j] = exp_det(__fsub_rn(s, m));
            }
        }
    }
    __syncthreads();

    // ---- step 4: denominators, one warp per head (the 32 chains of a sum are one warp's lanes) ----
    for (int g = warp; g < G; g += kAttnWarps) {
        float a = 0.0f;
        for (int c = 0; c < T; c += 128) {
            const int j = c + 4 * lane;
            if (j + 3 < T) {
                const float4 ev = *reinterpret_cast<const float4*>(e_s + g * t_pitch + j);
                a = __fadd_rn(a, ev.x);
                a = __fadd_rn(a, ev.y);
                a = __fadd_rn(a, ev.z);
                a = __fadd_rn(a, ev.w);
            } else {
#pragma unroll
                for (int jj = 0; jj < 4; ++jj)
                    if (j + jj < T) a = __fadd_rn(a, e_s[g * t_pitch + j + jj]);
            }
        }
        a = lane_tree_sum(a);
        if (lane == 0) l_s[g] = a;
    }

    // ---- step 5: P.V, a warp per 256-key segment, a lane per four consecutive d ----
    for (int sgm = warp; sgm < n_seg; sgm += kAttnWarps) {
        float4 acc[G][DC];
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int c = 0; c < DC; ++c) acc[g][c] = make_float4(0.f, 0.f, 0.f, 0.f);
        const int j_lo = sgm * kSegKeys, j_hi = min(T, j_lo + kSegKeys);
        for (int j0 = j_lo; j0 < j_hi; j0 += 8) {
            float4 vv[8][DC];
#pragma unroll
            for (int p = 0; p < 8; ++p)
#pragma unroll
                for (int c = 0; c < DC; ++c)
                    vv[p][c] = (j0 + p < j_hi && d_ok[c]) ? __ldg(reinterpret_cast<const float4*>(vb + (size_t)(j0 + p) * D + 128 * c + 4 * lane))
                                                          : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int p = 0; p < 8; ++p) {
                if (j0 + p < j_hi) {                             // keys beyond the segment are skipped
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const float w = e_s[g * t_pitch + j0 + p];
#pragma unroll
                        for (int c = 0; c < DC; ++c) {
                            acc[g][c].x = __fmaf_rn(w, vv[p][c].x, acc[g][c].x);
                            acc[g][c].y = __fmaf_rn(w, vv[p][c].y, acc[g][c].y);
                            acc[g][c].z = __fmaf_rn(w, vv[p][c].z, acc[g][c].z);
                            acc[g][c].w = __fmaf_rn(w, vv[p][c].w, acc[g][c].w);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int c = 0; c < DC; ++c)
                if (d_ok[c]) *reinterpret_cast<float4*>(part + ((size_t)sgm * G + g) * D + 128 * c + 4 * lane) = acc[g][c];
    }
    __syncthreads();

    // ---- fold the segment sums in ascending order, divide ----
    for (int i = threadIdx.x; i < G * D; i += kAttnThreads) {
        const int g = i / D;
        float t = part[i];
        for (int sgm = 1; sgm < n_seg; ++sgm) t = __fadd_rn(t, part[(size_t)sgm * G * D + i]);
        ob[i] = __fdiv_rn(t, l_s[g]);
    }
}

template <int G, int DC>
cudaError_t launch_attention_t(const float* q, const float* k, const float* v, float scale, int B, int Hq, int Hkv, int T, int D,
                               float* o, size_t smem, int t_pitch, cudaStream_t stream)
{
    static bool configured[kMaxDevices];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    auto kern = attention_decode_kernel<G, DC>;
    if (!configured[dev]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    kern<<<(unsigned)(B * Hkv), kAttnThreads, smem, stream>>>(q, k, v, scale, Hq, Hkv, T, D, t_pitch, o);
    return cudaGetLastError();
}

}  // namespace

size_t attention_smem_bytes(int G, int T, int D)
{
    const size_t t_pitch = ((size_t)T + 3) / 4 * 4;
    const size_t n_seg = ((size_t)T + kSegKeys - 1) / kSegKeys;
    return 4 * ((size_t)G * t_pitch + n_seg * G * D + 8 + (size_t)kAttnWarps * G);
}

cudaError_t launch_attention_decode(const float* q, const float* k, const float* v, float scale, int B, int Hq, int Hkv, int T, int D,
                                    float* o, cudaStream_t stream)
{
    const int G = Hq / Hkv;
    const int dc = (D + 127) / 128;
    const int t_pitch = (T + 3) / 4 * 4;
    const size_t smem = attention_smem_bytes(G, T, D);
#define DET_ATTN(GG, DD) return launch_attention_t<GG, DD>(q, k, v, scale, B, Hq, Hkv, T, D, o, smem, t_pitch, stream)
    if (dc == 1) {
        switch (G) { case 1: DET_ATTN(1, 1); case 2: DET_ATTN(2, 1); case 4: DET_ATTN(4, 1); case 8: DET_ATTN(8, 1); default: break; }
    } else if (dc == 2) {
        switch (G) { case 1: DET_ATTN(1, 2); case 2: DET_ATTN(2, 2); case 4: DET_ATTN(4, 2); case 8: DET_ATTN(8, 2); default: break; }
    }
#undef DET_ATTN
    return cudaErrorInvalidValue;
}

}  // namespace detlin
