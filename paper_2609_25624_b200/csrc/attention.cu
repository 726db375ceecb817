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
// Schedule (numerically inert): a cluster of C thread blocks (C = 1, 2, 4, 8 or 16) per (batch, KV head) serves
// the G = Hq / Hkv query heads that share the head's keys and values, so K and V cross the memory bus once
// per group.  Block r of the cluster owns the keys [r Tc, (r + 1) Tc), Tc a whole number of 256-key
// segments; everything that crosses the blocks goes through distributed shared memory behind hardware
// cluster barriers (no spinning): the exact row maxima (comparisons, order-free), the weights that block 0
// reads to form the denominators in the lane order over ALL keys, and the segment sums that every block
// reads to fold its slice of the outputs in ascending segment order.  C only depends on how many blocks
// fill the GPU and on the shared memory a block may use; every C gives the same bits.
// Inside a block, eight warps: in step 1 a warp takes eight keys at a time and folds the 8 G lane trees into
// one butterfly reduce-scatter (one shuffle per (key, head) instead of five); scores and weights live in
// shared memory; in step 5 a warp owns (segment, slice of d) items, as wide as keeps every warp busy.
#include "internal.h"
#include "device_utils.cuh"
#include <cooperative_groups.h>

namespace detlin {

namespace {

namespace cg = cooperative_groups;

constexpr int kAttnThreads = 256;
constexpr int kAttnWarps = kAttnThreads / 32;
constexpr int kKeysPerPass = 8;          // keys a warp scores together
constexpr int kSegKeys = 256;            // P.V segment length (part of the order)
constexpr int kMaxCluster = 16;          // blocks per row at most (8 is the portable cluster size, 16 needs the opt-in below)

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

// P.V work items of one block (see step 5 of the kernel).  VW = consecutive d per lane (1, 2 or 4; D % 4 == 0, so a
// lane's VW elements are all inside or all outside D).
template <int G, int VW>
__device__ __forceinline__ void pv_items(const float* e_s, float* part, const float* __restrict__ vb, int Tc, int Tl, int D,
                                         int n_seg_l, int warp, int lane)
{
    constexpr int kKeys = (VW == 4) ? 8 : 16;                  // keys loaded together
    const int n_slices = (D + 32 * VW - 1) / (32 * VW);
    for (int item = warp; item < n_seg_l * n_slices; item += kAttnWarps) {
        const int sgm = item / n_slices, d = 32 * VW * (item % n_slices) + VW * lane;
        const bool ok = d < D;
        float acc[G][VW];
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int e = 0; e < VW; ++e) acc[g][e] = 0.0f;
        const int j_lo = sgm * kSegKeys, j_hi = min(Tl, j_lo + kSegKeys);
        const float* vp = vb + (ok ? d : 0);
        for (int j0 = j_lo; j0 < j_hi; j0 += kKeys) {
            float vv[kKeys][VW];
#pragma unroll
            for (int p = 0; p < kKeys; ++p) {
                const float* src = vp + (size_t)(j0 + p) * D;
                const bool in = j0 + p < j_hi && ok;
                if constexpr (VW == 4) {
                    const float4 t = in ? __ldg(reinterpret_cast<const float4*>(src)) : make_float4(0.f, 0.f, 0.f, 0.f);
                    vv[p][0] = t.x; vv[p][1] = t.y; vv[p][2] = t.z; vv[p][3] = t.w;
                } else if constexpr (VW == 2) {
                    const float2 t = in ? __ldg(reinterpret_cast<const float2*>(src)) : make_float2(0.f, 0.f);
                    vv[p][0] = t.x; vv[p][1] = t.y;
                } else {
                    vv[p][0] = in ? __ldg(src) : 0.0f;
                }
            }
#pragma unroll
            for (int p4 = 0; p4 < kKeys; p4 += 4) {
                float4 ew[G];                                    // the weights of four keys (j0 is a multiple of 8)
#pragma unroll
                for (int g = 0; g < G; ++g) ew[g] = *reinterpret_cast<const float4*>(e_s + g * Tc + j0 + p4);
#pragma unroll
                for (int pp = 0; pp < 4; ++pp) {
                    if (j0 + p4 + pp < j_hi) {                   // keys beyond the segment are skipped
#pragma unroll
                        for (int g = 0; g < G; ++g) {
                            const float w = pp == 0 ? ew[g].x : pp == 1 ? ew[g].y : pp == 2 ? ew[g].z : ew[g].w;
#pragma unroll
                            for (int e = 0; e < VW; ++e) acc[g][e] = __fmaf_rn(w, vv[p4 + pp][e], acc[g][e]);
                        }
                    }
                }
            }
        }
        if (ok) {
#pragma unroll
            for (int g = 0; g < G; ++g)
#pragma unroll
                for (int e = 0; e < VW; ++e) part[((size_t)sgm * G + g) * D + d + e] = acc[g][e];
        }
    }
}

// G: query heads per KV head (1, 2, 4 or 8); DC: 128-element chunks of the head dimension (1 or 2).
// Grid (C, B Hkv) in clusters of (C, 1, 1); Tc = keys per block (a multiple of 256), t_pitch = Tc.
template <int G, int DC>
__global__ void __launch_bounds__(kAttnThreads)
attention_decode_kernel(const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v, float scale,
                        int Hq, int Hkv, int T, int D, int Tc, float* __restrict__ o)
{
    extern __shared__ __align__(16) float smem_f[];
    cg::cluster_group cluster = cg::this_cluster();
    const int C = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    // the same layout in every block of the cluster (remote addresses are computed from it)
    const int segs_per_block = Tc / kSegKeys;
    float* e_s = smem_f;                                       // [G][Tc]: scores, then weights, of the block's keys
    float* part = e_s + (size_t)G * Tc;                        // [segs_per_block][G][D]
    float* l_s = part + (size_t)segs_per_block * G * D;        // [8] denominators (block 0)
    float* cmax = l_s + 8;                                     // [8] the block's row maxima
    float* red = cmax + 8;                                     // [kAttnWarps][G]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.y / Hkv, hk = blockIdx.y % Hkv;
    const int j_begin = rank * Tc;                             // first key of this block
    const int Tl = max(0, min(T - j_begin, Tc));               // keys of this block
    const int n_seg = (T + kSegKeys - 1) / kSegKeys;           // segments of the row
    const int n_seg_l = (Tl + kSegKeys - 1) / kSegKeys;        // segments of this block
    const float* qb = q + ((size_t)b * Hq + (size_t)hk * G) * D;
    const float* kb = k + (((size_t)b * Hkv + hk) * (size_t)T + j_begin) * D;
    const float* vb = v + (((size_t)b * Hkv + hk) * (size_t)T + j_begin) * D;
    float* ob = o + ((size_t)b * Hq + (size_t)hk * G) * D;

    // the lane's elements of a row of D floats: d = 128 c + 4 lane + jj (all four inside or outside D: D % 4 == 0)
    bool d_ok[DC];
#pragma unroll
    for (int c = 0; c < DC; ++c) d_ok[c] = 128 * c + 4 * lane < D;

    // ---- step 1: scores of the block's keys ----
    {
        float4 qv[G][DC];
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int c = 0; c < DC; ++c)
                qv[g][c] = d_ok[c] ? __ldg(reinterpret_cast<const float4*>(qb + (size_t)g * D + 128 * c + 4 * lane)) : make_float4(0.f, 0.f, 0.f, 0.f);
        for (int j0 = warp * kKeysPerPass; j0 < Tl; j0 += kAttnWarps * kKeysPerPass) {
            float4 kv[kKeysPerPass][DC];
#pragma unroll
            for (int p = 0; p < kKeysPerPass; ++p)
#pragma unroll
                for (int c = 0; c < DC; ++c)
                    kv[p][c] = (j0 + p < Tl && d_ok[c]) ? __ldg(reinterpret_cast<const float4*>(kb + (size_t)(j0 + p) * D + 128 * c + 4 * lane))
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
                    if (j0 + p < Tl) e_s[g * Tc + j0 + p] = __fmul_rn(a[t], scale);
                }
            }
        }
    }
    __syncthreads();

    // ---- step 2: row maxima (exact): the block's, then the cluster's ----
    {
        float mx[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float m = -INFINITY;
            for (int j = threadIdx.x; j < Tl; j += kAttnThreads) m = fmaxf(m, e_s[g * Tc + j]);
#pragma unroll
            for (int dlt = 16; dlt > 0; dlt >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, dlt));
            mx[g] = m;
        }
        if (lane == 0) {
#pragma unroll
            for (int g = 0; g < G; ++g) red[warp * G + g] = mx[g];
        }
        __syncthreads();
        if (threadIdx.x < G) {
            float m = red[threadIdx.x];
            for (int w = 1; w < kAttnWarps; ++w) m = fmaxf(m, red[w * G + threadIdx.x]);
            cmax[threadIdx.x] = m;
        }
        cluster.sync();
        // ---- step 3: weights of the block's keys ----
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float m = cmax[g];
            for (int r = 0; r < C; ++r)
                if (r != rank) m = fmaxf(m, cluster.map_shared_rank(cmax, r)[g]);
            for (int j = threadIdx.x; j < Tl; j += kAttnThreads) {
                const float s = e_s[g * Tc + j];
                e_s[g * Tc + j] = exp_det(__fsub_rn(s, m));
            }
        }
    }
    cluster.sync();                                            // every block's weights are in place

    // ---- step 4 (block 0): denominators, one warp per head; the 32 chains of a sum are the warp's lanes and
    // run over ALL keys in ascending chunks of 128, reading the other blocks' weights in place ----
    if (rank == 0) {
        for (int g = warp; g < G; g += kAttnWarps) {
            float a = 0.0f;
            for (int c0 = 0; c0 < T; c0 += Tc) {               // owner block c0 / Tc
                const float* er = cluster.map_shared_rank(e_s, c0 / Tc) + g * Tc;
                const int t_hi = min(T - c0, Tc);
                for (int c = 0; c < t_hi; c += 128) {
                    const int j = c + 4 * lane;
                    if (j + 3 < t_hi) {
                        const float4 ev = *reinterpret_cast<const float4*>(er + j);
                        a = __fadd_rn(a, ev.x);
                        a = __fadd_rn(a, ev.y);
                        a = __fadd_rn(a, ev.z);
                        a = __fadd_rn(a, ev.w);
                    } else {
#pragma unroll
                        for (int jj = 0; jj < 4; ++jj)
                            if (j + jj < t_hi) a = __fadd_rn(a, er[j + jj]);
                    }
                }
            }
            a = lane_tree_sum(a);
            if (lane == 0) l_s[g] = a;
        }
    }

    // ---- step 5: P.V.  A work item is (256-key segment of the block, slice of 32 VW consecutive d): a lane owns VW
    // consecutive d and runs their G chains a = fma(e_j, v_j[d], a) over the segment's keys in ascending order.
    // Items are dealt to the warps round robin; the slices are as wide as still leaves every warp an item, so a
    // block with two segments keeps all eight warps loading and a block with many uses 16-byte loads ----
    if (n_seg_l * ((D + 127) / 128) >= kAttnWarps) pv_items<G, 4>(e_s, part, vb, Tc, Tl, D, n_seg_l, warp, lane);
    else if (n_seg_l * ((D + 63) / 64) >= kAttnWarps) pv_items<G, 2>(e_s, part, vb, Tc, Tl, D, n_seg_l, warp, lane);
    else pv_items<G, 1>(e_s, part, vb, Tc, Tl, D, n_seg_l, warp, lane);
    cluster.sync();                                            // segment sums and denominators are in place

    // ---- fold the segment sums in ascending order, divide: block r takes the r-th slice of the G D outputs ----
    {
        const int per = (G * D + C - 1) / C;
        const int i_lo = rank * per, i_hi = min(G * D, i_lo + per);
        const float* l0 = cluster.map_shared_rank(l_s, 0);
        for (int i = i_lo + (int)threadIdx.x; i < i_hi; i += kAttnThreads) {
            const int g = i / D;
            float t = cluster.map_shared_rank(part, 0)[i];
            for (int sgm = 1; sgm < n_seg; ++sgm)
                t = __fadd_rn(t, cluster.map_shared_rank(part, sgm / segs_per_block)[(size_t)(sgm % segs_per_block) * G * D + i]);
            ob[i] = __fdiv_rn(t, l0[g]);
        }
    }
    cluster.sync();                                            // nobody leaves while its shared memory may still be read
}

int g_attention_force_split = 0;        // test hook: 0 = automatic, else the cluster size to use (1, 2, 4, 8)

// shared memory of one block that owns Tc keys
size_t block_smem_bytes(int G, int Tc, int D)
{
    return 4 * ((size_t)G * Tc + (size_t)(Tc / kSegKeys) * G * D + 8 + 8 + (size_t)kAttnWarps * G);
}

// keys per block for a cluster of C blocks: the row's 256-key segments dealt out in equal whole numbers
int keys_per_block(int T, int C)
{
    const int n_seg = (T + kSegKeys - 1) / kSegKeys;
    return (n_seg + C - 1) / C * kSegKeys;
}

template <int G, int DC>
cudaError_t launch_attention_t(const float* q, const float* k, const float* v, float scale, int B, int Hq, int Hkv, int T, int D,
                               float* o, size_t smem, int C, int Tc, cudaStream_t stream)
{
    static bool configured[kMaxDevices];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    auto kern = attention_decode_kernel<G, DC>;
    if (!configured[dev]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);   // clusters of 16
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1];
    for (;;) {
        cfg.gridDim = dim3((unsigned)C, (unsigned)(B * Hkv));
        cfg.blockDim = dim3(kAttnThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)C;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        // a cluster this large may not fit where the stream runs (few SMs, a partition): halve it while the scores
        // of a block still fit (schedule only: same bits)
        int n_clusters = 0;
        e = cudaOccupancyMaxActiveClusters(&n_clusters, kern, &cfg);
        if (e == cudaSuccess && n_clusters >= 1) break;
        cudaGetLastError();
        if (C == 1) return e != cudaSuccess ? e : cudaErrorLaunchOutOfResources;
        C /= 2;
        Tc = keys_per_block(T, C);
        smem = block_smem_bytes(G, Tc, D);
        if (smem > 227u * 1024u) return cudaErrorLaunchOutOfResources;
    }
    return cudaLaunchKernelEx(&cfg, kern, q, k, v, scale, Hq, Hkv, T, D, Tc, o);
}

}  // namespace

// Cluster size for a shape: the largest power of two that still lets all blocks be resident at once (two blocks of
// 256 threads per SM: one wave, measured best at about 256 blocks on 148 SMs), never more blocks than the row has
// segments, and at least as many as it takes for a block's scores and segment sums to fit in the shared memory
// that lets two blocks share an SM (or in a block's maximum, if that is all that fits).  Schedule only.
int attention_split(int B, int Hkv, int G, int T, int D, int sm_count)
{
    const int n_seg = (T + kSegKeys - 1) / kSegKeys;
    int c_max = 1;
    while (c_max < kMaxCluster && 2 * c_max <= n_seg) c_max *= 2;
    if (g_attention_force_split) return g_attention_force_split <= c_max ? g_attention_force_split : c_max;
    // clusters of 16 (not portable, one GPC each) only pay for very few, very long rows (measured: 8 rows of 16384 keys
    // or more; 16 rows, or 4096 keys, are faster in clusters of 8)
    const bool few_long_rows = (long long)B * Hkv * 16 <= sm_count && n_seg >= 64;
    const int c_auto = (c_max > 8 && !few_long_rows) ? 8 : c_max;
    int c = 1;
    while (c < c_auto && (long long)B * Hkv * (2 * c) <= 2ll * sm_count) c *= 2;
    while (c < c_max && block_smem_bytes(G, keys_per_block(T, c), D) > 110u * 1024u) c *= 2;
    return c;
}

// Dynamic shared memory of a block for the most finely split schedule the shape allows (the least the shape needs).
size_t attention_smem_bytes(int G, int T, int D)
{
    const int n_seg = (T + kSegKeys - 1) / kSegKeys;
    int c_max = 1;
    while (c_max < kMaxCluster && 2 * c_max <= n_seg) c_max *= 2;
    return block_smem_bytes(G, keys_per_block(T, c_max), D);
}

size_t attention_block_smem_bytes(int G, int T, int D, int C) { return block_smem_bytes(G, keys_per_block(T, C), D); }

void attention_test_force_split(int c) { g_attention_force_split = (c == 1 || c == 2 || c == 4 || c == 8 || c == 16) ? c : 0; }

cudaError_t launch_attention_decode(const float* q, const float* k, const float* v, float scale, int B, int Hq, int Hkv, int T, int D,
                                    float* o, cudaStream_t stream)
{
    const int G = Hq / Hkv;
    const int dc = (D + 127) / 128;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        sms = 148;
    int C = attention_split(B, Hkv, G, T, D, sms);
    while (C < kMaxCluster && block_smem_bytes(G, keys_per_block(T, C), D) > 227u * 1024u) C *= 2;   // must fit at all
    const int Tc = keys_per_block(T, C);
    const size_t smem = block_smem_bytes(G, Tc, D);
    if (smem > 227u * 1024u) return cudaErrorInvalidValue;
#define DET_ATTN(GG, DD) return launch_attention_t<GG, DD>(q, k, v, scale, B, Hq, Hkv, T, D, o, smem, C, Tc, stream)
    if (dc == 1) {
        switch (G) { case 1: DET_ATTN(1, 1); case 2: DET_ATTN(2, 1); case 4: DET_ATTN(4, 1); case 8: DET_ATTN(8, 1); default: break; }
    } else if (dc == 2) {
        switch (G) { case 1: DET_ATTN(1, 2); case 2: DET_ATTN(2, 2); case 4: DET_ATTN(4, 2); case 8: DET_ATTN(8, 2); default: break; }
    }
#undef DET_ATTN
    return cudaErrorInvalidValue;
}

}  // namespace detlin
