// Prefill kernel (bucket M > 64): register-tiled FP32 GEMM on the CUDA cores (rule R1:
// IEEE FMA only, never tensor cores) in the frozen prefill order (V=1, L=1, P=1): every output is one
// accumulation chain per K segment, strictly ascending in k; segments are summed in ascending order and
// the bias comes last (rule R3).
//
// One packed fma.rn.f32x2 advances the chains of two neighbouring output columns (n, n+1) of the same row
// by one element; each half is an ordinary fma.rn.f32, so the pairing is invisible in the bits.
//
// What bounds this loop on B200 (measured): a scheduler issues one instruction every other cycle while the
// packed FMA, which occupies the pipe for two cycles, dominates, so every instruction that is not a packed
// FMA costs an FMA slot.  The sustained fraction of the FP32 peak is therefore the share of packed FMAs in
// the instruction stream, and the schedule below exists to keep everything else out of it:
//   * 8 x 8 outputs per thread: four 16-byte shared loads per 32 packed FMAs;
//   * a thread wants its eight activations of one k in two 16-byte loads, which needs the tile k-major in
//     shared memory.  A small first kernel transposes x into a workspace xT [K][M]; TMA brings tiles
//     [32 k][16 TR rows] of it to shared memory.  No thread spends registers, loads, stores, address
//     arithmetic or bounds checks on staging activations, and the multiply loop keeps few values live (the
//     128-register budget of two blocks per SM otherwise forces the compiler to recompute addresses);
//   * the weight tile arrives by TMA too, in its stored format; it has to become FP32 (Eq. 2: the
//     upcast is exact) and k-major, so that one 16-byte load yields two (n, n+1) operand pairs.  Each thread
//     converts 16 weights per slab: one 16-byte shared load, eight widenings and eight stores, twice.  TMA
//     fills out-of-range rows and columns with zeros, so there are no bounds checks;
//   * all shared-memory offsets of the multiply loop are immediates (the loop over a slab is unrolled).
// Schedule (numerically inert): 256 threads, block tile 16 TR rows x 128 columns (TR = 5 .. 8 rows per
// thread, whichever pads the batch least), two blocks per SM, K walked in slabs of 32; two activation
// stages, two raw weight stages, two converted weight buffers, all indexed by the parity of the slab.  One block-wide barrier per slab orders the
// converted buffers and frees the stages that were just read, which one thread then refills through TMA.
//
// Every wait on a TMA completion is bounded: a wait that expires records the fact in the device status
// word and the block returns without storing.
#include "internal.h"
#include "device_utils.cuh"
#include "pipeline_utils.cuh"
#include <type_traits>

namespace detlin {

namespace {

using namespace pipe;

constexpr int BN = 128, BK = 32;
constexpr int kThreads = 256;
constexpr int kXStages = 2;                          // activation stages (slab parity)
// raw weight stage: [128 rows][32 k] in the stored format (64-byte rows for 16-bit weights, 128-byte rows for FP32)
template <int WF> struct Raw { static constexpr int kBytes = BN * BK * WeightElem<WF>::bytes; };
constexpr int kWfBytes = BK * BN * 4;                // converted weight buffer: [32 k][128 n] FP32, columns swizzled

template <int WF, int TR> struct Tile {
    static constexpr int kRawBytes = Raw<WF>::kBytes;
    static constexpr int BM = 16 * TR;
    static constexpr int kXBytes = BK * BM * 4;      // [32 k][BM rows] FP32
    // stages and buffers, then barriers and the abort word; 128 bytes of slack to align the first stage
    static constexpr int kSmemBytes = kXStages * kXBytes + 2 * kRawBytes + 2 * kWfBytes + 128 + 128;
};

__device__ __forceinline__ void sts32(uint32_t addr, float v)
{
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
// n consecutive floats from shared memory (n <= 4; the address is 4 n-byte aligned for n = 1, 2, 4)
template <int N_>
__device__ __forceinline__ void lds_floats(uint32_t addr, float* v)
{
    if constexpr (N_ == 4) {
        const float4 t = lds128(addr);
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    } else if constexpr (N_ == 2) {
        asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v[0]), "=f"(v[1]) : "r"(addr));
    } else {
#pragma unroll
        for (int i = 0; i < N_; ++i) asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v[i]) : "r"(addr + 4 * i));
    }
}
__device__ __forceinline__ uint4 lds128u(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

template <int WF, int TR>
__global__ void __launch_bounds__(kThreads, 2)
prefill_tma_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                   const float* __restrict__ bias, float* __restrict__ out, int M, int N, int K, int seg_len, int direct,
                   int tiles_m, int tiles_n, long long ldy, DeviceStatus* status, unsigned long long wait_limit_ns,
                   int test_flags, float* __restrict__ y, unsigned* __restrict__ tile_counters, int S)
{
    __shared__ int fold_here;                        // split-K: this block wrote the last partial of its tile
    typedef Tile<WF, TR> T;
    constexpr int kRawBytes = T::kRawBytes;
    constexpr int TB = TR - 4;                       // rows of a thread in the upper group (1 .. 4)
    extern __shared__ unsigned char smem_raw[];
    const uint32_t xring = (smem_u32(smem_raw) + 127u) & ~127u;
    const uint32_t raw0 = xring + kXStages * T::kXBytes;
    const uint32_t wf0 = raw0 + 2 * kRawBytes;
    const uint32_t xfull0 = wf0 + 2 * kWfBytes;
    const uint32_t wfull0 = xfull0 + 8 * kXStages;
    const uint32_t abort_flag = wfull0 + 8 * 2;

    const int tid = threadIdx.x;
    // 16 x 16 threads; a warp = 16 column groups x 2 row groups
    const int tx = tid & 15, ty = tid >> 4;

    // block -> (m tile fastest, then n tile, then segment)
    long long u = blockIdx.x;
    const int tm = (int)(u % tiles_m);
    u /= tiles_m;
    const int tn = (int)(u % tiles_n);
    const int s = (int)(u / tiles_n);
    const int m0 = tm * T::BM, n0 = tn * BN;
    const int k_lo = s * seg_len;
    const int k_hi = min(K, k_lo + seg_len);
    const int n_slabs = (k_hi - k_lo + BK - 1) / BK;

    if (tid == 0) {
        for (int i = 0; i < kXStages; ++i) mbar_init(xfull0 + 8 * i, 1);
        for (int i = 0; i < 2; ++i) mbar_init(wfull0 + 8 * i, 1);
        sts_volatile_i32(abort_flag, 0);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    auto fill_x = [&](int slab) {                     // one thread: the activation tile of a slab into its stage
        const int st = slab % kXStages;
        mbar_arrive_expect_tx(xfull0 + 8 * st, T::kXBytes);
        tma_load_2d_plain(xring + (uint32_t)st * T::kXBytes, &map_x, m0, k_lo + slab * BK, xfull0 + 8 * st);
    };
    auto fill_w = [&](int slab) {                     // one thread: the raw weight tile of a slab into its stage
        const int st = slab & 1;
        mbar_arrive_expect_tx(wfull0 + 8 * st, kRawBytes);
        tma_load_2d_plain(raw0 + (uint32_t)st * kRawBytes, &map_w, k_lo + slab * BK, n0, wfull0 + 8 * st);
    };
    if (tid == 0) {
        // (test hook: block 0 never requests its first activation tile, so its first wait expires)
        for (int i = ((test_flags & 1) && blockIdx.x == 0) ? 1 : 0; i < kXStages && i < n_slabs; ++i) fill_x(i);
        for (int i = 0; i < 2 && i < n_slabs; ++i) fill_w(i);
    }

    // ---- conversion of a raw weight stage.  Piece p = tid + 256 j (j = 0, 1): row r = p >> 2, octet c = p & 3: the
    //   eight lanes of a load phase read 128 contiguous bytes.  Weight (r, k = 8 c + e) goes to k row 8 c + e of
    //   the converted buffer; inside a k row the 16-byte column group g = r >> 2 is stored at g ^ 2 c, which makes
    //   the 32 lanes of a store (8 rows x 4 octets) hit 32 different banks.  The multiply loop reads whole
    //   groups at one k, so the swizzle costs it one exclusive-or per octet.
    // FP32 weights: 128 rows x 8 quads (4 weights = 16 bytes), piece p = tid + 256 j (j = 0 .. 3): row r = p >> 3, quad
    //   c = p & 7; weight (r, k = 4 c + e) goes to k row 4 c + e with the same column swizzle g ^ 2 (k >> 3) (the two
    //   quads of an octet then collide pairwise in a store: 16 stores per thread and slab, two-way conflicts).
    constexpr int NP = (WF == 2) ? 4 : 2;            // 16-byte pieces per thread and slab
    uint32_t cv_src[NP], cv_dst[NP];
#pragma unroll
    for (int j = 0; j < NP; ++j) {
        const int p = tid + 256 * j;
        if constexpr (WF == 2) {
            const int r = p >> 3, c = p & 7;
            cv_src[j] = (uint32_t)(r * 128 + c * 16);
            cv_dst[j] = (uint32_t)((4 * c) * BN + ((((r >> 2) ^ (2 * (c >> 1))) << 2) | (r & 3))) * 4u;
        } else {
            const int r = p >> 2, c = p & 3;
            cv_src[j] = (uint32_t)(r * 64 + c * 16);
            cv_dst[j] = (uint32_t)((8 * c) * BN + ((((r >> 2) ^ (2 * c)) << 2) | (r & 3))) * 4u;
        }
    }
    // Slabs alternate between two sets of buffers; the parity P of a slab is a compile-time constant of the code
    // that handles it (the slab loop is unrolled by two), so every shared-memory address of the multiply loop is a
    // per-thread base plus an immediate.
    auto convert = [&](int slab, auto par) -> bool {
        constexpr int P = decltype(par)::value;
        if (!mbar_wait(wfull0 + 8 * P, (uint32_t)(slab >> 1) & 1u, abort_flag, status, wait_limit_ns, 3)) return false;
#pragma unroll
        for (int j = 0; j < NP; ++j) {
            const uint4 v = lds128u(raw0 + P * kRawBytes + cv_src[j]);
            const uint32_t a = wf0 + P * kWfBytes + cv_dst[j];
            if constexpr (WF == 2) {
                sts32(a, __uint_as_float(v.x));
                sts32(a + 1 * BN * 4, __uint_as_float(v.y));
                sts32(a + 2 * BN * 4, __uint_as_float(v.z));
                sts32(a + 3 * BN * 4, __uint_as_float(v.w));
            } else {
                sts32(a, up16_lo<WF>(v.x));
                sts32(a + 1 * BN * 4, up16_hi<WF>(v.x));
                sts32(a + 2 * BN * 4, up16_lo<WF>(v.y));
                sts32(a + 3 * BN * 4, up16_hi<WF>(v.y));
                sts32(a + 4 * BN * 4, up16_lo<WF>(v.z));
                sts32(a + 5 * BN * 4, up16_hi<WF>(v.z));
                sts32(a + 6 * BN * 4, up16_lo<WF>(v.w));
                sts32(a + 7 * BN * 4, up16_hi<WF>(v.w));
            }
        }
        return true;
    };

    // acc[i][j]: rows m0 + (i < 4 ? 4 ty + i : 64 + TB ty + i - 4); column pair j:
    //   (n0 + 4 tx + 2 j, +1) for j < 2, (n0 + 64 + 4 tx + 2 (j - 2), +1) for j >= 2
    float2 acc[TR][4];
#pragma unroll
    for (int i = 0; i < TR; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = make_float2(0.0f, 0.0f);

    // this thread's two row groups inside a k row of an activation stage, and its column group inside a k row
    // of a converted weight buffer for each octet of k (the swizzle of the conversion)
    const uint32_t x_lo = xring + (uint32_t)(4 * ty) * 4u, x_hi = xring + (uint32_t)(64 + TB * ty) * 4u;
    uint32_t w_oct[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) w_oct[c] = wf0 + (uint32_t)(8 * c * BN) * 4u + (uint32_t)((tx ^ (2 * c)) << 4);

    // one octet of k: k = 8 c + e inside the slab (ne = 8; ne = 4 for the last four k of an FP32-weight layer whose K is
    // a multiple of 4 only)
    auto octet = [&](uint32_t xlo, uint32_t xhi, uint32_t wc, auto ne_c) {
        constexpr int NE = decltype(ne_c)::value;
#pragma unroll
        for (int e = 0; e < NE; ++e) {
            float xv[TR];
            lds_floats<4>(xlo + (uint32_t)(e * T::BM) * 4u, xv);
            lds_floats<TB>(xhi + (uint32_t)(e * T::BM) * 4u, xv + 4);
            const float4 wa = lds128(wc + (uint32_t)(e * BN) * 4u);
            const float4 wd = lds128(wc + (uint32_t)(e * BN + 64) * 4u);
            const float2 wp[4] = {make_float2(wa.x, wa.y), make_float2(wa.z, wa.w), make_float2(wd.x, wd.y),
                                  make_float2(wd.z, wd.w)};
            // column pair outermost: consecutive instructions share the weight operand (measured faster)
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int i = 0; i < TR; ++i) acc[i][j] = __ffma2_rn(make_float2(xv[i], xv[i]), wp[j], acc[i][j]);
        }
    };

    // one slab of parity P; returns false when a wait expired somewhere in the block (then nobody stores)
    auto do_slab = [&](int slab, auto par) -> bool {
        constexpr int P = decltype(par)::value;
        bool ok = true;
        if (slab + 1 < n_slabs) ok = convert(slab + 1, std::integral_constant<int, P ^ 1>());
        if (ok) ok = mbar_wait(xfull0 + 8 * P, (uint32_t)(slab >> 1) & 1u, abort_flag, status, wait_limit_ns, 4);
        // k beyond the end of the segment is skipped, not zero-filled; segments end on multiples of 8 (16-bit weights)
        // or 4 (FP32 weights)
        const int n_k = ok ? min(BK, k_hi - (k_lo + slab * BK)) : 0;
        const int n_oct = n_k >> 3;
        using Eight = std::integral_constant<int, 8>;
        using Four = std::integral_constant<int, 4>;
        if (n_oct == 4) {
#pragma unroll
            for (int c = 0; c < 4; ++c)
                octet(x_lo + P * T::kXBytes + (uint32_t)(8 * c * T::BM) * 4u, x_hi + P * T::kXBytes + (uint32_t)(8 * c * T::BM) * 4u,
                      w_oct[c] + P * kWfBytes, Eight());
        } else {
#pragma unroll 1
            for (int c = 0; c < n_oct; ++c)
                octet(x_lo + P * T::kXBytes + (uint32_t)(8 * c * T::BM) * 4u, x_hi + P * T::kXBytes + (uint32_t)(8 * c * T::BM) * 4u,
                      wf0 + P * kWfBytes + (uint32_t)(8 * c * BN) * 4u + (uint32_t)((tx ^ (2 * c)) << 4), Eight());
            if (WF == 2 && (n_k & 4)) {
                const int c = n_oct;
                octet(x_lo + P * T::kXBytes + (uint32_t)(8 * c * T::BM) * 4u, x_hi + P * T::kXBytes + (uint32_t)(8 * c * T::BM) * 4u,
                      wf0 + P * kWfBytes + (uint32_t)(8 * c * BN) * 4u + (uint32_t)((tx ^ (2 * c)) << 4), Four());
            }
        }
        // the barrier carries the vote
        if (!__syncthreads_and(ok)) return false;
        // every thread has finished reading this slab's activation stage and the raw stage of the next slab
        if (tid == 0) {
            if (slab + 2 < n_slabs) fill_x(slab + 2);
            if (slab + 3 < n_slabs) fill_w(slab + 3);
        }
        return true;
    };

    if (!__syncthreads_and(convert(0, std::integral_constant<int, 0>()))) return;
    if (tid == 0 && 2 < n_slabs) fill_w(2);
    for (int slab = 0; slab < n_slabs; slab += 2) {
        if (!do_slab(slab, std::integral_constant<int, 0>())) return;
        if (slab + 1 < n_slabs && !do_slab(slab + 1, std::integral_constant<int, 1>())) return;
    }

    // ---- epilogue: bias (direct) or the segment's partial ----
    const bool vec_ok = direct ? (ldy % 4 == 0) : (N % 4 == 0);     // rows of the destination start 16-byte aligned
#pragma unroll
    for (int i = 0; i < TR; ++i) {
        const int m = m0 + (i < 4 ? 4 * ty + i : 64 + TB * ty + (i - 4));
        if (m >= M) continue;
        float* orow = direct ? out + (long long)m * ldy : out + ((long long)s * M + m) * N;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int n = n0 + 64 * h + 4 * tx;
            float v[4] = {acc[i][2 * h].x, acc[i][2 * h].y, acc[i][2 * h + 1].x, acc[i][2 * h + 1].y};
            if (direct && bias) {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (n + e < N) v[e] = __fadd_rn(v[e], bias[n + e]);
            }
            if (vec_ok && n + 3 < N) {
                *reinterpret_cast<float4*>(orow + n) = make_float4(v[0], v[1], v[2], v[3]);
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (n + e < N) orow[n + e] = v[e];
            }
        }
    }
    if (direct || tile_counters == nullptr) return;

    // ---- split-K fold without a second launch (rule R3): the block that completes a tile's count of S partials adds
    // them in ascending segment order, then the bias, and stores.  Which block that is depends on timing; what it
    // computes does not.  Nobody waits for anybody.  The counter returns to zero for the next run. ----
    __threadfence();                                 // this block's partials are visible before its count
    __syncthreads();
    if (tid == 0) {
        unsigned* cnt = tile_counters + ((long long)tn * tiles_m + tm);
        const unsigned before = atomicAdd(cnt, 1u);
        fold_here = (before == (unsigned)(S - 1));
        if (fold_here) *cnt = 0u;
    }
    __syncthreads();
    if (!fold_here) return;
    __threadfence();                                 // the other blocks' partials, counted before ours, are visible
    const bool y_vec = (ldy % 4 == 0) && (N % 4 == 0);
#pragma unroll 1
    for (int i = 0; i < TR; ++i) {
        const int m = m0 + (i < 4 ? 4 * ty + i : 64 + TB * ty + (i - 4));
        if (m >= M) continue;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int n = n0 + 64 * h + 4 * tx;
            if (n >= N) continue;
            const float* p0 = out + (long long)m * N + n;
            const long long seg_stride = (long long)M * N;
            float v[4];
            if (y_vec && n + 3 < N) {
                float4 t = __ldcg(reinterpret_cast<const float4*>(p0));
                for (int s2 = 1; s2 < S; ++s2) {
                    const float4 u4 = __ldcg(reinterpret_cast<const float4*>(p0 + s2 * seg_stride));
                    t.x = __fadd_rn(t.x, u4.x); t.y = __fadd_rn(t.y, u4.y); t.z = __fadd_rn(t.z, u4.z); t.w = __fadd_rn(t.w, u4.w);
                }
                v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
                if (bias) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) v[e] = __fadd_rn(v[e], bias[n + e]);
                }
                *reinterpret_cast<float4*>(y + (long long)m * ldy + n) = make_float4(v[0], v[1], v[2], v[3]);
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (n + e >= N) continue;
                    float t = __ldcg(p0 + e);
                    for (int s2 = 1; s2 < S; ++s2) t = __fadd_rn(t, __ldcg(p0 + e + s2 * seg_stride));
                    y[(long long)m * ldy + n + e] = bias ? __fadd_rn(t, bias[n + e]) : t;
                }
            }
        }
    }
}

// First pass: xT[k][m] = x[m][k] for m < M, 0 for M <= m < ldt (ldt = M rounded up to a multiple of 4, the row pitch
// of xT).  32 x 32 tiles through shared memory: reads and writes are both 128-byte rows.
// (x, xT, M and m_pad are those of the slab of rows this launch covers: m_pad = the slab's share of ldt.)
__global__ void __launch_bounds__(256) transpose_x_kernel(const float* __restrict__ x, float* __restrict__ xT, int M, int m_pad, int K, int ldt)
{
    __shared__ float tile[32][33];
    const int k0 = blockIdx.x * 32, m0 = blockIdx.y * 32;
    const int c = threadIdx.x & 31, r0 = threadIdx.x >> 5;
#pragma unroll
    for (int r = r0; r < 32; r += 8) {
        const int m = m0 + r, k = k0 + c;
        tile[r][c] = (m < M && k < K) ? x[(long long)m * K + k] : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int r = r0; r < 32; r += 8) {
        const int k = k0 + r, m = m0 + c;
        if (k < K && m < m_pad) xT[(long long)k * ldt + m] = tile[c][r];
    }
}

template <int WF, int TR>
cudaError_t launch_t(const LaunchArgs& a, const CUtensorMap* map_w, const CUtensorMap* map_x)
{
    typedef Tile<WF, TR> T;
    static bool configured[kMaxDevices];             // function attributes belong to a device
    int dev = 0;
    cudaError_t de = cudaGetDevice(&dev);
    if (de != cudaSuccess) return de;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(prefill_tma_kernel<WF, TR>, cudaFuncAttributeMaxDynamicSharedMemorySize, T::kSmemBytes);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    const int tiles_m = (int)((a.M + T::BM - 1) / T::BM), tiles_n = (int)((a.N + BN - 1) / BN);
    const long long units = (long long)tiles_m * tiles_n * a.S;
    if (units > 0x7fffffffLL) return cudaErrorInvalidValue;
    const int direct = (a.S == 1);
    prefill_tma_kernel<WF, TR><<<(unsigned)units, kThreads, T::kSmemBytes, a.stream>>>(
        *map_x, *map_w, a.b, direct ? a.y : a.partials, (int)a.M, (int)a.N, (int)a.K, (int)a.seg_len, direct, tiles_m, tiles_n,
        (long long)a.ldy, a.status, a.wait_limit_ns, a.test_flags, a.y, a.tile_counters, a.S);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (!direct && !a.tile_counters) return launch_combine(a);
    return cudaSuccess;
}

template <int WF>
cudaError_t launch_f(const LaunchArgs& a, int tr, const CUtensorMap* map_w, const CUtensorMap* map_x)
{
    switch (tr) {
    case 5: return launch_t<WF, 5>(a, map_w, map_x);
    case 6: return launch_t<WF, 6>(a, map_w, map_x);
    case 7: return launch_t<WF, 7>(a, map_w, map_x);
    default: return launch_t<WF, 8>(a, map_w, map_x);
    }
}

}  // namespace

cudaError_t launch_transpose_x(const float* x, float* xT, int64_t M, int64_t K, int64_t ldt, cudaStream_t stream)
{
    const long long by = (ldt + 31) / 32, bx = (K + 31) / 32;
    dim3 grid((unsigned)bx, 1);
    // grid.y carries the rows (at most 65535 blocks per launch): larger M is cut into slabs of rows
    for (long long y0 = 0; y0 < by; y0 += 32768) {
        grid.y = (unsigned)((by - y0 < 32768) ? by - y0 : 32768);
        const long long m0 = y0 * 32;
        transpose_x_kernel<<<grid, 256, 0, stream>>>(x + m0 * K, xT + m0, (int)(M - m0), (int)(ldt - m0), (int)K, (int)ldt);
    }
    return cudaGetLastError();
}

// Tensor maps the caller builds, both without swizzle: the transposed activations xT [K][ldt] FP32 with box
// [32][16 tr]; W [N][K] 16-bit with box [128][32].
cudaError_t launch_prefill_tma(const LaunchArgs& a, int tr, const CUtensorMap* map_w, const CUtensorMap* map_x)
{
    if (!a.status) return cudaErrorInvalidValue;
    switch (a.wfmt) {
    case DET_WEIGHT_BF16: return launch_f<0>(a, tr, map_w, map_x);
    case DET_WEIGHT_FP16: return launch_f<1>(a, tr, map_w, map_x);
    case DET_WEIGHT_FP32: return launch_f<2>(a, tr, map_w, map_x);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace detlin
