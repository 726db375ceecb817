// Register-staged prefill kernel (bucket M > 64; the fallback of plans without an activation workspace, see
// prefill_tma.cu for the kernel that normally runs): register-tiled FP32 GEMM on the CUDA cores (rule R1: IEEE FMA only,
// never tensor cores) in the frozen prefill order (V=1, L=1, P=1): every output is one accumulation
// chain per K segment, strictly ascending in k (the order of the paper's own kernels, supplement C on
// rule R2); segments are summed in ascending order and the bias comes last.
//
// One packed fma.rn.f32x2 advances the chains of two neighbouring output columns (n, n+1) of the
// same row m by one element: operands (x[m,k], x[m,k]) and (up(W[n,k]), up(W[n+1,k])), accumulator
// (acc[m,n], acc[m,n+1]).  Each half is an ordinary fma.rn.f32, so the pairing is invisible in the
// bits.  Measured on B200 this loop sustains more than the scalar-FMA form of the same tile: the packed
// instruction needs an issue slot every other cycle only.
//
// Schedule (numerically inert): 128 x 128 output tile per block (16 TR x 128 with TR = 5 .. 7 rows per
// thread when that pads the batch less), 256 threads, 8 x 8 outputs per
// thread (4 column pairs), two blocks per SM, K walked in slabs of 32 with two slab buffers.  Both
// operands are staged k-major ([k][m] and [k][n]) so that a thread reads its eight x values and its
// eight weights of one k with four 16-byte loads.  16-bit weights are widened to FP32 once per block
// while the slab is staged (HBM and L2 only ever carry the stored format, Eq. 2).  Global loads of slab
// i+1 are in flight while slab i is multiplied.
#include "internal.h"
#include "device_utils.cuh"

namespace detlin {

namespace {

constexpr int BN = 128, BK = 32;
constexpr int kThreads = 256;
constexpr int kPitch = 132;                         // floats per k row: 128 + 4 keeps 16-byte alignment
constexpr int kTileFloats = BK * kPitch;
constexpr int kSmemBytes = 2 /*buffers*/ * 2 /*operands*/ * kTileFloats * 4;

__device__ __forceinline__ float4 lds128(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts32(uint32_t addr, float v)
{
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ uint4 ldg128_nc(const void* p)
{
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
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

// WF: weight format (0 BF16, 1 FP16: octets of 16-bit weights; 2 FP32: quads, staged like x)
// TR: output rows per thread (5 .. 8); the block tile is BM = 16 TR rows by 128 columns.  The row count
//     of the tile is schedule only: batch sizes between two multiples of 128 (the "mid bucket"
//     65 <= M < 128 in particular) get the tile height that wastes the fewest rows.
template <int WF, int TR>
__global__ void __launch_bounds__(kThreads, 2)
prefill_kernel(const float* __restrict__ x, const typename WeightElem<WF>::type* __restrict__ W, const float* __restrict__ bias,
               float* __restrict__ out, int M, int N, int K, int seg_len, int S, int direct, int tiles_m, int tiles_n,
               long long ldy)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const uint32_t smem = (uint32_t)__cvta_generic_to_shared(smem_raw);
    // buffer b: x tile at smem + b*2*T, w tile at smem + (b*2+1)*T, T = kTileFloats*4 bytes
    constexpr uint32_t T = kTileFloats * 4;

    constexpr int BM = 16 * TR;
    constexpr int TB = TR - 4;                       // rows of a thread in the upper group (1 .. 4)
    constexpr int XP = (BM * 8 + 255) / 256;         // 16-byte pieces of x per thread and slab
    const int tid = threadIdx.x;
    // 16 x 16 threads; a warp = 16 column groups x 2 row groups (8 x 4 and 4 x 8 warps measured 7 % slower)
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

    // ---- staging assignment (global rows are k-contiguous, shared tiles are k-major: a transpose) ----
    // x tile: BM rows x 8 quads (4 floats = 16 bytes).  Piece p = tid + 256 j: o = p & 3,
    //   row r = (p >> 2) mod BM, quad q = 4 * ((p >> 2) / BM) + o.  Four neighbouring lanes read 64
    //   contiguous bytes of a row, so a warp's load touches 8 rows (with two lanes per row and 16 rows
    //   per load the kernel measured 4 % slower; with eight lanes per row 6 % slower again because of
    //   four-way store conflicts).  The four scalar stores of a lane go to k rows 4q .. 4q+3, two-way
    //   bank conflicts (bank = 16 o + 4 e + r mod 32 over o in 0..3 and 8 consecutive r); a column
    //   swizzle that removes them cost more in the multiply loop than it saved.
    // w tile: 128 rows x 4 octets (8 BF16 = 16 bytes).  Piece p = tid + 256 j: half o = p & 1,
    //   row r = (p >> 1) & 127, octet c = 2 * (p >> 8) + o; eight scalar stores to k rows 8c .. 8c+7
    //   (two-way bank conflicts between the two halves; 16 stores per thread and slab).
    const float* xg[XP];
    uint32_t xs_off[XP];
    int xk[XP];
    bool xok[XP];
#pragma unroll
    for (int j = 0; j < XP; ++j) {
        const int p = tid + 256 * j;
        const int o = p & 3, r = (p >> 2) % BM, q = 4 * ((p >> 2) / BM) + o;
        const int m = m0 + r;
        xok[j] = m < M && p < BM * 8;
        xk[j] = q * 4;
        xg[j] = x + (long long)(xok[j] ? m : 0) * K + q * 4;
        xs_off[j] = (uint32_t)((q * 4) * kPitch + r) * 4;
    }
    // FP32 weights: 128 rows x 8 quads, the same assignment as the x tile.
    constexpr int NW = (WF == 2) ? 4 : 2;            // 16-byte pieces of W per thread and slab
    constexpr int WE = (WF == 2) ? 4 : 8;            // weights per piece
    const typename WeightElem<WF>::type* wg[NW];
    uint32_t ws_off[NW];
    int wk[NW];
    bool wok[NW];
#pragma unroll
    for (int j = 0; j < NW; ++j) {
        const int p = tid + 256 * j;
        const int o = p & 1, r = (p >> 1) & 127, c = 2 * (p >> 8) + o;
        const int n = n0 + r;
        wok[j] = n < N;
        wk[j] = c * WE;
        wg[j] = W + (long long)(wok[j] ? n : 0) * K + c * WE;
        ws_off[j] = (uint32_t)((c * WE) * kPitch + r) * 4;
    }

    uint4 xr[XP];
    uint4 wr[NW];
    auto load_slab = [&](int k0) {
        // the row pitch is a whole number of 16-byte pieces: a piece of weights / a quad of activations is
        // entirely inside or outside [.., k_hi)
#pragma unroll
        for (int j = 0; j < XP; ++j) {
            if (xok[j] && k0 + xk[j] < k_hi) xr[j] = ldg128_nc(xg[j] + k0);
            else xr[j] = make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int j = 0; j < NW; ++j) {
            if (wok[j] && k0 + wk[j] < k_hi) wr[j] = ldg128_nc(wg[j] + k0);
            else wr[j] = make_uint4(0u, 0u, 0u, 0u);
        }
    };
    auto store_slab = [&](int buf) {
        const uint32_t xb = smem + (uint32_t)(buf * 2) * T, wb = xb + T;
#pragma unroll
        for (int j = 0; j < XP; ++j) {
            if ((BM * 8) % 256 != 0 && tid + 256 * j >= BM * 8) continue;   // odd TR: the last round is half empty
            const uint32_t a = xb + xs_off[j];
            sts32(a, __uint_as_float(xr[j].x));
            sts32(a + kPitch * 4, __uint_as_float(xr[j].y));
            sts32(a + 2 * kPitch * 4, __uint_as_float(xr[j].z));
            sts32(a + 3 * kPitch * 4, __uint_as_float(xr[j].w));
        }
#pragma unroll
        for (int j = 0; j < NW; ++j) {
            const uint32_t a = wb + ws_off[j];
            if constexpr (WF == 2) {
                sts32(a, __uint_as_float(wr[j].x));
                sts32(a + kPitch * 4, __uint_as_float(wr[j].y));
                sts32(a + 2 * kPitch * 4, __uint_as_float(wr[j].z));
                sts32(a + 3 * kPitch * 4, __uint_as_float(wr[j].w));
            } else {
                // widen the eight 16-bit weights to FP32 (exact) on the way to shared memory
                sts32(a, up16_lo<WF>(wr[j].x));
                sts32(a + kPitch * 4, up16_hi<WF>(wr[j].x));
                sts32(a + 2 * kPitch * 4, up16_lo<WF>(wr[j].y));
                sts32(a + 3 * kPitch * 4, up16_hi<WF>(wr[j].y));
                sts32(a + 4 * kPitch * 4, up16_lo<WF>(wr[j].z));
                sts32(a + 5 * kPitch * 4, up16_hi<WF>(wr[j].z));
                sts32(a + 6 * kPitch * 4, up16_lo<WF>(wr[j].w));
                sts32(a + 7 * kPitch * 4, up16_hi<WF>(wr[j].w));
            }
        }
    };

    // acc[i][j]: rows m0 + (i < 4 ? 4 ty + i : 64 + TB ty + i - 4); column pair j:
    //   (n0 + 4 tx + 2 j, +1) for j < 2, (n0 + 64 + 4 tx + 2 (j - 2), +1) for j >= 2
    float2 acc[TR][4];
#pragma unroll
    for (int i = 0; i < TR; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = make_float2(0.0f, 0.0f);

    load_slab(k_lo);
    store_slab(0);
    __syncthreads();

    int buf = 0;
    for (int k0 = k_lo; k0 < k_hi; k0 += BK) {
        const bool more = k0 + BK < k_hi;
        if (more) load_slab(k0 + BK);
        const uint32_t xb = smem + (uint32_t)(buf * 2) * T + (uint32_t)(ty * 4) * 4;
        const uint32_t xb2 = xb + (uint32_t)(64 + ty * (TB - 4)) * 4;     // upper group: rows 64 + TB ty ..
        const uint32_t wb = smem + (uint32_t)(buf * 2 + 1) * T + (uint32_t)(tx * 4) * 4;
        // k beyond the end of the segment is skipped, not zero-filled
        const int nk = min(BK, k_hi - k0);
#pragma unroll 4
        for (int kk = 0; kk < nk; ++kk) {
            float xv[TR];
            lds_floats<4>(xb + (uint32_t)(kk * kPitch) * 4, xv);
            lds_floats<TB>(xb2 + (uint32_t)(kk * kPitch) * 4, xv + 4);
            const float4 wa = lds128(wb + (uint32_t)(kk * kPitch) * 4);
            const float4 wc = lds128(wb + (uint32_t)(kk * kPitch + 64) * 4);
            const float2 wp[4] = {make_float2(wa.x, wa.y), make_float2(wa.z, wa.w), make_float2(wc.x, wc.y),
                                  make_float2(wc.z, wc.w)};
            // column pair outermost: consecutive instructions share the weight operand.  Measured on B200, this
            // order sustains 6 % more than rows outermost (fewer register-bank stalls in the FMA pipe).
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int i = 0; i < TR; ++i) acc[i][j] = __ffma2_rn(make_float2(xv[i], xv[i]), wp[j], acc[i][j]);
        }
        if (more) store_slab(buf ^ 1);
        __syncthreads();
        buf ^= 1;
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
}

}  // namespace

namespace {

template <int WF, int TR>
cudaError_t launch_prefill_t(const LaunchArgs& a)
{
    constexpr int BM = 16 * TR;
    static bool configured[kMaxDevices];             // function attributes belong to a device
    int dev = 0;
    cudaError_t de = cudaGetDevice(&dev);
    if (de != cudaSuccess) return de;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(prefill_kernel<WF, TR>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    const int tiles_m = (int)((a.M + BM - 1) / BM), tiles_n = (int)((a.N + BN - 1) / BN);
    const long long units = (long long)tiles_m * tiles_n * a.S;
    if (units > 0x7fffffffLL) return cudaErrorInvalidValue;
    const int direct = (a.S == 1);
    prefill_kernel<WF, TR><<<(unsigned)units, kThreads, kSmemBytes, a.stream>>>(
        a.x, static_cast<const typename WeightElem<WF>::type*>(a.W), a.b, direct ? a.y : a.partials, (int)a.M, (int)a.N,
        (int)a.K, (int)a.seg_len, a.S, direct, tiles_m, tiles_n, (long long)a.ldy);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (!direct) return launch_combine(a);
    return cudaSuccess;
}

template <int WF>
cudaError_t launch_prefill_f(const LaunchArgs& a, int tr)
{
    switch (tr) {
    case 5: return launch_prefill_t<WF, 5>(a);
    case 6: return launch_prefill_t<WF, 6>(a);
    case 7: return launch_prefill_t<WF, 7>(a);
    default: return launch_prefill_t<WF, 8>(a);
    }
}

}  // namespace

// Rows per thread (tile height 16 TR) that pads the batch least; ties go to the taller tile.  Schedule
// only: every height gives the same bits.  a.variant 15 .. 18 forces 5 .. 8 rows here (tests).
int prefill_rows_per_thread(int64_t M)
{
    int best = 8;
    int64_t best_rows = ((M + 127) / 128) * 128;
    for (int tr = 7; tr >= 5; --tr) {
        const int64_t bm = 16 * tr, rows = ((M + bm - 1) / bm) * bm;
        if (rows < best_rows) { best_rows = rows; best = tr; }
    }
    return best;
}

cudaError_t launch_prefill(const LaunchArgs& a)
{
    const int tr = (a.variant >= 15 && a.variant <= 18) ? a.variant - 10 : prefill_rows_per_thread(a.M);
    switch (a.wfmt) {
    case DET_WEIGHT_BF16: return launch_prefill_f<0>(a, tr);
    case DET_WEIGHT_FP16: return launch_prefill_f<1>(a, tr);
    case DET_WEIGHT_FP32: return launch_prefill_f<2>(a, tr);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace detlin
