// Decode kernel (bucket M <= 64): streams BF16 weight tiles from HBM through a TMA -> shared-memory
// ring, widens them to FP32 in registers (Eq. 2) and accumulates with packed IEEE FP32 FMAs
// (fma.rn.f32x2; rule R1) in the frozen decode order (V=4, L=32, P=1):
//
//   lane l of a warp owns k = c + 4l + j (j = 0..3) of every 128-element chunk c and accumulates
//   them in ascending order into one chain per output; the 32 lane sums of an output are then
//   added adjacent-first (lanes xor 1, 2, 4, 8, 16).
//
// One FP32x2 instruction advances the chains of two neighbouring weight rows (n, n+1) of the same
// batch row by one element each: its operands are (x[m,k], x[m,k]) and (up(W[n,k]), up(W[n+1,k])),
// its accumulator the pair (acc[m,n], acc[m,n+1]).  Each half is an ordinary fma.rn.f32, so the
// pairing is invisible in the bits.
//
// Everything else is schedule and therefore numerically inert (supplement C on rule R2: tile
// sizes, warp counts and pipeline depth do not change the reduction tree): one producer warp
// issues the bulk-tensor copies, WM x WR consumer warps each own an (MT batch rows) x (RT weight
// rows) register tile, thread blocks walk (row tile, segment, batch block) work units in a strided
// loop.  Rule R4 holds by construction: nothing that touches the order reads M.
//
// Every wait on a completion barrier is bounded; a wait that expires records the fact in the
// plan's device status word and the block drains and returns.
#pragma once
#include "internal.h"
#include "device_utils.cuh"

namespace detlin {

namespace decode_detail {

constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s per wait
constexpr unsigned kTryWaitHintNs = 2000;                   // a waiting thread may sleep this long per try

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(kTryWaitHintNs)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ float4 lds128(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr)
{
    uint2 v;
    asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  Returns false if the block is aborting or the wait expired (then it marks the
// block as aborting and records the site in the device status word).
__device__ __forceinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, DeviceStatus* status,
                                           unsigned site)
{
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_timer_ns() - t0 > kWaitLimitNs) {
            *abort_flag = 1;
            atomicExch(&status->where, site);
            atomicExch(&status->timeout_flag, 1u);
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, DeviceStatus* status,
                                          unsigned site)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, status, site);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar,
                                            unsigned long long policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dst),
        "l"(map), "r"(c0), "r"(c1), "r"(bar), "l"(policy)
        : "memory");
}

// The four consecutive weights of one row that a lane owns in a chunk: one 8-byte load for the
// 16-bit formats, one 16-byte load for FP32; element kk widened exactly to FP32.
template <int WF> struct WVec { typedef uint2 type; };
template <> struct WVec<2> { typedef float4 type; };
template <int WF>
__device__ __forceinline__ typename WVec<WF>::type wload(uint32_t addr)
{
    if constexpr (WF == 2) return lds128(addr);
    else return lds64(addr);
}
template <int WF>
__device__ __forceinline__ float wget(const typename WVec<WF>::type& v, int kk)
{
    if constexpr (WF == 2) {
        return kk == 0 ? v.x : kk == 1 ? v.y : kk == 2 ? v.z : v.w;
    } else {
        const uint32_t w = (kk < 2) ? v.x : v.y;
        return (kk & 1) ? up16_hi<WF>(w) : up16_lo<WF>(w);
    }
}

// PG = warps in the producer group: 1 (plain) or 4 (a whole warpgroup, which lets the kernel move
// registers from the producer to the consumers with setmaxnreg when the consumer tile is large).
template <int MT, int WM, int RT, int WR, int KC, int STAGES, int PG, int WF>
struct Cfg {
    static constexpr int kConsumerWarps = WM * WR;
    static constexpr int kThreads = (kConsumerWarps + PG) * 32;
    static constexpr int kMB = MT * WM;                       // batch rows per x box
    static constexpr int kRB = RT * WR;                       // weight rows per block tile
    static constexpr int kXBytes = kMB * KC * 4;
    static constexpr int kEB = WeightElem<WF>::bytes;         // bytes per weight element
    static constexpr int kWBoxBytes = RT * KC * kEB;
    static constexpr int kStageBytes = kXBytes + WR * kWBoxBytes;
    static constexpr int kBarBytes = 256;                     // 2*STAGES barriers + abort flag
    static constexpr int kSmemBytes = STAGES * kStageBytes + kBarBytes + 128;   // +128 for alignment
    // With a producer warpgroup the block is compiled for kMinBlocks blocks per SM and then moves
    // registers inside its own allocation (threads x launch registers): producers shrink to
    // kProducerRegs, consumers grow to kConsumerRegs.  setmaxnreg.inc blocks until the registers
    // exist, so the request must never exceed what the block owns.
    static constexpr int kMinBlocks = (PG == 4 && kConsumerWarps == 4) ? 2 : 1;
    static constexpr int kLaunchRegsRaw = (65536 / (kMinBlocks * kThreads)) / 8 * 8;
    static constexpr int kLaunchRegs = kLaunchRegsRaw > 255 ? 248 : kLaunchRegsRaw;
    static constexpr int kProducerRegs = 32;
    static constexpr int kConsumerRegsRaw =
        PG == 4 ? ((kThreads * kLaunchRegs - PG * 32 * kProducerRegs) / (kConsumerWarps * 32)) / 8 * 8 : 0;
    static constexpr int kConsumerRegs = kConsumerRegsRaw > 240 ? 240 : kConsumerRegsRaw;
    static_assert(PG == 1 || kConsumerRegs * kConsumerWarps * 32 + kProducerRegs * PG * 32 <= kThreads * kLaunchRegs,
                  "register move must fit in the block's own allocation");
    static_assert(PG == 1 || kConsumerRegs >= kLaunchRegs, "consumers only ever grow");
    static_assert(kSmemBytes <= 227 * 1024, "a block's ring must fit in shared memory");
    static_assert(RT % 2 == 0, "weight rows are processed in pairs (one FP32x2 accumulator per pair)");
    static_assert(PG == 1 || (PG == 4 && kConsumerWarps % 4 == 0), "setmaxnreg works on whole warpgroups");
    static_assert(STAGES >= 2 && STAGES <= 12, "ring depth");
    static_assert(KC % 128 == 0 && KC <= 256, "a stage holds whole 128-element chunks; TMA boxes are <= 256 wide");
    static_assert(kXBytes % 128 == 0 && kWBoxBytes % 128 == 0, "TMA destinations are 128-byte aligned");
};

// Butterfly reduce-scatter over the 32 lanes that realises the adjacent-first tree.  At step i
// (i = 0..4) lanes l and l ^ (1 << i) are partners.  While the number of values a lane holds is even,
// the partners exchange halves and add (the lane with bit i set keeps the upper half), so the work
// per step halves; once it is odd, the remaining steps add whole arrays (both partners then hold
// the same sums).  kScatterSteps<NV> = number of halving steps, kScatterKeep<NV> = values a lane
// holds at the end; lanes whose bits kScatterSteps..4 are zero own distinct results.
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

template <int REGS>
__device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS)); }
template <int REGS>
__device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS)); }

// Programmatic dependent launch: let the next kernel in the stream start its prologue early, and
// wait for the previous kernel's results before touching anything it may have produced.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

struct Unit {
    int tile, s, mb, k_lo, k_hi;
};
// Work unit u -> (batch block fastest, then row tile, then segment): the batch blocks of one row tile
// run side by side, so the tile's weights come from HBM once and from L2 for the other blocks.
__device__ __forceinline__ Unit decode_unit(long long u, int n_row_tiles, int n_mblocks, int seg_len, int K)
{
    Unit r;
    r.mb = (int)(u % n_mblocks);
    const long long q = u / n_mblocks;
    r.tile = (int)(q % n_row_tiles);
    r.s = (int)(q / n_row_tiles);
    r.k_lo = r.s * seg_len;
    r.k_hi = min(K, r.k_lo + seg_len);
    return r;
}

template <int MT, int WM, int RT, int WR, int KC, int STAGES, int PG, int WF>
__global__ void __launch_bounds__((WM * WR + PG) * 32, (Cfg<MT, WM, RT, WR, KC, STAGES, PG, WF>::kMinBlocks))
decode_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
              const float* __restrict__ bias, float* __restrict__ out, int M, int N, int K, int seg_len, int S, int direct,
              int n_row_tiles, int n_mblocks, long long ldy, DeviceStatus* status)
{
    using C = Cfg<MT, WM, RT, WR, KC, STAGES, PG, WF>;
    extern __shared__ unsigned char smem_raw[];
    // 128-byte aligned base (TMA destination requirement)
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    const uint32_t smem_base = smem_u32(smem);
    unsigned char* bar_mem = smem + STAGES * C::kStageBytes;
    const uint32_t full0 = smem_u32(bar_mem);                 // full[s]  at full0 + 8 s
    const uint32_t empty0 = full0 + 8 * STAGES;               // empty[s] at empty0 + 8 s
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_mem + 16 * STAGES);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, C::kConsumerWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    pdl_launch_dependents();

    const long long total_units = (long long)n_row_tiles * S * n_mblocks;

    if (warp < PG) {
        // ---------------- producer group: one lane issues all bulk-tensor copies ----------------
        if (PG == 4) reg_dec<C::kProducerRegs>();
        if (warp == 0 && lane == 0) {
            unsigned long long pol_w, pol_x;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_w));
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_x));
            unsigned it = 0;
            bool ok = true;
            // Weights never depend on the previous kernel, activations may: the first ring of
            // weight boxes is requested before waiting for the previous kernel to finish.
            unsigned pre = 0;
            {
                long long u = blockIdx.x;
                unsigned j = 0;
                while (u < total_units && j < (unsigned)STAGES) {
                    const Unit un = decode_unit(u, n_row_tiles, n_mblocks, seg_len, K);
                    for (int k0 = un.k_lo; k0 < un.k_hi && j < (unsigned)STAGES; k0 += KC, ++j) {
                        const uint32_t fb = full0 + 8 * j;
                        mbar_arrive_expect_tx(fb, C::kStageBytes);
                        const uint32_t sbase = smem_u32(smem + j * C::kStageBytes);
#pragma unroll
                        for (int wr = 0; wr < WR; ++wr)
                            tma_load_2d(sbase + C::kXBytes + wr * C::kWBoxBytes, &map_w, k0, un.tile * C::kRB + wr * RT, fb, pol_w);
                    }
                    u += gridDim.x;
                }
                pre = j;
            }
            pdl_wait();
            for (long long u = blockIdx.x; ok && u < total_units; u += gridDim.x) {
                const Unit un = decode_unit(u, n_row_tiles, n_mblocks, seg_len, K);
                const int n0 = un.tile * C::kRB;
                for (int k0 = un.k_lo; k0 < un.k_hi; k0 += KC, ++it) {
                    const int st = it % STAGES;
                    const unsigned use = it / STAGES;
                    const uint32_t fb = full0 + 8 * st;
                    const uint32_t sbase = smem_u32(smem + st * C::kStageBytes);
                    if (it >= pre) {
                        if (use > 0 && !mbar_wait(empty0 + 8 * st, (use - 1) & 1, abort_flag, status, 1)) { ok = false; break; }
                        mbar_arrive_expect_tx(fb, C::kStageBytes);
#pragma unroll
                        for (int wr = 0; wr < WR; ++wr)
                            tma_load_2d(sbase + C::kXBytes + wr * C::kWBoxBytes, &map_w, k0, n0 + wr * RT, fb, pol_w);
                    }
                    tma_load_2d(sbase, &map_x, k0, un.mb * C::kMB, fb, pol_x);
                }
            }
            if (!ok) {
                // aborting: wait (bounded) for the copies this thread still has in flight
                const unsigned first = it > (unsigned)STAGES ? it - STAGES : 0u;
                for (unsigned j = first; j < it; ++j) {
                    const unsigned long long t0 = global_timer_ns();
                    while (!mbar_try_wait(full0 + 8 * (j % STAGES), (j / STAGES) & 1))
                        if (global_timer_ns() - t0 > kWaitLimitNs) break;
                }
            }
        }
    } else {
        // ---------------- consumer warps ----------------
        if (PG == 4) reg_inc<C::kConsumerRegs>();
        const int cw = warp - PG;
        const int wm = cw % WM;
        const int wr = cw / WM;
        unsigned it = 0;
        bool ok = true;
        bool waited = false;
        for (long long u = blockIdx.x; ok && u < total_units; u += gridDim.x) {
            const Unit un = decode_unit(u, n_row_tiles, n_mblocks, seg_len, K);

            float2 acc[MT][RT / 2];      // [m][j] = chains of outputs (m, row 2j) and (m, row 2j+1)
#pragma unroll
            for (int m = 0; m < MT; ++m)
#pragma unroll
                for (int j = 0; j < RT / 2; ++j) acc[m][j] = make_float2(0.0f, 0.0f);

            for (int k0 = un.k_lo; k0 < un.k_hi; k0 += KC, ++it) {
                const int st = it % STAGES;
                if (!mbar_wait(full0 + 8 * st, (it / STAGES) & 1, abort_flag, status, 2)) { ok = false; break; }
                const uint32_t xs = smem_base + st * C::kStageBytes + (wm * MT) * (KC * 4) + lane * 16;
                const uint32_t ws = smem_base + st * C::kStageBytes + C::kXBytes + wr * C::kWBoxBytes + lane * (4 * C::kEB);
                // One 128-element chunk: the lane's four elements of every row / batch row of the warp tile.
                // Row pairs are processed in passes of at most four pairs so that only a few widened
                // weights are live at a time (the accumulators already take most of the registers).
                auto chunk = [&](int cc) {
                    float4 xv[MT];
#pragma unroll
                    for (int m = 0; m < MT; ++m) xv[m] = lds128(xs + m * (KC * 4) + cc * 512);
                    constexpr int kPairs = RT / 2;
#pragma unroll
                    for (int p0 = 0; p0 < kPairs; p0 += 4) {
                        constexpr int kMaxPass = 4;
                        const int np = (kPairs - p0) < kMaxPass ? (kPairs - p0) : kMaxPass;   // compile-time after unrolling
                        typename WVec<WF>::type w[2 * kMaxPass];
#pragma unroll
                        for (int q = 0; q < 2 * kMaxPass; ++q)
                            if (q < 2 * np) w[q] = wload<WF>(ws + (2 * p0 + q) * (KC * C::kEB) + cc * (128 * C::kEB));
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) {          // the lane's four elements, ascending
                            float2 wp[kMaxPass];
#pragma unroll
                            for (int j = 0; j < kMaxPass; ++j) {
                                if (j < np) wp[j] = make_float2(wget<WF>(w[2 * j], kk), wget<WF>(w[2 * j + 1], kk));
                            }
#pragma unroll
                            for (int m = 0; m < MT; ++m) {
                                const float xk = kk == 0 ? xv[m].x : kk == 1 ? xv[m].y : kk == 2 ? xv[m].z : xv[m].w;
                                const float2 x2 = make_float2(xk, xk);
#pragma unroll
                                for (int j = 0; j < kMaxPass; ++j)
                                    if (j < np) acc[m][p0 + j] = __ffma2_rn(x2, wp[j], acc[m][p0 + j]);
                            }
                        }
                    }
                };
                if (k0 + KC <= un.k_hi) {
                    // whole stage inside the segment: no per-lane test
#pragma unroll(MT * RT >= 64 ? 1 : 2)
                    for (int cc = 0; cc < KC / 128; ++cc) chunk(cc);
                } else {
                    // Last stage of a ragged K: elements beyond the end are skipped, not zero-filled
                    // (K % 4 == 0 here, so a lane's four elements are all inside or all outside).
#pragma unroll 1
                    for (int cc = 0; cc < KC / 128; ++cc)
                        if (k0 + cc * 128 + 4 * lane < un.k_hi) chunk(cc);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8 * st);
            }
            if (!ok) break;

            // ---- epilogue: lane tree, bias, store ----
            float v[MT * RT];
#pragma unroll
            for (int m = 0; m < MT; ++m)
#pragma unroll
                for (int j = 0; j < RT / 2; ++j) {
                    v[m * RT + 2 * j] = acc[m][j].x;
                    v[m * RT + 2 * j + 1] = acc[m][j].y;
                }
            constexpr int NV = MT * RT;
            constexpr int kKeep = Scatter<NV>::kKeep;
            constexpr int kSteps = Scatter<NV>::kSteps;
            // index of v[0] in the (m, q) tile after the scatter: bit i of the lane selects the upper
            // half at step i
            int base = 0;
            {
                int n = NV;
#pragma unroll
                for (int i = 0; i < kSteps; ++i) { n >>= 1; base += ((lane >> i) & 1) * n; }
            }
            // lanes that differ only in the bits above the halving steps hold the same sums; the one
            // whose high bits are zero stores them
            const bool owner = (lane >> kSteps) == 0;
            // bias values are requested before the lane tree so that their latency hides behind it
            float bv[kKeep];
#pragma unroll
            for (int t = 0; t < kKeep; ++t) {
                const int n = un.tile * C::kRB + wr * RT + (base + t) % RT;
                bv[t] = (direct && bias != nullptr && owner && n < N) ? __ldg(bias + n) : 0.0f;
            }
            lane_tree_scatter<MT * RT>(v, lane);
            // the output buffer may still be read by the previous kernel in the stream
            if (!waited) { pdl_wait(); waited = true; }
            if (owner) {
#pragma unroll
                for (int t = 0; t < kKeep; ++t) {
                    const int idx = base + t;
                    const int m = un.mb * C::kMB + wm * MT + idx / RT;
                    const int n = un.tile * C::kRB + wr * RT + idx % RT;
                    if (m < M && n < N) {
                        float r0 = v[t];
                        if (direct) {
                            if (bias) r0 = __fadd_rn(r0, bv[t]);
                            out[(long long)m * ldy + n] = r0;
                        } else {
                            out[((long long)un.s * M + m) * N + n] = r0;
                        }
                    }
                }
            }
        }
    }
    __syncthreads();
}

typedef cudaError_t (*DecodeLaunchFn)(const LaunchArgs&, const CUtensorMap*, const CUtensorMap*);
typedef int (*DecodeOccupancyFn)();

// Resident blocks per SM of one tiling (also opts the kernel into its dynamic shared memory).
// Returns 0 if the query fails.
template <int MT, int WM, int RT, int WR, int KC, int STAGES, int PG, int WF>
int decode_occupancy_t()
{
    using C = Cfg<MT, WM, RT, WR, KC, STAGES, PG, WF>;
    // function attributes belong to a device: opt in to the large shared-memory carve-out and cache
    // the answer once per device (benign if two threads race: both store the same value)
    static int blocks_per_sm[kMaxDevices];
    static bool known[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return 0; }
    if (!known[dev]) {
        auto kern = decode_kernel<MT, WM, RT, WR, KC, STAGES, PG, WF>;
        int occ = 0;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, C::kThreads, C::kSmemBytes) != cudaSuccess) {
            cudaGetLastError();
            return 0;
        }
        blocks_per_sm[dev] = occ;
        known[dev] = true;
    }
    return blocks_per_sm[dev];
}

template <int MT, int WM, int RT, int WR, int KC, int STAGES, int PG, int WF>
cudaError_t launch_decode_t(const LaunchArgs& a, const CUtensorMap* map_w, const CUtensorMap* map_x)
{
    using C = Cfg<MT, WM, RT, WR, KC, STAGES, PG, WF>;
    auto kern = decode_kernel<MT, WM, RT, WR, KC, STAGES, PG, WF>;
    const int blocks_per_sm = decode_occupancy_t<MT, WM, RT, WR, KC, STAGES, PG, WF>();
    if (blocks_per_sm <= 0) return cudaErrorLaunchOutOfResources;
    const int n_row_tiles = (int)((a.N + C::kRB - 1) / C::kRB);
    const int n_mblocks = (int)((a.M + C::kMB - 1) / C::kMB);
    const long long units = (long long)n_row_tiles * a.S * n_mblocks;
    long long grid = (long long)a.sm_count * blocks_per_sm;
    if (a.max_blocks > 0 && grid > a.max_blocks) grid = a.max_blocks;
    if (grid > units) grid = units;
    const int direct = (a.S == 1);

    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(C::kThreads);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = a.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, *map_w, *map_x, a.b, direct ? a.y : a.partials, (int)a.M, (int)a.N,
                                       (int)a.K, (int)a.seg_len, a.S, direct, n_row_tiles, n_mblocks, (long long)a.ldy, a.status);
    if (e != cudaSuccess) return e;
    if (!direct) return launch_combine(a);
    return cudaSuccess;
}

struct DecodeEntry {
    DecodeConfig cfg;
    DecodeLaunchFn fn;
    DecodeOccupancyFn occupancy;
};

#ifndef DET_WF
#define DET_WF 0
#endif
#define DEC(MT, WM, RT, WR, KC, ST, PG) \
    { {MT, WM, RT, WR, KC, ST, 0}, &launch_decode_t<MT, WM, RT, WR, KC, ST, PG, DET_WF>, &decode_occupancy_t<MT, WM, RT, WR, KC, ST, PG, DET_WF> }

}  // namespace decode_detail

// One table of tilings per weight format and batch class, defined in the decode_inst_*.cu files
// (separate files, compiled once per format, only to build in parallel).  All entries of a class
// produce identical bits.
struct DecodeClassTable {
    const decode_detail::DecodeEntry* entries;
    int count;
};
#define DET_CAT3(a, b, c) a##b##c
#define DET_TABLE_NAME(cls, wf) DET_CAT3(kDecodeClass, cls, _wf##wf)
#define DET_DECLARE_TABLES(wf)                                                                         \
    extern const DecodeClassTable DET_TABLE_NAME(0, wf), DET_TABLE_NAME(1, wf), DET_TABLE_NAME(2, wf), \
        DET_TABLE_NAME(3, wf), DET_TABLE_NAME(4, wf), DET_TABLE_NAME(5, wf);
DET_DECLARE_TABLES(0)
DET_DECLARE_TABLES(1)
DET_DECLARE_TABLES(2)

}  // namespace detlin
