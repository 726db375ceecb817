// Decode kernel (bucket M <= 64): streams BF16 weight tiles from HBM through TMA -> shared-memory
// rings, widens them to FP32 in registers (Eq. 2) and accumulates with packed IEEE FP32 FMAs
// (fma.rn.f32x2; rule R1) in the frozen decode order (V=4, L=32, P=1, K cut into S segments):
//
//   lane l of a warp owns k = c + 4l + j (j = 0..3) of every 128-element chunk c of a segment and
//   accumulates them in ascending order into one chain per output; the 32 lane sums of an output
//   are added adjacent-first (lanes xor 1, 2, 4, 8, 16); the S segment sums of an output are added
//   in ascending segment order (rule R3), the bias last.
//
// One FP32x2 instruction advances the chains of two weight rows (n, n+1) of the same batch row by
// one element each: its operands are (x[m,k], x[m,k]) and (up(W[n,k]), up(W[n+1,k])), its
// accumulator the pair (acc[m,n], acc[m,n+1]).  Each half is an ordinary fma.rn.f32, so the
// pairing is invisible in the bits.
//
// Everything else is schedule and therefore numerically inert (supplement C on rule R2: tile
// sizes, warp counts and pipeline depth do not change the reduction tree).  A thread block owns
// one (row tile, batch block) work unit at a time and ALL its K segments: SK groups of WM x WR
// consumer warps work on SK segments side by side (each group has its own ring of stages, fed by
// one producer thread), the remaining segments follow in further rounds, and the block folds the S
// segment sums itself -- in registers when SK = 1, through shared memory otherwise -- so no
// workspace, no atomics and no second launch are needed.  Rule R4 holds by construction: nothing
// that touches the order reads M.
//
// Every wait on a completion barrier is bounded; a wait that expires records the fact in the
// plan's device status word and the block drains and returns.
#pragma once
#include "internal.h"
#include "device_utils.cuh"
#include "pipeline_utils.cuh"

namespace detlin {

namespace decode_detail {

using namespace pipe;


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

constexpr int ilog2(int v) { return v <= 1 ? 0 : 1 + ilog2(v / 2); }

template <int MT, int WM, int RT, int WR, int SK, int KC, int STAGES, int WF>
struct Cfg {
    static constexpr int kGroupWarps = WM * WR;               // consumer warps that share one ring
    static constexpr int kConsumerWarps = SK * kGroupWarps;
    // Producers: two warps per segment group, one requesting the weight tiles and one the activation tiles
    // (a bulk-tensor request costs its issuing thread some 200 cycles, and the activations can only be
    // requested once the previous kernel in the stream has finished).  Where the consumers hold 8-row
    // register tiles in whole warpgroups, the producers fill a warpgroup of their own and the kernel moves
    // registers from them to the consumers with setmaxnreg: the register file is split over the four
    // schedulers, so nine or ten warps per SM would cap every thread at 168 registers, less than an 8 x 14
    // tile needs.
    static constexpr bool kMoveRegs = (MT == 8 && (kConsumerWarps == 4 || kConsumerWarps == 8));
    // (8-row tiles in six consumer warps keep a single producer warp per group, which then requests both:
    // a tenth warp would bring the 168-register cap back.)
    static constexpr bool kSplitProducers = kMoveRegs || MT < 8;
    static constexpr int kPG = kMoveRegs ? 4 : (kSplitProducers ? 2 * SK : SK);
    static constexpr int kThreads = (kConsumerWarps + kPG) * 32;   // the producer group comes last
    static constexpr int kMB = MT * WM;                       // batch rows per x box
    static constexpr int kRB = RT * WR;                       // weight rows per W box (= per work unit)
    static constexpr int kEB = WeightElem<WF>::bytes;         // bytes per weight element
    static constexpr int kKB = KC < 256 ? KC : 256;           // k elements per TMA box (boxes are at most 256 wide)
    static constexpr int kSubs = KC / kKB;                    // boxes per operand and stage, laid out one after the other
    static constexpr int kXPitch = kKB * 4;                   // bytes between batch rows in a box
    static constexpr int kWPitch = kKB * kEB;                 // bytes between weight rows in a box
    static constexpr int kXBytes = kMB * kXPitch;
    static constexpr int kWBytes = kRB * kWPitch;
    static constexpr int kSubBytes = kXBytes + kWBytes;       // one x box followed by one W box
    static constexpr int kStageBytes = kSubs * kSubBytes;     // one stage of one group
    static constexpr int kRingBytes = SK * STAGES * kStageBytes;
    static constexpr int kBarBytes = (16 * SK * STAGES + 16 + 127) / 128 * 128;   // full + empty barriers, abort flag
    static constexpr int kTile = kMB * kRB;                   // outputs of a work unit
    static constexpr int kFixedSmem = kRingBytes + kBarBytes + 128;               // + 128 for alignment
    static constexpr int kLM = ilog2(MT);
    static constexpr int kKeep = RT / 2;                      // sums a lane holds after the lane tree
    static constexpr int kOwnerLanes = 2 * MT;                // lanes 0 .. 2 MT - 1 hold distinct sums
    // Small blocks run two to an SM; the register cap follows from that.
    static constexpr int kMinBlocks = (kConsumerWarps <= 4) ? 2 : 1;
    // With a producer warpgroup the block is compiled for kMinBlocks blocks per SM and then moves
    // registers inside its own allocation (threads x launch registers): producers shrink to
    // kProducerRegs, consumers grow to kConsumerRegs.  setmaxnreg.inc blocks until the registers
    // exist, so the request must never exceed what the block owns.
    static constexpr int kLaunchRegsRaw = (65536 / (kMinBlocks * kThreads)) / 8 * 8;
    static constexpr int kLaunchRegs = kLaunchRegsRaw > 255 ? 248 : kLaunchRegsRaw;
    static constexpr int kProducerRegs = 40;
    static constexpr int kConsumerRegsRaw =
        kMoveRegs ? ((kThreads * kLaunchRegs - kPG * 32 * kProducerRegs) / (kConsumerWarps * 32)) / 8 * 8 : 0;
    static constexpr int kConsumerRegs = kConsumerRegsRaw > 240 ? 240 : kConsumerRegsRaw;
    static_assert(!kMoveRegs || kConsumerRegs * kConsumerWarps * 32 + kProducerRegs * kPG * 32 <= kThreads * kLaunchRegs,
                  "register move must fit in the block's own allocation");
    static_assert(!kMoveRegs || kConsumerRegs >= kLaunchRegs, "consumers only ever grow");
    static_assert((kSplitProducers ? 2 : 1) * SK <= kPG, "one or two producer warps per segment group");
    // shared memory of a launch whose order has S segments (the S partial tiles when SK > 1)
    static constexpr int smem_bytes(int S) { return kFixedSmem + (SK > 1 ? S * kTile * 4 : 0); }
    static_assert(RT % 2 == 0, "weight rows are processed in pairs (one FP32x2 accumulator per pair)");
    static_assert(MT == 1 || MT == 2 || MT == 4 || MT == 8, "batch rows per warp: a power of two up to 8");
    static_assert(STAGES >= 2 && STAGES <= 12, "ring depth");
    static_assert(KC == 128 || KC == 256 || KC == 512, "a stage holds whole 128-element chunks in boxes of at most 256");
    static_assert(kRB <= 256 && kMB <= 256, "TMA boxes are at most 256 rows high");
    static_assert(kXBytes % 128 == 0 && kWBytes % 128 == 0, "TMA destinations are 128-byte aligned");
    static_assert(kFixedSmem <= 227 * 1024, "a block's rings must fit in shared memory");
};

template <int REGS>
__device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS)); }
template <int REGS>
__device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS)); }

// Programmatic dependent launch: let the next kernel in the stream start its prologue early, and
// wait for the previous kernel's results before touching anything it may have produced.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ void consumer_barrier(int threads)
{
    asm volatile("bar.sync 1, %0;" ::"r"(threads) : "memory");
}

// Test hook bits (LaunchArgs::test_flags): never set outside the tests.
constexpr int kTestWithholdFirstX = 1;   // block 0 never requests the activations of its first stage


template <int MT, int WM, int RT, int WR, int SK, int KC, int STAGES, int WF>
__global__ void __launch_bounds__((Cfg<MT, WM, RT, WR, SK, KC, STAGES, WF>::kThreads), (Cfg<MT, WM, RT, WR, SK, KC, STAGES, WF>::kMinBlocks))
decode_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
              const float* __restrict__ bias, float* __restrict__ y, int M, int N, int K, int seg_len, int S,
              int n_row_tiles, int n_mblocks, long long ldy, DeviceStatus* status, unsigned long long wait_limit_ns,
              int test_flags)
{
    using C = Cfg<MT, WM, RT, WR, SK, KC, STAGES, WF>;
    extern __shared__ unsigned char smem_raw[];
    // 128-byte aligned base (TMA destination requirement)
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    const uint32_t smem_base = smem_u32(smem);
    unsigned char* bar_mem = smem + C::kRingBytes;
    const uint32_t full0 = smem_u32(bar_mem);                 // full[g][st]  at full0 + 8 (g STAGES + st)
    const uint32_t empty0 = full0 + 8 * SK * STAGES;          // empty[g][st] likewise
    const uint32_t abort_flag = empty0 + 8 * SK * STAGES;     // shared-memory address of the block's abort word
    float* part = reinterpret_cast<float*>(bar_mem + C::kBarBytes);   // [S][kMB][kRB] when SK > 1

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // Set-up without a block-wide stop: the producer of group g initialises that group's barriers and goes
    // straight on to request weight tiles; producer warps only ARRIVE at named barrier 2, the consumers wait
    // on it (so they see initialised barriers), nobody waits for the consumers.
    if (warp >= C::kConsumerWarps) {
        const int pg = warp - C::kConsumerWarps;
        if (pg < SK && lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
            for (int i = 0; i < STAGES; ++i) {
                mbar_init(full0 + 8 * (pg * STAGES + i), 1);
                mbar_init(empty0 + 8 * (pg * STAGES + i), C::kGroupWarps);
            }
            if (pg == 0) sts_volatile_i32(abort_flag, 0);
            // make the initialised barriers visible to the bulk-copy engine
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            if (!C::kSplitProducers) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        } else if (C::kSplitProducers && pg < 2 * SK && lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        }
        __syncwarp();
        asm volatile("bar.arrive 2, %0;" ::"r"(C::kThreads) : "memory");
    } else {
        asm volatile("bar.sync 2, %0;" ::"r"(C::kThreads) : "memory");
    }
    pdl_launch_dependents();

    const int total_units = n_row_tiles * n_mblocks;          // the host keeps this below 2^31
    const int rounds = S / SK;                                // the host only picks tilings with S % SK == 0

    // Work unit u -> (batch block fastest, then row tile): the batch blocks of one row tile run side
    // by side, so the tile's weights come from HBM once and from L2 for the other blocks.
    auto seg_range = [&](int s, int& k_lo, int& k_hi) {
        k_lo = s * seg_len;
        k_hi = min(K, k_lo + seg_len);
    };

    if (warp >= C::kConsumerWarps) {
        // ---------------- producers: lane 0 of producer warp g requests the weight tiles of group g, lane 0 of
        // producer warp SK + g its activation tiles ----------------
        if (C::kMoveRegs) reg_dec<C::kProducerRegs>();
        const int pw = warp - C::kConsumerWarps;
        if (pw >= (C::kSplitProducers ? 2 : 1) * SK || lane != 0) return;
        const bool do_x = !C::kSplitProducers || pw >= SK;          // requests activation tiles
        const bool do_w = !C::kSplitProducers || pw < SK;           // requests weight tiles
        const int g = pw >= SK ? pw - SK : pw;
        unsigned long long pol_w, pol_x;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_w));
        asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_x));
        const uint32_t fullg = full0 + 8 * g * STAGES;
        const uint32_t emptyg = empty0 + 8 * g * STAGES;
        const uint32_t ringg = smem_base + (uint32_t)(g * STAGES * C::kStageBytes);

        // Position in the group's stream of stages: work unit (row tile, batch block), round, first k.
        struct Cursor {
            int u, tile, mb, r, k0, k_hi;
        };
        auto start = [&](Cursor& c) -> bool {
            c.u = (int)blockIdx.x;
            c.r = 0;
            if (c.u >= total_units) return false;
            c.tile = c.u / n_mblocks;
            c.mb = c.u - c.tile * n_mblocks;
            seg_range(g, c.k0, c.k_hi);
            return true;
        };
        auto advance = [&](Cursor& c) -> bool {             // to the group's next stage; false at the end
            c.k0 += KC;
            if (c.k0 < c.k_hi) return true;
            if (++c.r == rounds) {
                c.r = 0;
                c.u += (int)gridDim.x;
                if (c.u >= total_units) return false;
                c.tile = c.u / n_mblocks;
                c.mb = c.u - c.tile * n_mblocks;
            }
            seg_range(c.r * SK + g, c.k0, c.k_hi);
            return true;
        };
        // The weight producer announces the stage's bytes (weights and activations) on its full barrier;
        // the activation producer only adds its copy (the byte count of a barrier may run ahead of the
        // announcement: the phase cannot complete before the announcing arrival).
        auto issue = [&](int st, const Cursor& c, bool w, bool x) {
            const uint32_t fb = fullg + 8 * st;
            if (w) mbar_arrive_expect_tx(fb, C::kStageBytes);
#pragma unroll
            for (int sub = 0; sub < C::kSubs; ++sub) {
                const uint32_t dst = ringg + (uint32_t)(st * C::kStageBytes + sub * C::kSubBytes);
                if (w) tma_load_2d(dst + C::kXBytes, &map_w, c.k0 + sub * C::kKB, c.tile * C::kRB, fb, pol_w);
                if (x) tma_load_2d(dst, &map_x, c.k0 + sub * C::kKB, c.mb * C::kMB, fb, pol_x);
            }
        };

        Cursor c;
        bool live = start(c);
        // Weights never depend on the previous kernel in the stream, activations may: weight requests start at
        // once, activation requests wait for that kernel to finish.  A thread that requests both sends the
        // first ring of weight requests ahead of the wait.
        int pre = 0;
        if (do_w && do_x) {
            const Cursor c0 = c;
            const bool live0 = live;
            while (live && pre < STAGES) {
                issue(pre, c, true, false);
                ++pre;
                live = advance(c);
            }
            c = c0;
            live = live0;
        }
        if (do_x) pdl_wait();
        int st = 0;
        unsigned phase = 0, n_issued = 0;
        bool ok = true;
        while (live) {
            if (n_issued >= (unsigned)STAGES) {
                // the slot's previous use must have been released by every consumer warp of the group
                if (!mbar_wait(emptyg + 8 * st, phase ^ 1, abort_flag, status, wait_limit_ns, 1)) { ok = false; break; }
            }
            const bool withhold = (test_flags & kTestWithholdFirstX) && blockIdx.x == 0 && g == 0 && n_issued == 0;
            issue(st, c, do_w && (int)n_issued >= pre, do_x && !withhold);
            ++n_issued;
            if (++st == STAGES) { st = 0; phase ^= 1; }
            live = advance(c);
        }
        if (!ok) {
            // aborting: wait (bounded) for the copies still in flight in the group's ring
            const unsigned first = n_issued > (unsigned)STAGES ? n_issued - STAGES : 0u;
            for (unsigned j = first; j < n_issued; ++j) {
                const unsigned long long t0 = global_timer_ns();
                while (!mbar_try_wait(fullg + 8 * (j % STAGES), (j / STAGES) & 1))
                    if (global_timer_ns() - t0 > wait_limit_ns) break;
            }
        }
        return;
    }

    // ---------------- consumer warps ----------------
    if (C::kMoveRegs) reg_inc<C::kConsumerRegs>();
    const int g = warp / C::kGroupWarps;
    const int gw = warp % C::kGroupWarps;
    const int wm = gw % WM;
    const int wr = gw / WM;
    // Lane roles in the lane tree (see lane_tree below): bit 0 of the lane selects the weight row of
    // each pair it ends up owning, bit 1 the upper half of the warp's batch rows.  The loads are
    // permuted accordingly so that the first two tree steps need no data-dependent register choice.
    const int b0 = lane & 1;
    const int b1 = (MT > 1) ? ((lane >> 1) & 1) : 0;
    const int x_lo_off = b1 * (MT / 2) * C::kXPitch;         // added for batch rows [0, MT/2), subtracted above
    const int w_off = b0 * C::kWPitch;                       // added for even row slots, subtracted for odd ones
    const uint32_t fullg = full0 + 8 * g * STAGES;
    const uint32_t emptyg = empty0 + 8 * g * STAGES;
    const uint32_t ringg = smem_base + (uint32_t)(g * STAGES * C::kStageBytes);

    int st = 0;                                               // ring position of the group's next stage, and its phase
    unsigned phase = 0;
    bool ok = true;
    bool waited = false;
    // Has the next stage landed?  Asked ahead of time (without blocking) so that the answer is already
    // there when the multiply loop needs it.
    bool ready = false;
    constexpr int kKeep = C::kKeep;
    for (int u = (int)blockIdx.x; u < total_units; u += (int)gridDim.x) {
        const int mb = u % n_mblocks;
        const int tile = u / n_mblocks;
        float tot[kKeep];                                     // running fold over the segments when SK == 1

        for (int r = 0; r < rounds; ++r) {
            const int s = r * SK + g;
            int k_lo, k_hi;
            seg_range(s, k_lo, k_hi);

            float2 acc[MT][RT / 2];      // [m][j] = chains of outputs (slot m, row slots 2j and 2j+1)
#pragma unroll
            for (int m = 0; m < MT; ++m)
#pragma unroll
                for (int j = 0; j < RT / 2; ++j) acc[m][j] = make_float2(0.0f, 0.0f);

            for (int k0 = k_lo; ok && k0 < k_hi; k0 += KC) {
                // (the votes keep the decision warp-uniform even if a wait expires for some lanes only)
                if (!__all_sync(0xffffffffu, ready)) {
                    if (!__all_sync(0xffffffffu, mbar_wait(fullg + 8 * st, phase, abort_flag, status, wait_limit_ns, 2))) { ok = false; break; }
                }
                const uint32_t sbase = ringg + (uint32_t)(st * C::kStageBytes);
                const uint32_t xs = sbase + (wm * MT) * C::kXPitch + lane * 16;
                const uint32_t ws = sbase + C::kXBytes + (wr * RT) * C::kWPitch + lane * (4 * C::kEB);
                const int st_cur = st;
                if (++st == STAGES) { st = 0; phase ^= 1; }
                // One 128-element chunk: the lane's four elements of every row / batch row of the warp tile.
                // Row pairs are processed in passes of at most four pairs so that only a few widened
                // weights are live at a time (the accumulators already take most of the registers).
                auto chunk = [&](int cc) {
                    // chunk cc lies in box cc / (kKB / 128) of the stage, at element (cc * 128) % kKB of its rows
                    const uint32_t box = (uint32_t)((cc * 128) / C::kKB) * C::kSubBytes;
                    const uint32_t kin = (uint32_t)((cc * 128) % C::kKB);
                    const uint32_t xc = xs + box + kin * 4, wc = ws + box + kin * C::kEB;
                    const uint32_t xs_lo = xc + x_lo_off, xs_hi = xc - x_lo_off;
                    const uint32_t ws_even = wc + w_off, ws_odd = wc - w_off;
                    float4 xv[MT];
#pragma unroll
                    for (int m = 0; m < MT; ++m)
                        xv[m] = lds128((m < (MT + 1) / 2 ? xs_lo : xs_hi) + m * C::kXPitch);
                    constexpr int kPairs = RT / 2;
#pragma unroll
                    for (int p0 = 0; p0 < kPairs; p0 += 4) {
                        constexpr int kMaxPass = 4;
                        const int np = (kPairs - p0) < kMaxPass ? (kPairs - p0) : kMaxPass;   // compile-time after unrolling
                        typename WVec<WF>::type w[2 * kMaxPass];
#pragma unroll
                        for (int q = 0; q < 2 * kMaxPass; ++q)
                            if (q < 2 * np)
                                w[q] = wload<WF>(((q & 1) ? ws_odd : ws_even) + (2 * p0 + q) * C::kWPitch);
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
                if (k0 + KC <= k_hi) {
                    // whole stage inside the segment: no per-lane test
                    {
#pragma unroll(MT * RT >= 64 ? 1 : 2)
                        for (int cc = 0; cc < KC / 128 - 1; ++cc) chunk(cc);
                        ready = mbar_test_wait(fullg + 8 * st, phase);          // look ahead: the stage after this one
                        chunk(KC / 128 - 1);
                    }
                } else {
                    ready = false;
                    // Last stage of a ragged K: elements beyond the end are skipped, not zero-filled
                    // (K % 4 == 0 here, so a lane's four elements are all inside or all outside).
#pragma unroll 1
                    for (int cc = 0; cc < KC / 128; ++cc)
                        if (k0 + cc * 128 + 4 * lane < k_hi) chunk(cc);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(emptyg + 8 * st_cur);
            }

            // ---- lane tree: the 32 lane sums of every output, adjacent lanes first ----
            // Step i adds the values of lanes l and l ^ (1 << i) (fadd is commutative, so both partners
            // would compute the same bits); instead of keeping every sum in both, the partners split the
            // outputs between them, which halves the work of every further step:
            //   step 0: the lane keeps the .x half of every accumulator pair and receives its partner's
            //           .y half -- the weight rows were loaded swapped in odd lanes, so .x is row 2j + b0;
            //   step 1: it keeps its first MT/2 register rows -- the batch rows were loaded with their halves
            //           swapped in lanes with b1 = 1, so those are batch rows [b1 MT/2, b1 MT/2 + MT/2);
            //   steps 2 .. kLM: halving by choice (the lane with the step's bit set keeps the upper half);
            //   remaining steps: plain exchanges (both partners keep the sum).
            // Lane l < 2 MT ends up with the sums of batch slot m(l) and row slots 2j + b0, j = 0 .. RT/2 - 1.
            float v[MT > 1 ? MT / 2 : 1][kKeep];
#pragma unroll
            for (int m = 0; m < MT; ++m)
#pragma unroll
                for (int j = 0; j < kKeep; ++j) acc[m][j].x = __fadd_rn(acc[m][j].x, __shfl_xor_sync(0xffffffffu, acc[m][j].y, 1));
            if constexpr (MT > 1) {
#pragma unroll
                for (int m = 0; m < MT / 2; ++m)
#pragma unroll
                    for (int j = 0; j < kKeep; ++j) v[m][j] = __fadd_rn(acc[m][j].x, __shfl_xor_sync(0xffffffffu, acc[m + MT / 2][j].x, 2));
            } else {
                // a single batch row: step 1 is already a plain exchange
#pragma unroll
                for (int j = 0; j < kKeep; ++j) v[0][j] = __fadd_rn(acc[0][j].x, __shfl_xor_sync(0xffffffffu, acc[0][j].x, 2));
            }
            int m_slot = b1 * (MT / 2);                           // batch slot of v[0] within the warp tile
            constexpr int kFirstFull = (MT > 1) ? C::kLM + 1 : 1;   // first step that is a plain exchange
#pragma unroll
            for (int i = 2; i < 5; ++i) {
                const int d = 1 << i;
                if (i < kFirstFull) {
                    // halving by choice on the next batch-row bit; `cnt` register rows are live before the step
                    const int cnt = (MT / 2) >> (i - 2);
                    const int half = cnt / 2;
                    const bool hi = (lane >> i) & 1;
#pragma unroll
                    for (int m = 0; m < (MT > 1 ? MT / 2 : 1); ++m) {
                        if (m < half) {
#pragma unroll
                            for (int j = 0; j < kKeep; ++j) {
                                const float send = hi ? v[m][j] : v[m + half][j];
                                const float keep = hi ? v[m + half][j] : v[m][j];
                                v[m][j] = __fadd_rn(keep, __shfl_xor_sync(0xffffffffu, send, d));
                            }
                        }
                    }
                    m_slot += hi ? half : 0;
                } else {
#pragma unroll
                    for (int j = 0; j < kKeep; ++j) v[0][j] = __fadd_rn(v[0][j], __shfl_xor_sync(0xffffffffu, v[0][j], d));
                }
            }
            const bool owner = lane < C::kOwnerLanes;
            if constexpr (SK == 1) {
#pragma unroll
                for (int j = 0; j < kKeep; ++j) tot[j] = (r == 0) ? v[0][j] : __fadd_rn(tot[j], v[0][j]);
            } else {
                if (owner) {
                    float* p = part + ((size_t)s * C::kMB + wm * MT + m_slot) * C::kRB + wr * RT + b0;
#pragma unroll
                    for (int j = 0; j < kKeep; ++j) p[2 * j] = v[0][j];
                }
            }
            if constexpr (SK == 1) {
                if (r == rounds - 1) {
                    // ---- bias and store straight from the owner lanes ----
                    const int m = mb * C::kMB + wm * MT + m_slot;
                    const int n0 = tile * C::kRB + wr * RT + b0;
                    float bv[kKeep];
#pragma unroll
                    for (int j = 0; j < kKeep; ++j) bv[j] = (bias != nullptr && owner && n0 + 2 * j < N) ? __ldg(bias + n0 + 2 * j) : 0.0f;
                    // the output buffer may still be read by the previous kernel in the stream
                    if (!waited) { pdl_wait(); waited = true; }
                    if (ok && owner && m < M) {
#pragma unroll
                        for (int j = 0; j < kKeep; ++j) {
                            const int n = n0 + 2 * j;
                            if (n < N) y[(long long)m * ldy + n] = bias ? __fadd_rn(tot[j], bv[j]) : tot[j];
                        }
                    }
                }
            }
        }

        if constexpr (SK > 1) {
            // ---- fold the S segment sums of every output in ascending order, bias last, store ----
            // (the bias of the thread's first output is requested before the barrier: its latency hides there)
            float b_first = 0.0f;
            {
                const int n = tile * C::kRB + (int)threadIdx.x % C::kRB;
                if (bias != nullptr && (int)threadIdx.x < C::kTile && n < N) b_first = __ldg(bias + n);
            }
            consumer_barrier(C::kConsumerWarps * 32);
            const bool aborting = lds_volatile_i32(abort_flag) != 0;
            if (!waited) { pdl_wait(); waited = true; }
            if (!aborting) {
                for (int o = threadIdx.x; o < C::kTile; o += C::kConsumerWarps * 32) {
                    const int ml = o / C::kRB, nl = o % C::kRB;
                    const int m = mb * C::kMB + ml, n = tile * C::kRB + nl;
                    if (m < M && n < N) {
                        float t = part[o];
                        for (int s2 = 1; s2 < S; ++s2) t = __fadd_rn(t, part[s2 * C::kTile + o]);
                        if (bias) t = __fadd_rn(t, o == (int)threadIdx.x ? b_first : __ldg(bias + n));
                        y[(long long)m * ldy + n] = t;
                    }
                }
            }
            consumer_barrier(C::kConsumerWarps * 32);         // the partial tiles are rewritten by the next unit
            if (aborting) break;                              // uniform: every warp read the flag after the same barrier
        } else {
            if (!ok) break;
        }
    }
}

typedef cudaError_t (*DecodeLaunchFn)(const LaunchArgs&, const CUtensorMap*, const CUtensorMap*);
typedef int (*DecodeOccupancyFn)(int S);

// Resident blocks per SM of one tiling for an order with S segments (also opts the kernel into its
// dynamic shared memory).  Returns 0 if the tiling cannot run (S not a multiple of its segment
// groups, shared memory, failed query).
template <int MT, int WM, int RT, int WR, int SK, int KC, int STAGES, int WF>
int decode_occupancy_t(int S)
{
    using C = Cfg<MT, WM, RT, WR, SK, KC, STAGES, WF>;
    if (S < 1 || S > kDecodeMaxSegments || S % SK != 0) return 0;
    if (C::smem_bytes(S) > 227 * 1024) return 0;
    // function attributes belong to a device: opt in to the large shared-memory carve-out and cache
    // the answer once per device and S (benign if two threads race: both store the same value)
    static int blocks_per_sm[kMaxDevices][kDecodeMaxSegments + 1];
    static bool known[kMaxDevices][kDecodeMaxSegments + 1];
    static bool attr_set[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return 0; }
    auto kern = decode_kernel<MT, WM, RT, WR, SK, KC, STAGES, WF>;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::smem_bytes(kDecodeMaxSegments) > 227 * 1024 ? 227 * 1024 : C::smem_bytes(kDecodeMaxSegments)) != cudaSuccess) {
            cudaGetLastError();
            return 0;
        }
        attr_set[dev] = true;
    }
    if (!known[dev][S]) {
        int occ = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, C::kThreads, C::smem_bytes(S)) != cudaSuccess) {
            cudaGetLastError();
            return 0;
        }
        blocks_per_sm[dev][S] = occ;
        known[dev][S] = true;
    }
    return blocks_per_sm[dev][S];
}

template <int MT, int WM, int RT, int WR, int SK, int KC, int STAGES, int WF>
cudaError_t launch_decode_t(const LaunchArgs& a, const CUtensorMap* map_w, const CUtensorMap* map_x)
{
    using C = Cfg<MT, WM, RT, WR, SK, KC, STAGES, WF>;
    auto kern = decode_kernel<MT, WM, RT, WR, SK, KC, STAGES, WF>;
    const int blocks_per_sm = decode_occupancy_t<MT, WM, RT, WR, SK, KC, STAGES, WF>(a.S);
    if (blocks_per_sm <= 0) return cudaErrorLaunchOutOfResources;
    const int n_row_tiles = (int)((a.N + C::kRB - 1) / C::kRB);
    const int n_mblocks = (int)((a.M + C::kMB - 1) / C::kMB);
    const long long units = (long long)n_row_tiles * n_mblocks;
    long long grid = (long long)a.sm_count * blocks_per_sm;
    if (a.max_blocks > 0 && grid > a.max_blocks) grid = a.max_blocks;
    if (grid > units) grid = units;

    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(C::kThreads);
    cfg.dynamicSmemBytes = C::smem_bytes(a.S);
    cfg.stream = a.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, *map_w, *map_x, a.b, a.y, (int)a.M, (int)a.N, (int)a.K, (int)a.seg_len, a.S,
                              n_row_tiles, n_mblocks, (long long)a.ldy, a.status, a.wait_limit_ns, a.test_flags);
}

struct DecodeEntry {
    DecodeConfig cfg;
    DecodeLaunchFn fn;
    DecodeOccupancyFn occupancy;
};

#ifndef DET_WF
#define DET_WF 0
#endif
#define DEC(MT, WM, RT, WR, SK, KC, ST) \
    { {MT, WM, RT, WR, SK, KC, ST, 0}, &launch_decode_t<MT, WM, RT, WR, SK, KC, ST, DET_WF>, &decode_occupancy_t<MT, WM, RT, WR, SK, KC, ST, DET_WF> }

// Ring depth of a tiling: as many stages as fit in the block's share of shared memory (blocks of at
// most 160 threads run two to an SM), leaving room for the partial tiles; between 2 and 8.
constexpr int auto_stages(int mt, int wm, int rt, int wr, int sk, int kc, int eb)
{
    const int stage = sk * (mt * wm * kc * 4 + rt * wr * kc * eb);
    const int tile_bytes = mt * wm * rt * wr * 4;
    // what the block may use: the SM's 227 KB (half of it for blocks that run two to an SM), less the
    // barriers and alignment slack and, with several segment groups, the partial tiles of up to 8 segments
    const int share = (wm * wr * sk <= 4 ? 113 : 227) * 1024;
    const int budget = share - 1024 - (sk > 1 ? kDecodeMaxSegments * tile_bytes : 0);
    const int n = budget / stage;
    return n > 8 ? 8 : n;
}
#define DEC_AUTO(MT, WM, RT, WR, SK, KC) \
    DEC(MT, WM, RT, WR, SK, KC, (auto_stages(MT, WM, RT, WR, SK, KC, DET_WF == 2 ? 4 : 2)))

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
