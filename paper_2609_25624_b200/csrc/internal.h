// Internal declarations shared by the host-side translation units of libdet_linear.
#pragma once
#include <cuda_runtime.h>
#include <cuda.h>
#include <cstdint>
#include <cstddef>
#include "det_linear.h"

namespace detlin {

constexpr int kOrderVersion = 2;
constexpr int kSegmentGranule = 256;   // segment boundaries are multiples of this many k elements
constexpr int64_t kDecodeNoSplitRows = 16384;   // decode bucket: weight matrices with at least this many rows are not split
constexpr int kDecodeMaxSegments = 8;  // most K segments the decode kernel folds inside a thread block
constexpr unsigned long long kDefaultWaitLimitNs = 2000000000ull;   // bound of one device-side wait: 2 s
constexpr int kDecodeMaxM = 64;        // decode bucket edge: rule R2 puts batches of up to 64 rows in the decode bucket

enum KernelId : int { kKernelGeneric = 0, kKernelDecode = 1, kKernelPrefill = 2 };

// Device-side status word written by kernels that give up a bounded wait.
struct DeviceStatus {
    unsigned int timeout_flag;   // nonzero: some wait expired
    unsigned int where;          // which wait (diagnostic)
};

constexpr int kMaxDevices = 64;     // per-device caches (function attributes, symbol addresses)

void set_error(const char* fmt, ...);
det_status_t fill_params(int64_t M, int64_t N, int64_t K, det_linear_params_t* out);

// ---- kernel launchers (defined in the .cu files) -------------------------------------------
struct LaunchArgs {
    const float* x;
    const void* W;        // [N,K] in weight format wfmt
    int wfmt;             // det_weight_format_t
    const float* b;
    float* y;             // final output [M,N], row pitch ldy
    int64_t ldy;          // floats between consecutive rows of y (N unless the plan is a column shard)
    float* partials;      // [S,M,N] when S > 1, else nullptr
    unsigned* tile_counters;   // prefill with S > 1: one zeroed counter per output tile (the TMA-fed kernel folds in place), or nullptr
    int64_t M, N, K;
    int64_t seg_len;
    int S;
    cudaStream_t stream;
    DeviceStatus* status; // device pointer
    int sm_count;
    int max_blocks;       // 0 = automatic
    int variant;          // 0 = automatic
    unsigned long long wait_limit_ns;   // bound of one device-side wait (TMA-fed kernels)
    int test_flags;       // decode kernel test hooks (0 outside the tests)
};

cudaError_t launch_generic(const LaunchArgs& a, int bucket);
// Second pass of split-K: y[m,n] = (((P0 + P1) + P2) + ...) (+ b[n]); rule R3.
cudaError_t launch_combine(const LaunchArgs& a);

// Register-staged prefill kernel (the fallback without an activation workspace; a.variant 15 .. 18 forces 5 .. 8 rows
// per thread).
cudaError_t launch_prefill(const LaunchArgs& a);
// Prefill kernel with both tiles fed by TMA (prefill_tma.cu).  It reads the
// activations from a workspace xT [K][ldt] (x transposed, ldt = M rounded up to a multiple of 4; launch_transpose_x
// writes it).  Tensor maps without swizzle: map_x: xT, box [32][16 tr]; map_w: W [N][K] in its format, box [128][32].
cudaError_t launch_transpose_x(const float* x, float* xT, int64_t M, int64_t K, int64_t ldt, cudaStream_t stream);
cudaError_t launch_prefill_tma(const LaunchArgs& a, int tr, const CUtensorMap* map_w, const CUtensorMap* map_x);
// rows per thread (tile height = 16 x this) the prefill kernel uses for batch size M; schedule only
int prefill_rows_per_thread(int64_t M);
// Fixed-order RMSNorm of M rows of H elements (rmsnorm.cu).
cudaError_t launch_rmsnorm(const float* x, const float* g, float eps, int64_t M, int64_t H, float* y, cudaStream_t stream);
// Fixed-order decode attention (attention.cu); attention_smem_bytes = dynamic shared memory it needs.
size_t attention_smem_bytes(int G, int T, int D);
// test hook: force the number of thread blocks that share one (batch, KV head) row (1, 2, 4, 8, 16; 0 = automatic)
void attention_test_force_split(int c);
// the cluster size the launcher would use on a device with sm_count SMs (pure function of its arguments and of
// the forced split), and the dynamic shared memory of one block for it
int attention_split(int B, int Hkv, int G, int T, int D, int sm_count);
size_t attention_block_smem_bytes(int G, int T, int D, int C);
cudaError_t launch_attention_decode(const float* q, const float* k, const float* v, float scale, int B, int Hq, int Hkv, int T,
                                    int D, float* o, cudaStream_t stream);
// Read `bytes` at buf through L2 (evicts what was there without leaving dirty lines); sink: 4 bytes of device memory.
cudaError_t launch_l2_evict(const void* buf, size_t bytes, unsigned* sink, int sm_count, cudaStream_t stream);
cudaError_t launch_argmax(const float* y, int64_t M, int64_t N, int32_t* idx, cudaStream_t stream);

// Decode-kernel tiling chosen for a shape (numerically inert); used by the host to build the
// tensor maps with matching box sizes.
struct DecodeConfig {
    int mt, wm, rt, wr, sk, kc, stages;   // warp tile (mt x rt), warps (wm x wr) x sk segment groups, k per stage, ring depth
    int id;
};
// S = number of K segments of the order (it only scales the unit count in the schedule's cost model)
bool decode_config_for(int64_t M, int64_t N, int64_t K, int S, int wfmt, int variant, DecodeConfig* out);
int decode_num_variants();
cudaError_t launch_decode(const LaunchArgs& a, const DecodeConfig& cfg, const CUtensorMap* map_w, const CUtensorMap* map_x);
// resident blocks per SM of a tiling on the current device for an order with S segments (schedule information only)
int decode_config_occupancy(int wfmt, const DecodeConfig& cfg, int S);

}  // namespace detlin

struct det_linear_plan {
    det_linear_params_t prm;
    int device;
    int sm_count;
    float* partials;                 // device, S*M*n_count floats or nullptr
    unsigned* tile_counters;         // device, inside the partials allocation (prefill, S > 1) or nullptr
    uint64_t n_tile_counters;
    float* x_t;                      // device, K * roundup(M, 4) floats: x transposed (prefill bucket) or nullptr
    int64_t n_begin, n_count, ldy;   // column shard computed by this plan (0, N, N for a whole layer)
    detlin::DeviceStatus* status;    // device
    float* x_stage;                  // device staging for det_linear_run_host
    float* y_stage;
    int forced_kernel;               // -1 automatic
    int max_blocks;
    int variant;
    unsigned long long wait_limit_ns;
    int test_flags;
    // the decode tiling chosen for this plan (schedule only; cached so that a run does no search)
    detlin::DecodeConfig decode_cfg;
    int decode_cfg_variant;          // variant the cached tiling was chosen for, -1 = none yet
    // tensor-map cache for the decode kernel (keyed by the pointers they were built for)
    const void* map_w_ptr;
    const void* map_x_ptr;
    int map_cfg_id;
    CUtensorMap map_w;
    CUtensorMap map_x;
};
