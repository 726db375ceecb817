// Shape -> order parameters.  Pure host integer arithmetic; no device query may influence any
// numeric parameter (rule R2: the configuration is a pure function of (M, N, K); rule R3: the split
// factor is shape-pure; rule R4: inside the decode bucket nothing depends on M).
#include "internal.h"

namespace detlin {

static int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Segment layout for a requested split: boundaries on multiples of the granule, every segment
// non-empty.
static void segments_for(int64_t K, int64_t s_req, int64_t* seg_len, int64_t* S)
{
    const int64_t n_gran = ceil_div(K, kSegmentGranule);
    const int64_t per_seg = ceil_div(n_gran, s_req < n_gran ? s_req : n_gran);
    *seg_len = per_seg * kSegmentGranule;
    *S = ceil_div(n_gran, per_seg);
}

// Requested split factor before clamping to what K allows.
//  decode : 1 when N >= 16384 (that many weight rows keep every SM busy on their own; the paper's
//           lm_head likewise takes no split), otherwise 2: two segments let one thread block keep
//           eight warps busy on a single 28-row weight tile -- 4096 rows over 148 SMs -- and fold
//           the two segment sums inside the block, without a workspace or a second launch.  Never
//           reads M (rule R4).  Measured on B200 before the freeze: against no split the small
//           matrices gain up to 1.9x at batch 4 .. 8; four segments cost the large batches 5 %
//           (one more lane tree per segment and output) and gain nothing further.
//  prefill: the request in 1..16 that minimises  rounds * (seg_len + overhead) * occupancy_factor
//           where tiles counts 128x128 output tiles, units = tiles * S, rounds = ceil(units / 148),
//           overhead = 8 k-steps per work unit plus 32 when partials have to be written and combined,
//           and occupancy_factor = 9 when units <= 148 (one block per SM) else 8; ties go to the
//           larger split.  148 and the overheads were measured once on a B200 and are frozen
//           constants of the order definition: the rule is a pure function of (M, N, K) and never
//           reads the device (rule R2: configurations are tuned once, offline, and then pinned).
static int split_request(int64_t M, int64_t N, int64_t K)
{
    if (M <= kDecodeMaxM) return N >= kDecodeNoSplitRows ? 1 : 2;
    const int64_t tiles = ceil_div(M, 128) * ceil_div(N, 128);
    int best = 1;
    int64_t best_cost = -1;
    for (int s_req = 1; s_req <= 16; ++s_req) {
        int64_t seg_len, S;
        segments_for(K, s_req, &seg_len, &S);
        const int64_t units = tiles * S;
        const int64_t rounds = ceil_div(units, 148);
        const int64_t cost = rounds * (seg_len + (S > 1 ? 40 : 8)) * (units <= 148 ? 9 : 8);
        if (best_cost < 0 || cost <= best_cost) { best_cost = cost; best = s_req; }
    }
    return best;
}

det_status_t fill_params(int64_t M, int64_t N, int64_t K, det_linear_params_t* out)
{
    if (!out) { set_error("params: out is NULL"); return DET_ERR_INVALID_ARG; }
    if (M < 1 || N < 1 || K < 1) {
        set_error("params: M, N, K must be >= 1 (got %lld, %lld, %lld)", (long long)M, (long long)N, (long long)K);
        return DET_ERR_INVALID_ARG;
    }
    const int64_t lim = (int64_t)1 << 31;
    if (M >= lim || N >= lim || K >= lim || M * N >= ((int64_t)1 << 40)) {
        set_error("params: shape too large (each dimension < 2^31, M*N < 2^40)");
        return DET_ERR_UNSUPPORTED_SHAPE;
    }
    det_linear_params_t p{};
    p.M = M; p.N = N; p.K = K;
    if (M <= kDecodeMaxM) { p.bucket = 0; p.V = 4; p.L = 32; p.P = 1; }
    else                  { p.bucket = 1; p.V = 1; p.L = 1;  p.P = 1; }
    int64_t seg_len, S;
    segments_for(K, split_request(M, N, K), &seg_len, &S);
    p.seg_len = seg_len;
    p.S = (int32_t)S;
    p.order_version = kOrderVersion;
    p.weight_format = DET_WEIGHT_BF16;
    p.kernel = (K % 8 == 0) ? (p.bucket == 0 ? kKernelDecode : kKernelPrefill) : kKernelGeneric;
    // the decode bucket folds its segments inside the kernels; the prefill bucket combines in a second pass
    p.workspace_bytes = (p.bucket == 1 && p.S > 1) ? (uint64_t)4 * (uint64_t)p.S * (uint64_t)M * (uint64_t)N : 0;
    *out = p;
    return DET_OK;
}

}  // namespace detlin
