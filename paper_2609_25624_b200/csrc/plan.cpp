// Shape -> order parameters.  Pure host integer arithmetic; no device query may influence any
// numeric parameter (rule R2: the configuration is a pure function of (M, N, K); rule R3: the split
// factor is shape-pure; rule R4: inside the decode bucket nothing depends on M).
#include "internal.h"

namespace detlin {

static int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Requested split factor before clamping to what K allows.
//  decode : no split once N alone provides 4096 rows of parallel work (like the paper's lm_head,
//           which "prefers no split"); below that the smallest power of two with N*S >= 4096.
//           Never reads M.
//  prefill: the smallest power of two S <= 16 that yields at least 1024 (128x128 tile, segment)
//           work units, while keeping segments at least 512 elements long.  The constants were
//           tuned once for a 148-SM part and are frozen; the SM count is never read.
static int split_request(int64_t M, int64_t N, int64_t K)
{
    int s = 1;
    if (M <= kDecodeMaxM) {
        while (N * s < 4096) s *= 2;
        return s;
    }
    const int64_t tiles = ceil_div(M, 128) * ceil_div(N, 128);
    while (s < 16 && tiles * s < 1024 && K / (2 * s) >= 512) s *= 2;
    return s;
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
    else                  { p.bucket = 1; p.V = 2; p.L = 1;  p.P = 2; }
    const int64_t s_req = split_request(M, N, K);
    const int64_t n_gran = ceil_div(K, kSegmentGranule);
    const int64_t per_seg = ceil_div(n_gran, s_req < n_gran ? s_req : n_gran);
    p.seg_len = per_seg * kSegmentGranule;
    p.S = (int32_t)ceil_div(n_gran, per_seg);
    p.order_version = kOrderVersion;
    p.kernel = (K % 8 == 0) ? (p.bucket == 0 ? kKernelDecode : kKernelPrefill) : kKernelGeneric;
    p.workspace_bytes = p.S > 1 ? (uint64_t)4 * (uint64_t)p.S * (uint64_t)M * (uint64_t)N : 0;
    *out = p;
    return DET_OK;
}

}  // namespace detlin
