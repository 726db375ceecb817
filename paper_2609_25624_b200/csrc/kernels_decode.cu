// Decode kernel dispatch: picks one of the compiled tilings for a shape.  The choice only changes
// the schedule (tile sizes, warp counts and ring depth are numerically inert: supplement C on
// rule R2), so it may read the SM count and the occupancy; the reduction order never does.
#include <cmath>

#include "decode_kernel.cuh"

namespace detlin {

namespace {

using decode_detail::DecodeEntry;

#define DET_TABLE_ROW(wf)                                                                                  \
    { &DET_TABLE_NAME(0, wf), &DET_TABLE_NAME(1, wf), &DET_TABLE_NAME(2, wf), &DET_TABLE_NAME(3, wf), \
      &DET_TABLE_NAME(4, wf), &DET_TABLE_NAME(5, wf) }

const DecodeClassTable* class_table(int wfmt, int cls)
{
    static const DecodeClassTable* const t[3][6] = {DET_TABLE_ROW(0), DET_TABLE_ROW(1), DET_TABLE_ROW(2)};
    return t[wfmt][cls];
}

int m_class(int64_t M) { return M <= 1 ? 0 : M <= 2 ? 1 : M <= 4 ? 2 : M <= 8 ? 3 : M <= 16 ? 4 : 5; }

// Predicted time of a tiling in SM clock cycles (schedule heuristic; its constants were fitted to sweeps of
// every tiling over the Llama-3-8B shapes at batch 1 .. 32 on a 148-SM B200, mean loss against the best
// tiling 0.5 %).  A work unit streams rb weight rows (2 K bytes each, at the SM's share of the HBM rate)
// and performs rb * mb * K multiply-adds at the FMA rate of an SM times an efficiency that depends on the
// warp tile; whichever is larger binds.  Units resident on one SM share it.  Fewer than eight consumer
// warps per SM hide latency badly; every unit pays for its lane trees (one per segment) and, with several
// segment groups, for the fold through shared memory.
double tiling_cost(const DecodeEntry& e, int64_t M, int64_t N, int64_t K, int S, int sm_count)
{
    const DecodeConfig& c = e.cfg;
    const int occ = e.occupancy(S);
    if (occ <= 0) return 1e300;
    const int64_t rb = (int64_t)c.rt * c.wr, mb = (int64_t)c.mt * c.wm;
    const int64_t mblocks = (M + mb - 1) / mb;
    const int64_t units = ((N + rb - 1) / rb) * mblocks;
    const int64_t rounds = (units + (int64_t)sm_count * occ - 1) / ((int64_t)sm_count * occ);
    const int64_t per_sm = (units + sm_count - 1) / sm_count;
    const double resident = (double)(per_sm < occ ? per_sm : occ);
    const double warps = resident * c.wm * c.wr * c.sk;
    double eff = c.mt >= 8 ? 0.707 : c.mt == 4 ? 0.70 : c.mt == 2 ? 0.345 : 0.2;
    if (c.kc >= 512 && c.mt >= 8) eff *= 1.2;          // half as many stage boundaries; smaller tiles prefer a deeper ring
    if (c.kc <= 128) eff *= 0.9;
    const double latency = warps >= 8.0 ? 1.0 : 8.0 / warps;
    const double fma = (double)rb * (double)mb * (double)K / 128.0 / eff * resident;
    // weights from HBM at 22.5 bytes per clock and SM; the unit's activations come again from L2 for every unit
    const double hbm = ((double)rb * (double)K * 2.0 / 22.5 + 0.06 * (double)mb * (double)K * 4.0 / 64.0) * resident;
    const double body = (fma > hbm ? fma : hbm) * latency;
    const double overhead = (double)S * 1020.0 * ((double)(mb * rb) / 896.0) + (c.sk > 1 ? 1500.0 : 0.0);
    return (double)rounds * (body + overhead);
}

// Tilings that can serve batch size M: those of M's own class and, for M > 8, the 8-row tilings
// (the batch is then walked in blocks of 8 rows that run side by side).
int candidate_classes(int64_t M, int* out)
{
    const int cls = m_class(M);
    int n = 0;
    out[n++] = cls;
    if (cls > 3) out[n++] = 3;
    return n;
}

}  // namespace

int decode_num_variants()
{
    int n = 0;
    for (int c = 0; c < 6; ++c) n = class_table(0, c)->count > n ? class_table(0, c)->count : n;
    return n;
}

// variant 0 = automatic; variant v >= 1 = the v-th tiling, among those that can run the shape, for this
// batch size (own class first, then the 8-row tilings when M > 8).  A tiling whose segment groups do
// not divide S, or that does not fit the device, cannot run the shape and is not counted.
bool decode_config_for(int64_t M, int64_t N, int64_t K, int S, int wfmt, int variant, DecodeConfig* out)
{
    int classes[2];
    const int n_classes = candidate_classes(M, classes);
    if (variant < 0 || S < 1 || S > kDecodeMaxSegments) return false;
    int sms = 148;
    if (variant == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
            sms = 148;
    }
    int pick_cls = classes[0], pick = -1, seen = 0;
    double best = 1e299;
    for (int ci = 0; ci < n_classes && (variant == 0 || pick < 0); ++ci) {
        const DecodeClassTable* t = class_table(wfmt, classes[ci]);
        for (int i = 0; i < t->count; ++i) {
            if (variant == 0) {
                const double c = tiling_cost(t->entries[i], M, N, K, S, sms);
                if (c < best) { best = c; pick_cls = classes[ci]; pick = i; }
            } else if (t->entries[i].occupancy(S) > 0 && ++seen == variant) {
                pick_cls = classes[ci];
                pick = i;
                break;
            }
        }
    }
    if (pick < 0) return false;
    *out = class_table(wfmt, pick_cls)->entries[pick].cfg;
    out->id = pick_cls * 64 + pick;
    return true;
}

int decode_config_occupancy(int wfmt, const DecodeConfig& cfg, int S)
{
    return class_table(wfmt, cfg.id / 64)->entries[cfg.id % 64].occupancy(S);
}

cudaError_t launch_decode(const LaunchArgs& a, const DecodeConfig& cfg, const CUtensorMap* map_w, const CUtensorMap* map_x)
{
    return class_table(a.wfmt, cfg.id / 64)->entries[cfg.id % 64].fn(a, map_w, map_x);
}

}  // namespace detlin
