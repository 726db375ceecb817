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

// Predicted cost of a tiling: the rows of W (padded to whole tiles) that the busiest SM has to
// process, corrected for how well the tile amortises shared-memory traffic and for having too few
// warps resident to hide latency.  Heuristic, checked against a sweep of every tiling on the Llama-3-8B
// shapes at batch sizes 1 .. 64 (mean loss against the best tiling 1.6 %, 0.6 % on the benchmark's sizes).
double tiling_cost(const DecodeEntry& e, int64_t M, int64_t N, int S, int sm_count)
{
    const DecodeConfig& c = e.cfg;
    const int occ = e.occupancy();
    if (occ <= 0) return 1e300;
    const int64_t rb = (int64_t)c.rt * c.wr, mb = (int64_t)c.mt * c.wm;
    const int64_t units = ((N + rb - 1) / rb) * S * ((M + mb - 1) / mb);
    const int64_t per_sm = (units + sm_count - 1) / sm_count;
    const double outputs = (double)per_sm * (double)rb * (double)mb;      // padded outputs on the busiest SM
    const int64_t resident = per_sm < occ ? per_sm : occ;
    const double warps = (double)resident * c.wm * c.wr;
    const double latency_penalty = warps >= 8.0 ? 1.0 : 8.0 / warps;
    // shared-memory wavefronts per packed FMA of an (mt x rt) warp tile
    const double r = (4.0 * c.mt + 2.0 * c.rt) / ((double)c.mt * c.rt);
    const double weight = M >= 5 ? 0.35 : 0.35 * (double)(M + 3) / 8.0;
    // walking the batch in several blocks re-reads the weights from L2 and repeats the epilogue; the
    // blocks of one row tile run side by side, so the cost grows much more slowly than their number
    const double block_penalty = 1.0 + 0.12 * pow((double)((M + mb - 1) / mb - 1), 0.3);
    return outputs * latency_penalty * block_penalty * (1.0 + weight * r);
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

// variant 0 = automatic; variant v >= 1 = the v-th candidate tiling for this batch size (own class
// first, then the 8-row tilings when M > 8).
bool decode_config_for(int64_t M, int64_t N, int64_t K, int S, int wfmt, int variant, DecodeConfig* out)
{
    (void)K;
    int classes[2];
    const int n_classes = candidate_classes(M, classes);
    int total = 0;
    for (int i = 0; i < n_classes; ++i) total += class_table(wfmt, classes[i])->count;
    if (variant < 0 || variant > total) return false;
    int pick_cls = classes[0], pick = 0;
    if (variant == 0) {
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
            sms = 148;
        double best = 1e301;
        for (int ci = 0; ci < n_classes; ++ci) {
            const DecodeClassTable* t = class_table(wfmt, classes[ci]);
            for (int i = 0; i < t->count; ++i) {
                const double c = tiling_cost(t->entries[i], M, N, S, sms);
                if (c < best) { best = c; pick_cls = classes[ci]; pick = i; }
            }
        }
    } else {
        int v = variant - 1;
        for (int ci = 0; ci < n_classes; ++ci) {
            const DecodeClassTable* t = class_table(wfmt, classes[ci]);
            if (v < t->count) { pick_cls = classes[ci]; pick = v; break; }
            v -= t->count;
        }
    }
    *out = class_table(wfmt, pick_cls)->entries[pick].cfg;
    out->id = pick_cls * 64 + pick;
    return true;
}

int decode_config_occupancy(int wfmt, const DecodeConfig& cfg)
{
    return class_table(wfmt, cfg.id / 64)->entries[cfg.id % 64].occupancy();
}

cudaError_t launch_decode(const LaunchArgs& a, const CUtensorMap* map_w, const CUtensorMap* map_x)
{
    DecodeConfig cfg;
    if (!decode_config_for(a.M, a.N, a.K, a.S, a.wfmt, a.variant, &cfg)) return cudaErrorInvalidValue;
    return class_table(a.wfmt, cfg.id / 64)->entries[cfg.id % 64].fn(a, map_w, map_x);
}

}  // namespace detlin
