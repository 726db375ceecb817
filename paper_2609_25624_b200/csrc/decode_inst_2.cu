// Tilings of the decode kernel for one or more batch classes (all numerically identical).  Compiled once
// per weight format (DET_WF = 0 BF16, 1 FP16, 2 FP32).  A row is (MT, WM, RT, WR, SK, KC): warp tile of MT
// batch rows x RT weight rows, WM x WR warps per segment group, SK segment groups side by side, KC
// elements of k per stage; the ring depth follows from the shared-memory budget.  FP32 weights take
// twice the shared memory per stage, so their stages are 128 elements wide.
#include "decode_kernel.cuh"

namespace detlin {
using namespace decode_detail;

#define DET_TABLE_NAME2(cls, wf) DET_TABLE_NAME(cls, wf)
#if DET_WF == 2
#define KCW(kc) 128
#else
#define KCW(kc) kc
#endif
#define ROW(MT, WM, RT, WR, SK, KC) DEC_AUTO(MT, WM, RT, WR, SK, KCW(KC))

static const DecodeEntry kEntries4[] = {
    ROW(8, 2, 14, 2, 2, 256),
    ROW(8, 2, 14, 1, 2, 256),
    ROW(8, 2, 14, 2, 1, 256),
    ROW(8, 2, 14, 4, 1, 256),
    ROW(8, 2, 14, 4, 1, 512),
    ROW(8, 2, 14, 3, 1, 256),
    ROW(4, 4, 14, 2, 1, 256),
};
extern const DecodeClassTable DET_TABLE_NAME2(4, DET_WF) = {kEntries4, (int)(sizeof(kEntries4) / sizeof(kEntries4[0]))};

}  // namespace detlin

