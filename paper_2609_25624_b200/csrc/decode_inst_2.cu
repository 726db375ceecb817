// Tilings of the decode kernel for one or more batch classes (all numerically identical).  Compiled once
// per weight format (DET_WF = 0 BF16, 1 FP16, 2 FP32); FP32 weights take twice the shared memory per
// stage, so their lists use narrower stages.
#include "decode_kernel.cuh"

namespace detlin {
using namespace decode_detail;

#define DET_TABLE_NAME2(cls, wf) DET_TABLE_NAME(cls, wf)

#if DET_WF == 2
static const DecodeEntry kEntries4[] = {
    DEC(8, 2, 6, 4, 128, 4, 4),
    DEC(8, 2, 8, 4, 128, 4, 4),
    DEC(8, 2, 10, 4, 128, 3, 4),
    DEC(8, 2, 12, 4, 128, 3, 4),
    DEC(8, 2, 14, 4, 128, 3, 4),
    DEC(8, 2, 8, 4, 256, 3, 4),
    DEC(8, 2, 12, 4, 256, 3, 4),
    DEC(8, 2, 14, 4, 256, 3, 4),
};
#else
static const DecodeEntry kEntries4[] = {
    DEC(8, 2, 6, 4, 256, 4, 4),
    DEC(8, 2, 8, 4, 256, 4, 4),
    DEC(8, 2, 10, 4, 256, 3, 4),
    DEC(8, 2, 12, 4, 256, 3, 4),
    DEC(8, 2, 14, 4, 256, 3, 4),
    DEC(8, 2, 16, 4, 256, 3, 4),
};
#endif
extern const DecodeClassTable DET_TABLE_NAME2(4, DET_WF) = {kEntries4, (int)(sizeof(kEntries4) / sizeof(kEntries4[0]))};

}  // namespace detlin
