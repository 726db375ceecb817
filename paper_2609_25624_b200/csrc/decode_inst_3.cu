// Tilings of the decode kernel for one or more batch classes (all numerically identical).  Compiled once
// per weight format (DET_WF = 0 BF16, 1 FP16, 2 FP32); FP32 weights take twice the shared memory per
// stage, so their lists use narrower stages.
#include "decode_kernel.cuh"

namespace detlin {
using namespace decode_detail;

#define DET_TABLE_NAME2(cls, wf) DET_TABLE_NAME(cls, wf)

#if DET_WF == 2
static const DecodeEntry kEntries5[] = {
    DEC(8, 4, 8, 2, 128, 4, 4),
    DEC(8, 4, 10, 2, 128, 3, 4),
    DEC(8, 4, 12, 2, 128, 3, 4),
    DEC(8, 4, 14, 2, 128, 3, 4),
    DEC(8, 4, 16, 2, 128, 3, 4),
    DEC(8, 4, 8, 2, 256, 3, 4),
    DEC(8, 4, 12, 2, 256, 3, 4),
    DEC(8, 4, 14, 2, 256, 3, 4),
    DEC(8, 4, 16, 2, 256, 3, 4),
};
#else
static const DecodeEntry kEntries5[] = {
    DEC(8, 4, 8, 2, 256, 4, 4),
    DEC(8, 4, 10, 2, 256, 3, 4),
    DEC(8, 4, 12, 2, 256, 3, 4),
    DEC(8, 4, 14, 2, 256, 3, 4),
    DEC(8, 4, 16, 2, 256, 3, 4),
    DEC(8, 4, 8, 3, 256, 3, 4),
};
#endif
extern const DecodeClassTable DET_TABLE_NAME2(5, DET_WF) = {kEntries5, (int)(sizeof(kEntries5) / sizeof(kEntries5[0]))};

}  // namespace detlin
