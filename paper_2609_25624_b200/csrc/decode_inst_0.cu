// Tilings of the decode kernel for one or more batch classes (all numerically identical).  Compiled once
// per weight format (DET_WF = 0 BF16, 1 FP16, 2 FP32); FP32 weights take twice the shared memory per
// stage, so their lists use narrower stages.
#include "decode_kernel.cuh"

namespace detlin {
using namespace decode_detail;

#define DET_TABLE_NAME2(cls, wf) DET_TABLE_NAME(cls, wf)

#if DET_WF == 2
static const DecodeEntry kEntries0[] = {
    DEC(1, 1, 4, 4, 256, 6, 1),
    DEC(1, 1, 8, 4, 128, 6, 1),
    DEC(1, 1, 8, 2, 256, 4, 1),
    DEC(1, 1, 2, 4, 256, 8, 1),
    DEC(1, 1, 8, 4, 256, 3, 1),
    DEC(1, 1, 16, 2, 128, 4, 1),
};
#else
static const DecodeEntry kEntries0[] = {
    DEC(1, 1, 4, 4, 256, 8, 1),
    DEC(1, 1, 8, 4, 256, 6, 1),
    DEC(1, 1, 8, 2, 256, 6, 1),
    DEC(1, 1, 16, 2, 256, 4, 1),
    DEC(1, 1, 2, 4, 256, 8, 1),
};
#endif
extern const DecodeClassTable DET_TABLE_NAME2(0, DET_WF) = {kEntries0, (int)(sizeof(kEntries0) / sizeof(kEntries0[0]))};

#if DET_WF == 2
static const DecodeEntry kEntries1[] = {
    DEC(2, 1, 4, 4, 256, 6, 1),
    DEC(2, 1, 8, 4, 128, 6, 1),
    DEC(2, 1, 8, 2, 256, 4, 1),
    DEC(2, 1, 2, 4, 256, 8, 1),
    DEC(2, 1, 8, 4, 256, 3, 1),
    DEC(2, 1, 16, 2, 128, 4, 1),
};
#else
static const DecodeEntry kEntries1[] = {
    DEC(2, 1, 4, 4, 256, 8, 1),
    DEC(2, 1, 8, 4, 256, 6, 1),
    DEC(2, 1, 8, 2, 256, 6, 1),
    DEC(2, 1, 16, 2, 256, 4, 1),
    DEC(2, 1, 2, 4, 256, 8, 1),
};
#endif
extern const DecodeClassTable DET_TABLE_NAME2(1, DET_WF) = {kEntries1, (int)(sizeof(kEntries1) / sizeof(kEntries1[0]))};

#if DET_WF == 2
static const DecodeEntry kEntries2[] = {
    DEC(4, 1, 4, 4, 256, 4, 1),
    DEC(4, 1, 8, 4, 128, 4, 1),
    DEC(4, 1, 6, 4, 128, 5, 1),
    DEC(4, 1, 14, 4, 128, 3, 1),
    DEC(4, 1, 8, 2, 128, 6, 1),
    DEC(4, 1, 8, 4, 256, 3, 1),
    DEC(4, 1, 6, 4, 256, 4, 1),
};
#else
static const DecodeEntry kEntries2[] = {
    DEC(4, 1, 4, 4, 256, 6, 1),
    DEC(4, 1, 8, 4, 256, 4, 1),
    DEC(4, 1, 6, 4, 256, 5, 1),
    DEC(4, 1, 14, 4, 256, 3, 1),
    DEC(4, 1, 8, 2, 256, 6, 1),
    DEC(4, 1, 16, 2, 256, 4, 1),
};
#endif
extern const DecodeClassTable DET_TABLE_NAME2(2, DET_WF) = {kEntries2, (int)(sizeof(kEntries2) / sizeof(kEntries2[0]))};

}  // namespace detlin
