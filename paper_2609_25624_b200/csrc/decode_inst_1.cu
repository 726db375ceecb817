// Tilings of the decode kernel for one or more batch classes (all numerically identical).
#include "decode_kernel.cuh"

namespace detlin {
using namespace decode_detail;

static const DecodeEntry kEntries3[] = {
    DEC(8, 1, 4, 4, 256, 5, 1),
    DEC(8, 1, 6, 4, 256, 4, 1),
    DEC(8, 1, 8, 4, 256, 4, 1),
    DEC(8, 1, 10, 4, 256, 3, 1),
    DEC(8, 1, 12, 4, 256, 3, 4),
    DEC(8, 1, 14, 4, 256, 3, 4),
    DEC(8, 1, 16, 4, 256, 3, 4),
    DEC(8, 1, 8, 2, 256, 6, 1),
};
const DecodeClassTable kDecodeClass3 = {kEntries3, 8};

}  // namespace detlin
