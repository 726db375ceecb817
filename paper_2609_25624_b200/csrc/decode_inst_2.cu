// Tilings of the decode kernel for one or more batch classes (all numerically identical).
#include "decode_kernel.cuh"

namespace detlin {
using namespace decode_detail;

static const DecodeEntry kEntries4[] = {
    DEC(8, 2, 6, 4, 256, 4, 4),
    DEC(8, 2, 8, 4, 256, 4, 4),
    DEC(8, 2, 10, 4, 256, 3, 4),
    DEC(8, 2, 12, 4, 256, 3, 4),
    DEC(8, 2, 14, 4, 256, 3, 4),
    DEC(8, 2, 16, 4, 256, 3, 4),
};
const DecodeClassTable kDecodeClass4 = {kEntries4, 6};

}  // namespace detlin
