// Tilings of the decode kernel for one or more batch classes (all numerically identical).
#include "decode_kernel.cuh"

namespace detlin {
using namespace decode_detail;

static const DecodeEntry kEntries5[] = {
    DEC(8, 4, 8, 2, 256, 4, 4),
    DEC(8, 4, 10, 2, 256, 3, 4),
    DEC(8, 4, 12, 2, 256, 3, 4),
    DEC(8, 4, 14, 2, 256, 3, 4),
    DEC(8, 4, 16, 2, 256, 3, 4),
    DEC(8, 4, 8, 3, 256, 3, 4),
};
const DecodeClassTable kDecodeClass5 = {kEntries5, 6};

}  // namespace detlin
