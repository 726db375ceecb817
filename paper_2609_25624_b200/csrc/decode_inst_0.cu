// Tilings of the decode kernel for one or more batch classes (all numerically identical).
#include "decode_kernel.cuh"

namespace detlin {
using namespace decode_detail;

static const DecodeEntry kEntries0[] = {
    DEC(1, 1, 4, 4, 256, 8, 1),
    DEC(1, 1, 8, 4, 256, 6, 1),
    DEC(1, 1, 8, 2, 256, 6, 1),
    DEC(1, 1, 16, 2, 256, 4, 1),
    DEC(1, 1, 2, 4, 256, 8, 1),
};
const DecodeClassTable kDecodeClass0 = {kEntries0, 5};

static const DecodeEntry kEntries1[] = {
    DEC(2, 1, 4, 4, 256, 8, 1),
    DEC(2, 1, 8, 4, 256, 6, 1),
    DEC(2, 1, 8, 2, 256, 6, 1),
    DEC(2, 1, 16, 2, 256, 4, 1),
    DEC(2, 1, 2, 4, 256, 8, 1),
};
const DecodeClassTable kDecodeClass1 = {kEntries1, 5};

static const DecodeEntry kEntries2[] = {
    DEC(4, 1, 4, 4, 256, 6, 1),
    DEC(4, 1, 8, 4, 256, 4, 1),
    DEC(4, 1, 6, 4, 256, 5, 1),
    DEC(4, 1, 14, 4, 256, 3, 1),
    DEC(4, 1, 8, 2, 256, 6, 1),
    DEC(4, 1, 16, 2, 256, 4, 1),
};
const DecodeClassTable kDecodeClass2 = {kEntries2, 6};

}  // namespace detlin
