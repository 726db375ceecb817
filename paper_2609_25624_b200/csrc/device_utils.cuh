// Device helpers shared by the kernels: the register upcast of Eq. 2 for each weight format and the
// adjacent-first lane tree.  (Rule R1: every multiply-accumulate in the kernels is an explicit fma
// intrinsic -- __fmaf_rn, __ffma2_rn -- never the compiler's contraction.)
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cstdint>

namespace detlin {

// Weight formats: WF = 0 BF16, 1 FP16, 2 FP32 (det_weight_format_t).  A 32-bit word of a 16-bit
// format holds elements (k, k+1) in its (low, high) half; both widenings are exact.
template <int WF>
__device__ __forceinline__ float up16_lo(uint32_t w)
{
    if (WF == 0) return __uint_as_float(w << 16);
    return __half2float(__ushort_as_half((unsigned short)(w & 0xffffu)));
}
template <int WF>
__device__ __forceinline__ float up16_hi(uint32_t w)
{
    if (WF == 0) return __uint_as_float(w & 0xffff0000u);
    return __half2float(__ushort_as_half((unsigned short)(w >> 16)));
}
template <int WF> struct WeightElem { typedef uint16_t type; static constexpr int bytes = 2; };
template <> struct WeightElem<2> { typedef float type; static constexpr int bytes = 4; };
template <int WF>
__device__ __forceinline__ float up_elem(typename WeightElem<WF>::type v)
{
    if constexpr (WF == 2) return v;
    else if constexpr (WF == 1) return __half2float(__ushort_as_half(v));
    else return __uint_as_float(((uint32_t)v) << 16);
}

// Balanced tree over the 32 lanes of a warp, adjacent lanes first (xor 1, 2, 4, 8, 16 in that
// order).  fadd is commutative, so both partners compute identical bits and every lane ends with
// the tree's root.
__device__ __forceinline__ float lane_tree_sum(float a)
{
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) a = __fadd_rn(a, __shfl_xor_sync(0xffffffffu, a, d));
    return a;
}

}  // namespace detlin
