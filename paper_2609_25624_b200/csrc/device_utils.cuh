// Device helpers shared by the kernels: the register upcast of Eq. 2, explicit IEEE FMA / add (rule
// R1: never rely on the compiler's contraction), packed FP32x2 FMA, and the adjacent-first lane tree.
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cstdint>

namespace detlin {

// up(): BF16 bit pattern -> binary32 with the pattern in the high half (exact).
__device__ __forceinline__ float up_bf16(uint16_t h) { return __uint_as_float(((uint32_t)h) << 16); }
// A 32-bit word holding two BF16 values (little endian: element k in the low half, k+1 in the high).
__device__ __forceinline__ float up_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float up_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

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

// fma.rn.f32x2: two independent IEEE-754 binary32 fused multiply-adds (round to nearest even, no
// flush to zero) in one instruction; each half behaves exactly like fma.rn.f32.
__device__ __forceinline__ void ffma2(unsigned long long& acc, unsigned long long a, unsigned long long b)
{
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}
// Two FP32 values as one 64-bit FP32x2 operand (low half = first element).  Written with integer
// operations so that the compiler can place the halves straight into a register pair.
__device__ __forceinline__ unsigned long long pack2(float lo, float hi)
{
    return ((unsigned long long)__float_as_uint(hi) << 32) | (unsigned long long)__float_as_uint(lo);
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi)
{
    lo = __uint_as_float((unsigned int)v);
    hi = __uint_as_float((unsigned int)(v >> 32));
}
// A 32-bit word holding BF16 elements (k, k+1) -> the FP32x2 operand (up(k), up(k+1)).
__device__ __forceinline__ unsigned long long up_pair(uint32_t w)
{
    return ((unsigned long long)(w & 0xffff0000u) << 32) | (unsigned long long)(w << 16);
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
