// The closeness rule and the element types it is applied to, shared by the kernels that
// judge elements (paper Section 3.1 Eq. 1 and Section 4.3: the candidate's output must match
// the reference output; the formula is fixed by this library, see evo.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "evo.h"
#include "plan.h"

namespace evo {

// Exact form, every special case: d = |c - r|, tol = atol + rtol*|r| (one rounding per
// operation, no fused multiply-add), close = (c == r) or (d finite and d <= tol).
__device__ __forceinline__ bool rule_mismatch(float c, float r, float atol, float rtol) {
    const float d = fabsf(__fsub_rn(c, r));
    const float tol = __fadd_rn(atol, __fmul_rn(rtol, fabsf(r)));
    const bool d_finite = d < __int_as_float(0x7f800000);          // false for NaN and Inf
    const bool close = (c == r) || (d_finite && d <= tol);
    return !close;
}

// Element types: how a 16-byte vector and a single stored value widen (exactly) to binary32.
template <int DT> struct Elem;
template <> struct Elem<EVO_F32> {
    static constexpr int kPerVec = 4;
    static constexpr int kVecs = kEpt / 4;          // 16-byte vectors per thread per tile
    using T = float;
    static __device__ __forceinline__ float at(const uint4& v, int i) {
        return __uint_as_float(i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w);
    }
    static __device__ __forceinline__ float widen(T x) { return x; }
};
template <> struct Elem<EVO_F16> {
    static constexpr int kPerVec = 8;
    static constexpr int kVecs = kEpt / 8;
    using T = __half;
    static __device__ __forceinline__ float at(const uint4& v, int i) {
        const uint32_t w = (i >> 1) == 0 ? v.x : (i >> 1) == 1 ? v.y : (i >> 1) == 2 ? v.z : v.w;
        const __half2 h = *reinterpret_cast<const __half2*>(&w);
        return (i & 1) ? __high2float(h) : __low2float(h);
    }
    static __device__ __forceinline__ float widen(T x) { return __half2float(x); }
};
template <> struct Elem<EVO_BF16> {
    static constexpr int kPerVec = 8;
    static constexpr int kVecs = kEpt / 8;
    using T = __nv_bfloat16;
    static __device__ __forceinline__ float at(const uint4& v, int i) {
        const uint32_t w = (i >> 1) == 0 ? v.x : (i >> 1) == 1 ? v.y : (i >> 1) == 2 ? v.z : v.w;
        return __uint_as_float((i & 1) ? (w & 0xffff0000u) : (w << 16));
    }
    static __device__ __forceinline__ float widen(T x) { return __bfloat162float(x); }
};


}  // namespace evo
