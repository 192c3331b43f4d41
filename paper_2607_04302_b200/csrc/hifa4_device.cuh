// Device-side helpers shared by the HiFA4 kernels: exact HIF4 scale selection
// (Background, "HIF4") on fp32 values that came from 16-bit inputs.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace hifa4 {

struct HeadMap {                       // head -> row of the [Hkv, d] scale table
    short kv_of[256];
};

// ---------------------------------------------------------------------------
// Level-1 scale.  The smallest E6M2 value S = 2^(e-48) (1+M/4) with 7*S >= A.
// With A = f * 2^E, f in [1,2): the candidates 7*S fall at f = 1.09375 (M=1),
// 1.3125 (M=2), 1.53125 (M=3), 1.75 (M=0, next exponent), then M=1 of the next
// exponent, so code = 4*(E+45) + 1 + (number of those four marks f exceeds).
// All comparisons are on the integer significand: exact.
// ---------------------------------------------------------------------------
__device__ __forceinline__ int e6m2_code_for_max(float A)   // A > 0, normal fp32
{
    uint32_t bits = __float_as_uint(A);
    int E = (int)(bits >> 23) - 127;
    uint32_t mant = bits & 0x7FFFFFu;
    int j = 1 + (mant > 0x0C0000u) + (mant > 0x280000u) + (mant > 0x440000u) + (mant > 0x600000u);
    int code = 4 * (E + 45) + j;
    return min(max(code, 0), 255);
}

__device__ __forceinline__ float e6m2_value(int code)       // S
{
    return __uint_as_float(((uint32_t)((code >> 2) + 79) << 23) | ((uint32_t)(code & 3) << 21));
}

// 4/S = RN(4/(4+M)) * 2^(50-e): the four reciprocals all err upward, so a
// round-toward-zero product p * (1/step) lands exactly on j+1/2 for every tie
// of a 16-bit-significand p (checked exhaustively on the host), and
// round-to-nearest-even of that product is the exact nearest code.
__device__ __forceinline__ float e6m2_inv4(int code)        // 4 / S
{
    const int M = code & 3;                                  // 1, .8, 2/3, 4/7 rounded to nearest
    const uint32_t r = M == 0 ? 0x3F800000u : M == 1 ? 0x3F4CCCCDu : M == 2 ? 0x3F2AAAABu : 0x3F124925u;
    return __uint_as_float(r + ((uint32_t)(50 - (code >> 2)) << 23));
}

template <typename T> struct In16;
template <> struct In16<__half> {
    static __device__ __forceinline__ float to_f(uint16_t u) { return __half2float(__ushort_as_half(u)); }
    static __device__ __forceinline__ float round(float x) { return __half2float(__float2half_rn(x)); }
    static __device__ __forceinline__ float round_d(double x) { return __half2float(__double2half(x)); }
};
template <> struct In16<__nv_bfloat16> {
    static __device__ __forceinline__ float to_f(uint16_t u) { return __uint_as_float((uint32_t)u << 16); }
    static __device__ __forceinline__ float round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }
    static __device__ __forceinline__ float round_d(double x) { return __bfloat162float(__double2bfloat16(x)); }
};

}  // namespace hifa4
