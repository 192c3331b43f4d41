// Device-side helpers shared by the HiFA4 kernels: exact HIF4 scale selection
// (Background, "HIF4") on fp32 values that came from 16-bit inputs.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "hifa4_ptx.cuh"

namespace hifa4 {

using namespace ptx;

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

// 16-bit input pairs <-> fp32, and the rounding of a smoothed pair back to the input dtype.
template <typename T> struct Pair16;
template <> struct Pair16<__nv_bfloat16> {
    static __device__ __forceinline__ void unpack(uint32_t w, float& lo, float& hi)
    {
        lo = __uint_as_float(w << 16);
        hi = __uint_as_float(w & 0xFFFF0000u);
    }
    static __device__ __forceinline__ uint32_t round_pack(float lo, float hi)
    {
        uint32_t r;
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
        return r;
    }
};
template <> struct Pair16<__half> {
    static __device__ __forceinline__ void unpack(uint32_t w, float& lo, float& hi)
    {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w));
        lo = f.x;
        hi = f.y;
    }
    static __device__ __forceinline__ uint32_t round_pack(float lo, float hi)
    {
        uint32_t r;
        asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
        return r;
    }
};

// ---------------------------------------------------------------------------
// HIF4 quantization of values that are exact in a 16-bit input type, one level-2 unit (8 elements =
// two level-3 subgroups) at a time.  All arithmetic is exact:
//   q = RZ(x * RN(4/S))             lands exactly on j + 1/2 on every rounding tie (see e6m2_inv4)
//   y = q + 1.5 * 2^(23+k)          rounds q to the nearest multiple of 2^k, ties to even:
//                                   bits(y) - bits(magic) = m, the signed element code under shift k
//   v = fma(y, S/4, -magic * S/4)   = m * 2^k * S/4, the dequantized value
// The shift of a subgroup with maximum At is need = max(bits(At) - bits(1.75 S) - 1 + 2^23, 0) >> 23;
// the pair rule is a = (n0 + n1 + 2) >> 2, k = max(need, a).
// ---------------------------------------------------------------------------
struct Hif4Group {                  // constants of a 64-element group whose maximum magnitude is A
    int code;                       // E6M2 code of the scale S (A = 0: code 0, an all-zero group)
    float top;                      // 7 S; larger magnitudes saturate (only above the E6M2 range)
    uint64_t inv44, s44;            // {4/S, 4/S}, {S/4, S/4}
    uint32_t c0_bits;               // bits(-1.5 * 2^23 * S/4)
    int tadd;
};
__device__ __forceinline__ Hif4Group hif4_group(float A)
{
    Hif4Group g;
    g.code = e6m2_code_for_max(A);
    const float S = e6m2_value(g.code);
    g.top = 7.f * S;
    const float inv4 = e6m2_inv4(g.code);
    const float S4 = __uint_as_float(__float_as_uint(S) - (2u << 23));
    g.inv44 = pack2(inv4, inv4);
    g.s44 = pack2(S4, S4);
    g.c0_bits = __float_as_uint(-12582912.f * S4);
    g.tadd = (1 << 23) - ((int)__float_as_uint(1.75f * S) + 1);
    return g;
}
// x: the unit's values (already clamped to +-top), a0 / a1: the maxima of its two subgroups.  w: BF16 image of
// the dequantized values (element 2i in the low half of word i); y: the biased quotients (the low byte of
// bits(y[i]) is the signed element code); a, k0, k1: level-2 shift and the subgroups' total shifts.
__device__ __forceinline__ void hif4_unit(const float (&x)[8], float a0, float a1, const Hif4Group& g,
                                          uint32_t (&w)[4], float (&y)[8], int& a, int& k0, int& k1)
{
    const int n0 = max((int)__float_as_uint(a0) + g.tadd, 0) >> 23;
    const int n1 = max((int)__float_as_uint(a1) + g.tadd, 0) >> 23;
    a = (n0 + n1 + 2) >> 2;
    k0 = max(n0, a);
    k1 = max(n1, a);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t ks = (uint32_t)(h ? k1 : k0) << 23;
        const uint32_t magic_bits = 0x4B400000u + ks;
        const float magic = __uint_as_float(magic_bits), ck = __uint_as_float(g.c0_bits + ks);
        const uint64_t mm = pack2(magic, magic), cc = pack2(ck, ck);
        const uint64_t y01 = add2(mul2_rz(pack2(x[4 * h], x[4 * h + 1]), g.inv44), mm);
        const uint64_t y23 = add2(mul2_rz(pack2(x[4 * h + 2], x[4 * h + 3]), g.inv44), mm);
        float v0, v1, v2, v3;
        unpack2(fma2(y01, g.s44, cc), v0, v1);
        unpack2(fma2(y23, g.s44, cc), v2, v3);
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w[2 * h]) : "f"(v1), "f"(v0));
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w[2 * h + 1]) : "f"(v3), "f"(v2));
        unpack2(y01, y[4 * h], y[4 * h + 1]);
        unpack2(y23, y[4 * h + 2], y[4 * h + 3]);
    }
}

// Packed sign-magnitude nibbles of one level-2 unit from the biased quotients y of hif4_unit: element i in nibble i.
// The low byte of bits(y) is the signed code m (the magic constant's low byte is 0): the bytes are gathered and
// turned into sign-magnitude nibbles with byte-parallel arithmetic.
__device__ __forceinline__ uint32_t hif4_unit_nibbles(const float (&y)[8])
{
    uint32_t xw[2];                                               // per subgroup: nibbles n0 | n1 << 4 in byte 0, n2 | n3 << 4 in byte 2
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t b01 = __byte_perm(__float_as_uint(y[4 * h]), __float_as_uint(y[4 * h + 1]), 0x0040);
        const uint32_t b23 = __byte_perm(__float_as_uint(y[4 * h + 2]), __float_as_uint(y[4 * h + 3]), 0x0040);
        const uint32_t bb = __byte_perm(b01, b23, 0x5410);                     // m0, m1, m2, m3 as signed bytes
        const uint32_t sg = bb & 0x80808080u;                                  // sign bits
        const uint32_t ng = sg >> 7;                                           // 1 in every negative byte
        const uint32_t ab = (bb ^ (ng * 0xFFu)) + ng;                          // |m| per byte (no carry between bytes: |m| <= 7)
        const uint32_t nb = ab | (sg >> 4);                                    // sign to bit 3 of the byte
        xw[h] = nb | (nb >> 4);
    }
    return __byte_perm(xw[0], xw[1], 0x6420);
}
// The unit's share of the group's metadata word: level-2 bit at 8 + j, the two level-3 bits at 16 + 2 j (j = unit
// index in the group); the scale code (bits 0..7) is added once per group.
__device__ __forceinline__ uint32_t hif4_unit_meta(int j, int a, int k0, int k1)
{
    return ((uint32_t)a << (8 + j)) | ((uint32_t)((k0 - a) | ((k1 - a) << 1)) << (16 + 2 * j));
}

// One thread quantizes one whole 64-element group (Algorithm 1 lines 1 and 3) held in registers as 32 words of
// 16-bit pairs (element 2i in the low half of word i): the words are replaced by the BF16 image of
// HIF4(round_in(x * s)).  scale: the 64 Smooth-QK factors of these elements or null.  Same arithmetic as the 8-lane
// team of the stand-alone quantizer (hif4_group / hif4_unit), with the group constants formed once and no shuffles;
// the packed codes are not formed (the caller consumes the image at once).
template <typename T>
__device__ __forceinline__ void hif4_quantize64_regs(uint32_t (&xw)[32], const float* __restrict__ scale)
{
    float Ap[4] = {0.f, 0.f, 0.f, 0.f};                    // four independent maximum chains
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        float sv[8];
        if (scale) {
            const float4 s0 = __ldg(reinterpret_cast<const float4*>(scale) + 2 * c);
            const float4 s1 = __ldg(reinterpret_cast<const float4*>(scale) + 2 * c + 1);
            sv[0] = s0.x; sv[1] = s0.y; sv[2] = s0.z; sv[3] = s0.w;
            sv[4] = s1.x; sv[5] = s1.y; sv[6] = s1.z; sv[7] = s1.w;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float lo, hi;
            Pair16<T>::unpack(xw[4 * c + i], lo, hi);
            if (scale) {                                   // FP32 product, rounded once to the activation dtype
                float a, b;
                unpack2(mul2(pack2(lo, hi), pack2(sv[2 * i], sv[2 * i + 1])), a, b);
                xw[4 * c + i] = Pair16<T>::round_pack(a, b);
                Pair16<T>::unpack(xw[4 * c + i], lo, hi);
            }
            Ap[i] = max3(Ap[i], fabsf(lo), fabsf(hi));
        }
    }
    const float A = fmaxf(max3(Ap[0], Ap[1], Ap[2]), Ap[3]);
    const Hif4Group g = hif4_group(A);                     // A = 0: code 0 and an all-zero group
    const bool sat = A > g.top;                            // only above the E6M2 range
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        float x[8], y[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) Pair16<T>::unpack(xw[4 * u + i], x[2 * i], x[2 * i + 1]);
        if (sat) {
#pragma unroll
            for (int i = 0; i < 8; ++i) x[i] = fminf(fmaxf(x[i], -g.top), g.top);
        }
        const float a0 = fmaxf(max3(fabsf(x[0]), fabsf(x[1]), fabsf(x[2])), fabsf(x[3]));
        const float a1 = fmaxf(max3(fabsf(x[4]), fabsf(x[5]), fabsf(x[6])), fabsf(x[7]));
        uint32_t w[4];
        int a, k0, k1;
        hif4_unit(x, a0, a1, g, w, y, a, k0, k1);
#pragma unroll
        for (int i = 0; i < 4; ++i) xw[4 * u + i] = w[i];
    }
}

// The same for a group that sits in shared memory as a 128-byte row of a 64-column tile with the 128-byte swizzle
// TMA applies (`row_addr` the row's start, `sw` = row % 8 the swizzle key): quantized in place.
template <typename T>
__device__ __forceinline__ void hif4_quantize_row64_inplace(uint32_t row_addr, int sw, const float* __restrict__ scale)
{
    uint32_t xw[32];
#pragma unroll
    for (int c = 0; c < 8; ++c)
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(xw[4 * c]), "=r"(xw[4 * c + 1]), "=r"(xw[4 * c + 2]), "=r"(xw[4 * c + 3])
                     : "r"(row_addr + (uint32_t)((c ^ sw) << 4)));
    hif4_quantize64_regs<T>(xw, scale);
#pragma unroll
    for (int c = 0; c < 8; ++c)
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                     ::"r"(row_addr + (uint32_t)((c ^ sw) << 4)), "r"(xw[4 * c]), "r"(xw[4 * c + 1]), "r"(xw[4 * c + 2]),
                       "r"(xw[4 * c + 3]) : "memory");
}

}  // namespace hifa4
