// Declarations shared by the attention kernels: launch arguments, the in-register HIF4 quantizer
// of P and the host-side TMA descriptor helper.
#pragma once
#include <cuda.h>

#include "hifa4_internal.h"
#include "hifa4_device.cuh"
#include "hifa4_ptx.cuh"

namespace hifa4 {

using namespace ptx;

struct DebugReq {
    int n_blocks;
    int blocks[HIFA4_MAX_DEBUG_BLOCKS * 3];
    uint8_t* p_codes;
    float* p_step;
    float* l_out;
    float* m_out;
};

struct AttnArgs {
    int B, Hq, Hkv, N;
    int causal, out_dtype;
    int group_heads;              // CTA order: groups of this many (batch, query head) pairs, one group after the other
    float c0, c1;                 // sigma, sigma * log2(e)
    int normalizer;               // 1: l accumulates the unquantized P (mismatched), not P-hat
    unsigned long long* hist;     // mass-error histogram [n_bins + 2] or null
    int n_bins;
    double hist_lo, hist_inv_w;   // bin = floor((eps - lo) * inv_w)
    int p_f32;                    // keep P in FP32 before quantization (variant; default FP16)
    int qmean;                    // add mu_i * k_sum_j to the raw scores (Algorithm 1 line 6)
    const float* q_mu;            // [B,Hq,N]
    const float* k_sum;           // [B,Hkv,N]
    // kind::f8f6f4 experiment (Q K^T on E4M3 images of element x micro-exponent, one accumulator per 64-channel group)
    const void *q_f8, *k_f8;      // [B,H,N,d] bytes, else null
    const float *q_gs, *k_gs;     // [B,H,N,d/64] group scales S/4
    const void* q_raw;            // raw-Q launch (Q is quantized inside the kernel): the 16-bit Q [B,Hq,N,d], else null
    const float* q_scale;         // raw-Q launch: Smooth-QK factors of Q [Hkv,d] or null
    int in_dtype;                 // raw-Q launch: HIFA4_F16 or HIFA4_BF16
    void* out;
    int* d_status;
    HeadMap map;
    DebugReq dbg;
};

template <int D, int BC>
struct Cfg {
    static constexpr int BR = 128;
    static constexpr int KSUB = D / 64;                    // 64-channel sub-tiles of Q and K
    static constexpr int PSUB = BC / 64;                   // 64-key chunks of P and V^T
    static constexpr int Q_SUB_BYTES = BR * 128;
    static constexpr int K_SUB_BYTES = BC * 128;
    static constexpr int V_CHUNK_BYTES = (D + 16) * 128;   // D rows of V^T + 16 rows of ones
    static constexpr int P_SUB_BYTES = BR * 128;
    static constexpr int Q_OFF = 0;
    static constexpr int K_OFF = Q_OFF + KSUB * Q_SUB_BYTES;
    static constexpr int V_OFF = K_OFF + KSUB * K_SUB_BYTES;
    static constexpr int P_OFF = V_OFF + PSUB * V_CHUNK_BYTES;
    static constexpr int BAR_OFF = P_OFF + PSUB * P_SUB_BYTES;
    static constexpr int SMEM_BYTES = BAR_OFF + 64 + 1024;  // + alignment slack
    static constexpr int O_COLS = D + 16;
    static constexpr int S_COL = (D == 64) ? 128 : (D == 128 ? 256 : 384);
    static constexpr int TMEM_COLS = (D == 64) ? 256 : 512;
    static_assert(S_COL + BC <= TMEM_COLS, "tensor memory budget");
};

__device__ __forceinline__ float f16_round(float x) { return __half2float(__float2half_rn(x)); }

// exp2 of two values, each result rounded to FP16 (one packed conversion) and widened back.
__device__ __forceinline__ void exp2_f16_pair(float t0, float t1, float& e0, float& e1)
{
    const float a = ex2_approx(t0), b = ex2_approx(t1);
    uint32_t h2;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(h2) : "f"(b), "f"(a));     // a -> low half, b -> high half
    asm("{\n\t.reg .b16 lo, hi;\n\t"
        "mov.b32 {lo, hi}, %2;\n\t"
        "cvt.f32.f16 %0, lo;\n\t"
        "cvt.f32.f16 %1, hi;\n\t}"
        : "=f"(e0), "=f"(e1) : "r"(h2));
}

// Quantize NU*8 consecutive softmax weights of one 64-key HIF4 group (already rounded to FP16,
// held as floats, all >= 0) and return the BF16 image of P-hat as NU*4 packed words (element 2i
// in the low half of word i).  A is the maximum of the whole group (the caller combines partial
// maxima when a group is split over threads) and At[t] the maxima of this thread's 4-key
// subgroups.  Optionally dumps nibbles and subgroup steps.
//
// Arithmetic (all exact): the element code is m = RNE(p / step).  q = RZ(p * (1/step)) lands
// exactly on j + 1/2 for every tie (see e6m2_inv4), y = q + 1.5 * 2^23 rounds q to the nearest
// integer with ties to even, and fma(y, step, -1.5 * 2^23 * step) = m * step without rounding.
// The shift of a 4-key subgroup with maximum At is read off the float bit patterns:
// n - 1 = max((bits(At) - bits(1.75 S) - 1) >> 23, -1); the pair rule "level-2 bit = 1 iff
// max(need) = 2 or min(need) >= 1" is a = (n0 + n1 + 2) >> 2 and the shifts are max(n, a).
template <int NU>
__device__ __forceinline__ void quantize_p_units(const float (&p)[NU * 8], const float (&At)[NU * 2], float A,
                                                 uint32_t (&w)[NU * 4], uint8_t* dump_codes, float* dump_step,
                                                 float* sum_out = nullptr)
{
    if (sum_out) *sum_out = 0.f;
    if (A == 0.f) {
#pragma unroll
        for (int i = 0; i < NU * 4; ++i) w[i] = 0u;
        if (dump_codes) {
#pragma unroll
            for (int i = 0; i < NU / 2; ++i) reinterpret_cast<uint4*>(dump_codes)[i] = make_uint4(0, 0, 0, 0);
        }
        if (dump_step) {
#pragma unroll
            for (int i = 0; i < NU / 2; ++i) reinterpret_cast<float4*>(dump_step)[i] = make_float4(0, 0, 0, 0);
        }
        return;
    }
    const int code = e6m2_code_for_max(A);
    const float S = e6m2_value(code);
    const uint32_t inv4_bits = __float_as_uint(e6m2_inv4(code));
    const uint32_t s4_bits = __float_as_uint(S) - (2u << 23);              // S / 4
    const int t1 = (int)__float_as_uint(1.75f * S) + 1;
    const float MAGIC = 12582912.f;                                        // 1.5 * 2^23
#pragma unroll
    for (int u = 0; u < NU; ++u) {                   // one level-2 unit = 8 keys
        const int n0 = max(((int)__float_as_uint(At[2 * u]) - t1) >> 23, -1);       // need - 1
        const int n1 = max(((int)__float_as_uint(At[2 * u + 1]) - t1) >> 23, -1);
        const int a = (n0 + n1 + 4) >> 2;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int k = max((h ? n1 : n0) + 1, a);
            const float inv_step = __uint_as_float(inv4_bits - ((uint32_t)k << 23));
            const float step = __uint_as_float(s4_bits + ((uint32_t)k << 23));
            const float negc = -MAGIC * step;
            float v[4];
            uint32_t packed = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float y = __fadd_rn(__fmul_rz(p[8 * u + 4 * h + i], inv_step), MAGIC);
                v[i] = fmaf(y, step, negc);
                if (sum_out) *sum_out += v[i];            // exact: every term is a multiple of S/4, the sum < 2^11 of them
                if (dump_codes) packed |= (__float_as_uint(y) & 15u) << (8 * i);
            }
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w[4 * u + 2 * h]) : "f"(v[1]), "f"(v[0]));
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w[4 * u + 2 * h + 1]) : "f"(v[3]), "f"(v[2]));
            if (dump_step) dump_step[2 * u + h] = step;
            if (dump_codes) reinterpret_cast<uint32_t*>(dump_codes)[2 * u + h] = packed;
        }
    }
}

// Fused form of Algorithm 1 lines 9-10 for NU*8 consecutive keys of one 64-key group: takes the raw
// score accumulators (masked ones already -inf), forms P = exp2(acc * c1 - mL) rounded to FP16 and
// quantizes it unit by unit, so that the exponentials (MUFU pipe) and the quantizer arithmetic
// (ALU/FMA pipes) of a warp interleave.  A is the group maximum of P, which the caller gets from
// the group maximum of the accumulators through the same instruction sequence
// (p_of_score): that is exact because fma, ex2.approx (checked exhaustively over [-40, 0]) and
// the FP16 rounding are all monotone non-decreasing.
template <bool PF32 = false>
__device__ __forceinline__ float p_of_score(float acc, float c1, float mL)
{
    const float e = ex2_approx(fmaf(acc, c1, -mL));
    return PF32 ? e : f16_round(e);                    // PF32: the variant that keeps P in FP32
}

// Arithmetic of the fused form (all exact except the exponential itself):
//   q = RZ(p * (4/S))            group-constant multiplier; exactly j + 1/2 (in units of the finest
//                                step S/4) on every rounding tie (see e6m2_inv4)
//   y = q + 1.5 * 2^(23+k)       rounds q to the nearest multiple of 2^k, ties to the even multiple:
//                                y - magic = m * 2^k with m the element code under shift k
//   v = fma(y, S/4, -magic*S/4)  = m * 2^k * S/4, the dequantized value, no rounding
// The shift k of a 4-key subgroup with maximum At is read off float bit patterns:
//   need = max(bits(At) - bits(1.75 S) - 1 + 2^23, 0) >> 23   (0, 1 or 2)
// (the shifts of the two subgroups of a level-2 unit are then combined by exp_quantize_units).
// Multiplications, additions and FMAs run two elements at a time (f32x2).
struct PQuantConst {              // per (row, 64-key group, tile) constants of the fused quantizer
    uint64_t c1c1, nml, inv44, s44;
    uint32_t c0_bits, s4_bits;
    int tadd;
};

// Constants from the group maximum A of P.  A = 0 (every key masked) needs no branch: the scale
// code clamps to 0, every p is 0 and every product below is an exact zero.
__device__ __forceinline__ PQuantConst p_quant_const(float c1, float mL, float A)
{
    PQuantConst k;
    const int code = e6m2_code_for_max(A);
    const float S = e6m2_value(code);
    const float inv4 = e6m2_inv4(code);
    const float S4 = __uint_as_float(__float_as_uint(S) - (2u << 23));     // S / 4
    k.tadd = (1 << 23) - ((int)__float_as_uint(1.75f * S) + 1);
    k.c0_bits = __float_as_uint(-12582912.f * S4);                         // -1.5 * 2^23 * S/4
    k.s4_bits = __float_as_uint(S4);
    k.c1c1 = pack2(c1, c1);
    k.nml = pack2(-mL, -mL);
    k.inv44 = pack2(inv4, inv4);
    k.s44 = pack2(S4, S4);
    return k;
}

// P = exp2(acc * c1 - mL) rounded to FP16 (PF32: left in FP32) for the 8 keys of unit u.
template <int NU, bool PF32 = false>
__device__ __forceinline__ void exp_unit(const float (&acc)[NU * 8], int u, const PQuantConst& k, float (&p)[8])
{
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
        float t0, t1;
        unpack2(fma2(pack2(acc[8 * u + i], acc[8 * u + i + 1]), k.c1c1, k.nml), t0, t1);
        if (PF32) { p[i] = ex2_approx(t0); p[i + 1] = ex2_approx(t1); }
        else exp2_f16_pair(t0, t1, p[i], p[i + 1]);
    }
}

// Units U0..U1-1 of a thread's NU units: acc -> P (FP16) -> P-hat image words w[4u..4u+3].
// The exponentials of unit u+1 are issued before unit u is quantized, so that the MUFU latency of
// one unit hides behind the ALU/FMA work of the previous one.
// A unit is two 4-key subgroups t = 0, 1 with shifts k_t = max(need_t, need_other - 1) (that is the
// pair rule: the level-2 bit is set iff max(need) = 2 or min(need) >= 1, and a subgroup that needs no
// shift of its own still gets one when its partner needs two).  On bit patterns, with
// x_t = max(bits(At_t) + tadd, 0) = need_t * 2^23 + fraction: k_t * 2^23 = max(x_t, x_other - 2^23)
// with the fraction masked off.  The packed operations pair key i of subgroup 0 with key i of
// subgroup 1, so that one pair of per-subgroup constants (magic, c) serves four packed operations.
template <int NU, int U0, int U1, bool DBG, bool PF32 = false>
__device__ __forceinline__ void exp_quantize_units(const float (&acc)[NU * 8], const PQuantConst& k, bool zero_group,
                                                   uint32_t (&w)[NU * 4], uint8_t* dump_codes, float* dump_step)
{
    const int MAGIC_BITS = 0x4B400000;                                    // 1.5 * 2^23
    float pn[8];
    exp_unit<NU, PF32>(acc, U0, k, pn);
#pragma unroll
    for (int u = U0; u < U1; ++u) {
        float p[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) p[i] = pn[i];
        if (u + 1 < U1) exp_unit<NU, PF32>(acc, u + 1, k, pn);
        const float At0 = fmaxf(max3(p[0], p[1], p[2]), p[3]);
        const float At1 = fmaxf(max3(p[4], p[5], p[6]), p[7]);
        const int x0 = max((int)__float_as_uint(At0) + k.tadd, 0);
        const int x1 = max((int)__float_as_uint(At1) + k.tadd, 0);
        const int ks0 = max(x0, x1 - (1 << 23)) & (int)0xFF800000;
        const int ks1 = max(x1, x0 - (1 << 23)) & (int)0xFF800000;
        const uint64_t mm = pack2(__int_as_float(MAGIC_BITS + ks0), __int_as_float(MAGIC_BITS + ks1));
        const uint64_t cc = pack2(__int_as_float((int)k.c0_bits + ks0), __int_as_float((int)k.c0_bits + ks1));
        float v[8];
        uint64_t y[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            y[i] = add2(mul2_rz(pack2(p[i], p[4 + i]), k.inv44), mm);
            unpack2(fma2(y[i], k.s44, cc), v[i], v[4 + i]);
        }
        // BF16 image: every value has at most 8 significant bits, so the upper halves of the FP32 patterns
        // are the BF16 values (a byte permute instead of a conversion)
#pragma unroll
        for (int i = 0; i < 4; ++i) w[4 * u + i] = __byte_perm(__float_as_uint(v[2 * i]), __float_as_uint(v[2 * i + 1]), 0x7632);
        if (DBG) {
            float c[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) unpack2(y[i], c[i], c[4 + i]);
            if (dump_step) {
                dump_step[2 * u] = zero_group ? 0.f : __int_as_float((int)k.s4_bits + ks0);
                dump_step[2 * u + 1] = zero_group ? 0.f : __int_as_float((int)k.s4_bits + ks1);
            }
            if (dump_codes) {
#pragma unroll
                for (int h = 0; h < 2; ++h)
                    reinterpret_cast<uint32_t*>(dump_codes)[2 * u + h] =
                        (__float_as_uint(c[4 * h]) & 15u) | ((__float_as_uint(c[4 * h + 1]) & 15u) << 8) |
                        ((__float_as_uint(c[4 * h + 2]) & 15u) << 16) | ((__float_as_uint(c[4 * h + 3]) & 15u) << 24);
            }
        }
    }
}

// Whole 64-key group held by one thread; the image goes to row `row` of a 128-byte-swizzled
// shared-memory tile (the layout a K-major tcgen05 operand descriptor with SWIZZLE_128B reads).
__device__ __forceinline__ void quantize_p64(const float (&p)[64], uint32_t p_sub_base, int row,
                                             uint8_t* dump_codes, float* dump_step, float* sum_out = nullptr)
{
    float At[16];
#pragma unroll
    for (int t = 0; t < 16; ++t) At[t] = fmaxf(max3(p[4 * t], p[4 * t + 1], p[4 * t + 2]), p[4 * t + 3]);
    float A4[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) A4[t] = fmaxf(max3(At[4 * t], At[4 * t + 1], At[4 * t + 2]), At[4 * t + 3]);
    const float A = fmaxf(max3(A4[0], A4[1], A4[2]), A4[3]);
    uint32_t w[32];
    quantize_p_units<8>(p, At, A, w, dump_codes, dump_step, sum_out);
    const uint32_t row_base = p_sub_base + (row >> 3) * 1024 + (row & 7) * 128;
    const int sw = row & 7;
#pragma unroll
    for (int u = 0; u < 8; ++u)
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                     ::"r"(row_base + ((u ^ sw) << 4)), "r"(w[4 * u]), "r"(w[4 * u + 1]), "r"(w[4 * u + 2]), "r"(w[4 * u + 3]) : "memory");
}

// BF16 tensor [heads][rows][cols] (cols contiguous), box [1][box_rows][64 cols], 128-byte swizzle,
// out-of-range elements read as zero.  Returns false if the driver entry point is unavailable or
// the encode fails.
bool make_bf16_map(CUtensorMap* m, void* base, uint64_t heads, uint64_t rows, uint64_t cols, uint32_t box_rows);

// Warp-specialised kernel for d = 128, Bc = 128 (hifa4_attention_ws.cu).
int launch_attention_ws(const hifa4_shape& sh, const hifa4_qkv& qkv, const AttnArgs& args, cudaStream_t st);

// Warp-specialised kernels for Bc = 64, d = 64, 128 or 256 (hifa4_attention_ws64.cu).
int launch_attention_ws64(const hifa4_shape& sh, const hifa4_qkv& qkv, const AttnArgs& args, cudaStream_t st);
// Self-test instantiation (d = 128): one bounded wait is made to run out (see hifa4_selftest_wait_timeout).
int launch_attention_ws64_selftest(const hifa4_shape& sh, const hifa4_qkv& qkv, const AttnArgs& args, cudaStream_t st);

}  // namespace hifa4
