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
    float c0, c1;                 // sigma, sigma * log2(e)
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

// Quantize 64 softmax weights (already rounded to FP16, held as floats, all >= 0) to HIF4 and
// write the BF16 image of P-hat into shared memory as row `row` of a 128-byte-swizzled tile.
// Optionally dumps nibbles and subgroup steps.
__device__ __forceinline__ void quantize_p64(const float (&p)[64], uint32_t p_sub_base, int row,
                                             uint8_t* dump_codes, float* dump_step)
{
    float At[16];
    float A = 0.f;
#pragma unroll
    for (int t = 0; t < 16; ++t) {
        At[t] = fmaxf(fmaxf(p[4 * t], p[4 * t + 1]), fmaxf(p[4 * t + 2], p[4 * t + 3]));
        A = fmaxf(A, At[t]);
    }
    const uint32_t row_base = p_sub_base + (row >> 3) * 1024 + (row & 7) * 128;
    const int sw = row & 7;
    if (A == 0.f) {
#pragma unroll
        for (int ch = 0; ch < 8; ++ch)
            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(row_base + ((ch ^ sw) << 4)), "r"(0) : "memory");
        if (dump_codes) {
#pragma unroll
            for (int i = 0; i < 4; ++i) reinterpret_cast<uint4*>(dump_codes)[i] = make_uint4(0, 0, 0, 0);
        }
        if (dump_step) {
#pragma unroll
            for (int i = 0; i < 4; ++i) reinterpret_cast<float4*>(dump_step)[i] = make_float4(0, 0, 0, 0);
        }
        return;
    }
    const int code = e6m2_code_for_max(A);
    const float S = e6m2_value(code);
    const float inv4 = e6m2_inv4(code);
#pragma unroll
    for (int u = 0; u < 8; ++u) {                    // one level-2 unit = 8 keys = one 16-byte chunk
        int a, b0, b1;
        hif4_pair_bits(hif4_need(At[2 * u], S), hif4_need(At[2 * u + 1], S), a, b0, b1);
        uint32_t w[4];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int k = a + (h ? b1 : b0);
            const float inv_step = scale_pow2(inv4, -k);
            const float step = scale_pow2(S, k - 2);
            float v[4];
            uint32_t packed = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int m = __float2int_rn(__fmul_rz(p[8 * u + 4 * h + i], inv_step));
                v[i] = (float)m * step;
                packed |= (uint32_t)m << (8 * i);
            }
            __nv_bfloat162 lo = __floats2bfloat162_rn(v[0], v[1]);
            __nv_bfloat162 hi = __floats2bfloat162_rn(v[2], v[3]);
            w[2 * h] = *reinterpret_cast<uint32_t*>(&lo);
            w[2 * h + 1] = *reinterpret_cast<uint32_t*>(&hi);
            if (dump_step) dump_step[2 * u + h] = step;
            if (dump_codes) reinterpret_cast<uint32_t*>(dump_codes)[2 * u + h] = packed;
        }
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                     ::"r"(row_base + ((u ^ sw) << 4)), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
    }
}


// BF16 tensor [heads][rows][cols] (cols contiguous), box [1][box_rows][64 cols], 128-byte swizzle,
// out-of-range elements read as zero.  Returns false if the driver entry point is unavailable or
// the encode fails.
bool make_bf16_map(CUtensorMap* m, void* base, uint64_t heads, uint64_t rows, uint64_t cols, uint32_t box_rows);

// Warp-specialised kernel for d = 128, Bc = 128 (hifa4_attention_ws.cu).
int launch_attention_ws(const hifa4_shape& sh, const hifa4_qkv& qkv, const AttnArgs& args, cudaStream_t st);

}  // namespace hifa4
