// The kind::f8f6f4 experiment (the MMA kind the paper's "HIF4 Cube" comments of Algorithm 1 point at): Q K^T on
// 8-bit operands with one accumulator per 64-channel HIF4 group.  A HIF4 value is sign * m * 2^k * S/4 with
// m in 0..7 and k = level-2 + level-3 micro-exponent in 0..2; m * 2^k (an integer up to 28 with three significant
// bits) is exact in E4M3, the E6M2 scale is not, so it stays outside the MMA as one FP32 factor S/4 per group.
// This file: the operand images from the packed codes and metadata, and the entry point.  The attention kernel is
// the F8QK instantiation of the 64-key kernel.
#include "hifa4_attention.cuh"

namespace hifa4 {

// One thread per level-2 unit (8 elements): 4 bytes of codes -> 8 bytes of E4M3; the unit-0 thread of a group
// also writes the group scale.  rows = B * H * N, groups along d.
__global__ void __launch_bounds__(256)
f8_image_kernel(const uint8_t* __restrict__ codes, const uint32_t* __restrict__ meta, long long n_units, uint8_t* __restrict__ img,
                float* __restrict__ gs)
{
    const long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= n_units) return;
    const uint32_t mw = meta[u >> 3];
    const int j = (int)(u & 7);                              // unit inside the group
    const int a = (mw >> (8 + j)) & 1;
    const int k0 = a + ((mw >> (16 + 2 * j)) & 1), k1 = a + ((mw >> (17 + 2 * j)) & 1);
    const uint32_t nib = reinterpret_cast<const uint32_t*>(codes)[u];
    uint32_t w[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        uint32_t word = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t c = (nib >> (4 * (4 * h + i))) & 15u;
            const uint32_t v = (c & 7u) << (h ? k1 : k0);    // 0..28
            uint32_t b = 0;
            if (v) {
                const int e = 31 - __clz((int)v);            // v = 2^e * (1 + mant/8): E4M3 with bias 7
                b = ((uint32_t)(e + 7) << 3) | (((v << 3) >> e) & 7u) | ((c & 8u) << 4);
            }
            word |= b << (8 * i);
        }
        w[h] = word;
    }
    reinterpret_cast<uint2*>(img)[u] = make_uint2(w[0], w[1]);
    if (j == 0) {
        const float S = e6m2_value((int)(mw & 255u));
        gs[u >> 3] = __uint_as_float(__float_as_uint(S) - (2u << 23));   // S / 4
    }
}

cudaError_t launch_f8_images(const hifa4_shape& sh, const hifa4_qkv& qkv, void* q_f8, float* q_gs, void* k_f8, float* k_gs,
                             cudaStream_t st)
{
    const long long uq = (long long)sh.B * sh.Hq * sh.N * sh.d / 8, uk = (long long)sh.B * sh.Hkv * sh.N * sh.d / 8;
    if (q_f8) {
        f8_image_kernel<<<(unsigned)((uq + 255) / 256), 256, 0, st>>>(qkv.q_codes, qkv.q_meta, uq, (uint8_t*)q_f8, q_gs);
        count_launch();
    }
    if (k_f8) {
        f8_image_kernel<<<(unsigned)((uk + 255) / 256), 256, 0, st>>>(qkv.k_codes, qkv.k_meta, uk, (uint8_t*)k_f8, k_gs);
        count_launch();
    }
    return cudaGetLastError();
}

}  // namespace hifa4
