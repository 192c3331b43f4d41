// Smooth-QK scaling fused with HIF4 quantization (Algorithm 1 lines 1 and 3) and the
// calibration reduction behind the Smooth-QK factors (Eq. "sqk").  HBM-bound kernels:
// 128-bit coalesced loads, one 8-lane team per 64-element group, shuffle reductions.
#include "hifa4_internal.h"
#include "hifa4_device.cuh"

namespace hifa4 {

// One lane owns 8 consecutive elements of a 64-element group = one level-2 unit = two
// level-3 subgroups; the 8 lanes of a team (aligned inside a warp) own the group.
// x[8]: values already smoothed and rounded to the input dtype.
// Returns the packed nibbles; img gets the dequantized values; meta_part gets this lane's
// OR-contribution (the team leader's includes the scale code).
__device__ __forceinline__ uint32_t quantize8(const float (&x)[8], int j, float (&img)[8],
                                              uint32_t& meta_word)
{
    float a0 = fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3])));
    float a1 = fmaxf(fmaxf(fabsf(x[4]), fabsf(x[5])), fmaxf(fabsf(x[6]), fabsf(x[7])));
    float A = fmaxf(a0, a1);
    A = fmaxf(A, __shfl_xor_sync(0xffffffffu, A, 1));
    A = fmaxf(A, __shfl_xor_sync(0xffffffffu, A, 2));
    A = fmaxf(A, __shfl_xor_sync(0xffffffffu, A, 4));
    uint32_t nib = 0, part = 0;
    if (A > 0.f) {
        int code = e6m2_code_for_max(A);
        float S = e6m2_value(code);
        float inv4 = e6m2_inv4(code);
        int a, b0, b1;
        hif4_pair_bits(hif4_need(a0, S), hif4_need(a1, S), a, b0, b1);
        part = ((uint32_t)a << (8 + j)) | ((uint32_t)(b0 | (b1 << 1)) << (16 + 2 * j));
        if (j == 0) part |= (uint32_t)code;
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            int k = a + (w ? b1 : b0);
            float inv_step = scale_pow2(inv4, -k);
            float step = scale_pow2(S, k - 2);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float v = x[4 * w + i];
                int m = hif4_code(fabsf(v), inv_step);
                float dq = (float)m * step;
                img[4 * w + i] = v < 0.f ? -dq : dq;
                nib |= (uint32_t)(m | ((v < 0.f && m > 0) ? 8 : 0)) << (4 * (4 * w + i));
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) img[i] = 0.f;
    }
    part |= __shfl_xor_sync(0xffffffffu, part, 1);
    part |= __shfl_xor_sync(0xffffffffu, part, 2);
    part |= __shfl_xor_sync(0xffffffffu, part, 4);
    meta_word = part;
    return nib;
}

__device__ __forceinline__ uint4 pack_bf16x8(const float (&v)[8])
{
    uint4 o;
    __nv_bfloat162 t;
    t = __floats2bfloat162_rn(v[0], v[1]); o.x = *reinterpret_cast<uint32_t*>(&t);
    t = __floats2bfloat162_rn(v[2], v[3]); o.y = *reinterpret_cast<uint32_t*>(&t);
    t = __floats2bfloat162_rn(v[4], v[5]); o.z = *reinterpret_cast<uint32_t*>(&t);
    t = __floats2bfloat162_rn(v[6], v[7]); o.w = *reinterpret_cast<uint32_t*>(&t);
    return o;
}

// Q and K: groups along d.  x [rows_total, d] with rows_total = B*H*N.  Thread t owns
// elements [8t, 8t+8).  scale (optional) is [Hkv, d]; head h reads row map.kv_of[h].
template <typename T>
__global__ void __launch_bounds__(256)
quantize_rows_kernel(const uint16_t* __restrict__ x, const float* __restrict__ scale, HeadMap map,
                     int H, int N, int d, long long n_units, uint8_t* __restrict__ codes,
                     uint32_t* __restrict__ meta, uint16_t* __restrict__ img,
                     float* __restrict__ mu_out, float* __restrict__ ksum_out)
{
    long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_units) return;                        // n_units % 32 == 0: whole warps leave together
    long long e0 = t * 8;
    long long row = e0 / d;
    int c0 = (int)(e0 - row * d);
    uint4 raw = __ldg(reinterpret_cast<const uint4*>(x) + t);
    const uint16_t* r16 = reinterpret_cast<const uint16_t*>(&raw);
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = In16<T>::to_f(r16[i]);
    if (scale) {
        int h = (int)((row / N) % H);
        const float4* sp = reinterpret_cast<const float4*>(scale + (long long)map.kv_of[h] * d + c0);
        float4 s0 = __ldg(sp), s1 = __ldg(sp + 1);
        const float sv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = In16<T>::round(v[i] * sv[i]);
    }
    if (mu_out || ksum_out) {
        // Q-Mean auxiliary (Algorithm 1 lines 2 and 6).  A row of d channels sits in d/8 consecutive,
        // aligned lanes; the sum runs in double, where it is exact for any row whose values span fewer
        // than ~40 binades, so its order does not matter.
        double sum = 0.0;
#pragma unroll
        for (int i = 0; i < 8; ++i) sum += (double)v[i];
        for (int off = 1; off < d / 8; off <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
        if (mu_out) {                                // q_z = round_in(q~ - mu), mu = FP16(mean)
            const float mu = __half2float(__double2half(sum / (double)d));
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = In16<T>::round_d((double)v[i] - (double)mu);
            if (c0 == 0) mu_out[row] = mu;
        } else if (c0 == 0) {
            ksum_out[row] = __half2float(__double2half(sum));
        }
    }
    float dq[8];
    uint32_t mw;
    uint32_t nib = quantize8(v, threadIdx.x & 7, dq, mw);
    reinterpret_cast<uint32_t*>(codes)[t] = nib;
    reinterpret_cast<uint4*>(img)[t] = pack_bf16x8(dq);
    if ((threadIdx.x & 7) == 0) meta[t >> 3] = mw;
}

// V: groups of 64 tokens per channel; outputs are stored transposed ([.., d, N]).
// One CTA transposes a 64-token x 64-channel tile through shared memory; 512 threads =
// 64 channels x 8 lanes.
template <typename T>
__global__ void __launch_bounds__(512)
quantize_tokens_kernel(const uint16_t* __restrict__ x, int N, int d, uint8_t* __restrict__ codes,
                       uint32_t* __restrict__ meta, uint16_t* __restrict__ img)
{
    __shared__ uint16_t tile[64][72];                // +8 pad: 144-byte rows keep 16-byte alignment
    const int tok0 = blockIdx.x * 64, ch0 = blockIdx.y * 64;
    const long long bh = blockIdx.z;
    const uint16_t* src = x + (bh * N + tok0) * (long long)d + ch0;
    {
        int r = threadIdx.x >> 3, c8 = threadIdx.x & 7;          // 64 rows x 8 chunks of 16 bytes
        uint4 raw = __ldg(reinterpret_cast<const uint4*>(src + (long long)r * d) + c8);
        *reinterpret_cast<uint4*>(&tile[r][c8 * 8]) = raw;
    }
    __syncthreads();
    const int c = threadIdx.x >> 3, j = threadIdx.x & 7;          // channel, level-2 unit
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = In16<T>::to_f(tile[8 * j + i][c]);
    float dq[8];
    uint32_t mw;
    uint32_t nib = quantize8(v, j, dq, mw);
    const long long orow = bh * d + ch0 + c;                      // row of the transposed outputs
    reinterpret_cast<uint32_t*>(codes + orow * (N / 2) + tok0 / 2)[j] = nib;
    reinterpret_cast<uint4*>(img + orow * (long long)N + tok0)[j] = pack_bf16x8(dq);
    if (j == 0) meta[orow * (N / 64) + tok0 / 64] = mw;
}

// Calibration: per (sample, kv head, channel) maximum magnitude over tokens (and over the query
// heads of the group).  Non-negative floats order like their bit patterns, so atomicMax on the
// uint view is exact.  ws [S, Hkv, d] is cleared by the caller.
template <typename T>
__global__ void __launch_bounds__(256)
absmax_kernel(const uint16_t* __restrict__ x, HeadMap map, int H, int Hkv, int Ncal, int d,
              int tokens_per_block, uint32_t* __restrict__ ws)
{
    const int sh = blockIdx.x;                       // sample * H + head
    const int smp = sh / H, h = sh % H;
    const int g = map.kv_of[h];
    const int chunks = d / 8;
    const int c8 = threadIdx.x % chunks, tl = threadIdx.x / chunks, tstep = blockDim.x / chunks;
    const int t0 = blockIdx.y * tokens_per_block;
    const int t1 = min(t0 + tokens_per_block, Ncal);
    float mx[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (tl < tstep) {
        for (int t = t0 + tl; t < t1; t += tstep) {
            uint4 raw = __ldg(reinterpret_cast<const uint4*>(x + ((long long)sh * Ncal + t) * d) + c8);
            const uint16_t* r16 = reinterpret_cast<const uint16_t*>(&raw);
#pragma unroll
            for (int i = 0; i < 8; ++i) mx[i] = fmaxf(mx[i], fabsf(In16<T>::to_f(r16[i])));
        }
#pragma unroll
        for (int i = 0; i < 8; ++i)
            atomicMax(ws + ((long long)smp * Hkv + g) * d + c8 * 8 + i, __float_as_uint(mx[i]));
    }
}

// s = Kagg^alpha / Qagg^(1-alpha) with RMS aggregation over samples; 1 where degenerate.
__global__ void smooth_finalize_kernel(const float* __restrict__ kmax, const float* __restrict__ qmax,
                                       int S, int n, double alpha, int bypass, float* __restrict__ s,
                                       float* __restrict__ inv_s)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    double ks = 0, qs = 0;
    for (int m = 0; m < S; ++m) {
        double a = kmax[(long long)m * n + i], b = qmax[(long long)m * n + i];
        ks += a * a;
        qs += b * b;
    }
    double kagg = sqrt(ks / S), qagg = sqrt(qs / S);
    double sv = 1.0;
    if (!bypass && kagg > 0 && qagg > 0) sv = pow(kagg, alpha) / pow(qagg, 1.0 - alpha);
    float sf = (float)sv;
    s[i] = sf;
    inv_s[i] = __frcp_rn(sf);
}

// ------------------------------------------------------------------------------- launchers
template <typename T>
static cudaError_t launch_rows(const void* x, const float* scale, const HeadMap& map, int B, int H,
                               int N, int d, uint8_t* codes, uint32_t* meta, void* img, float* mu_out,
                               float* ksum_out, cudaStream_t st)
{
    long long units = (long long)B * H * N * d / 8;
    unsigned blocks = (unsigned)((units + 255) / 256);
    quantize_rows_kernel<T><<<blocks, 256, 0, st>>>((const uint16_t*)x, scale, map, H, N, d, units,
                                                    codes, meta, (uint16_t*)img, mu_out, ksum_out);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_quantize_rows(int dtype, const void* x, const float* scale, const HeadMap& map,
                                 int B, int H, int N, int d, uint8_t* codes, uint32_t* meta,
                                 void* img, float* mu_out, float* ksum_out, cudaStream_t st)
{
    return dtype == HIFA4_F16
               ? launch_rows<__half>(x, scale, map, B, H, N, d, codes, meta, img, mu_out, ksum_out, st)
               : launch_rows<__nv_bfloat16>(x, scale, map, B, H, N, d, codes, meta, img, mu_out, ksum_out, st);
}

cudaError_t launch_quantize_tokens(int dtype, const void* x, int B, int H, int N, int d,
                                   uint8_t* codes, uint32_t* meta, void* img, cudaStream_t st)
{
    dim3 grid(N / 64, d / 64, B * H);
    if (dtype == HIFA4_F16)
        quantize_tokens_kernel<__half><<<grid, 512, 0, st>>>((const uint16_t*)x, N, d, codes, meta, (uint16_t*)img);
    else
        quantize_tokens_kernel<__nv_bfloat16><<<grid, 512, 0, st>>>((const uint16_t*)x, N, d, codes, meta, (uint16_t*)img);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_absmax(int dtype, const void* x, const HeadMap& map, int S, int H, int Hkv,
                          int Ncal, int d, float* ws, cudaStream_t st)
{
    const int tpb = 256;
    dim3 grid(S * H, (Ncal + tpb - 1) / tpb);
    if (dtype == HIFA4_F16)
        absmax_kernel<__half><<<grid, 256, 0, st>>>((const uint16_t*)x, map, H, Hkv, Ncal, d, tpb, (uint32_t*)ws);
    else
        absmax_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const uint16_t*)x, map, H, Hkv, Ncal, d, tpb, (uint32_t*)ws);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_smooth_finalize(const float* kmax, const float* qmax, int S, int n, double alpha,
                                   int bypass, float* s, float* inv_s, cudaStream_t st)
{
    smooth_finalize_kernel<<<(n + 127) / 128, 128, 0, st>>>(kmax, qmax, S, n, alpha, bypass, s, inv_s);
    count_launch();
    return cudaGetLastError();
}

}  // namespace hifa4
