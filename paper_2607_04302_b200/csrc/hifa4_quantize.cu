// Smooth-QK scaling fused with HIF4 quantization (Algorithm 1 lines 1 and 3) and the
// calibration reduction behind the Smooth-QK factors (Eq. "sqk").  Q, K and V are quantized by one
// launch: 128-bit coalesced loads, one 8-lane team per 64-element group, shuffle reductions,
// packed f32x2 arithmetic.
#include "hifa4_internal.h"
#include "hifa4_device.cuh"
#include "hifa4_ptx.cuh"

namespace hifa4 {

using namespace ptx;

// One lane owns 8 consecutive elements of a 64-element group = one level-2 unit = two
// level-3 subgroups; the 8 lanes of a team (aligned inside a warp) own the group.
// x[8]: values already smoothed and rounded to the input dtype.  Returns the packed nibbles; w gets
// the BF16 image of the dequantized values (element 2i in the low half of word i); meta_word the
// group's metadata (every lane of the team gets the same word).
// The arithmetic is hif4_group / hif4_unit (exact; the same scheme as the in-register quantizer of P).
__device__ __forceinline__ uint32_t quantize8(float (&x)[8], int j, uint32_t (&w)[4], uint32_t& meta_word)
{
    float a0 = fmaxf(max3(fabsf(x[0]), fabsf(x[1]), fabsf(x[2])), fabsf(x[3]));
    float a1 = fmaxf(max3(fabsf(x[4]), fabsf(x[5]), fabsf(x[6])), fabsf(x[7]));
    float A = fmaxf(a0, a1);
    A = fmaxf(A, __shfl_xor_sync(0xffffffffu, A, 1));
    A = fmaxf(A, __shfl_xor_sync(0xffffffffu, A, 2));
    A = fmaxf(A, __shfl_xor_sync(0xffffffffu, A, 4));
    const Hif4Group g = hif4_group(A);                            // A = 0 gives code 0 and an all-zero group
    if (A > g.top) {                                              // only above the E6M2 range: saturate
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = fminf(fmaxf(x[i], -g.top), g.top);
        a0 = fminf(a0, g.top);
        a1 = fminf(a1, g.top);
    }
    float y[8];
    int a, k0, k1;
    hif4_unit(x, a0, a1, g, w, y, a, k0, k1);
    uint32_t part = hif4_unit_meta(j, a, k0, k1);
    if (j == 0) part |= (uint32_t)g.code;
    const uint32_t nib = hif4_unit_nibbles(y);
    part |= __shfl_xor_sync(0xffffffffu, part, 1);
    part |= __shfl_xor_sync(0xffffffffu, part, 2);
    part |= __shfl_xor_sync(0xffffffffu, part, 4);
    meta_word = part;
    return nib;
}

struct QuantJob {                     // one launch quantizes Q, K and V (any of them may be absent)
    const uint16_t *q, *k, *v;        // [B,Hq,N,d], [B,Hkv,N,d], [B,Hkv,N,d]
    const float *s, *inv_s;           // [Hkv,d] Smooth-QK factors for Q and K, or null
    uint8_t *q_codes, *k_codes, *v_codes;
    uint32_t *q_meta, *k_meta, *v_meta;
    uint16_t *q_img, *k_img, *v_img;
    float *q_mu, *k_sum;              // Q-Mean auxiliary outputs or null
    int Hq, Hkv, N, d;
    unsigned q_blocks, k_blocks;      // CTAs [0, q_blocks) take Q, the next k_blocks K, the rest V
    unsigned row_blocks_per_head;     // N * d / 8 / (256 * UPT)
    HeadMap qmap;
};

constexpr int QUANT_THREADS = 256;
// Row units per thread (template parameter UPT): 4 where a head holds a multiple of 1024 units, which
// keeps 64 bytes of loads in flight per thread (the kernel is latency-bound below that), else 2.

// Q and K: groups along d.  One head is N*d/8 units of 8 channels; a CTA takes 256 * UPT consecutive
// units, thread t the units t, t + 256, ... (all loads are issued before any arithmetic).  The two
// units share their channel offset, hence their Smooth-QK factors.
template <typename T, int UPT>
__device__ __forceinline__ void quantize_rows_cta(const uint16_t* __restrict__ x, const float* __restrict__ scale,
                                                  int kv_row, long long head, unsigned blk_in_head, int N, int d,
                                                  uint8_t* __restrict__ codes, uint32_t* __restrict__ meta,
                                                  uint16_t* __restrict__ img, float* __restrict__ mu_out,
                                                  float* __restrict__ ksum_out)
{
    const int upr = d >> 3;                                                   // units per row
    const unsigned u0 = blk_in_head * (QUANT_THREADS * UPT) + threadIdx.x;    // unit inside the head
    const long long base = head * (long long)N * upr;                         // first unit of the head
    const int c0 = (int)(u0 & (unsigned)(upr - 1)) << 3;
    uint4 raw[UPT];
#pragma unroll
    for (int r = 0; r < UPT; ++r)
        raw[r] = __ldg(reinterpret_cast<const uint4*>(x) + base + u0 + r * QUANT_THREADS);
    float sv[8];
    if (scale) {
        const float4* sp = reinterpret_cast<const float4*>(scale + (long long)kv_row * d + c0);
        const float4 s0 = __ldg(sp), s1 = __ldg(sp + 1);
        sv[0] = s0.x; sv[1] = s0.y; sv[2] = s0.z; sv[3] = s0.w;
        sv[4] = s1.x; sv[5] = s1.y; sv[6] = s1.z; sv[7] = s1.w;
    }
#pragma unroll
    for (int r = 0; r < UPT; ++r) {
        const unsigned u = u0 + r * QUANT_THREADS;
        const long long t = base + u;
        const uint32_t rw[4] = {raw[r].x, raw[r].y, raw[r].z, raw[r].w};
        float v[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) Pair16<T>::unpack(rw[i], v[2 * i], v[2 * i + 1]);
        if (scale) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float a, b;
                unpack2(mul2(pack2(v[2 * i], v[2 * i + 1]), pack2(sv[2 * i], sv[2 * i + 1])), a, b);
                Pair16<T>::unpack(Pair16<T>::round_pack(a, b), v[2 * i], v[2 * i + 1]);
            }
        }
        if (mu_out || ksum_out) {
            // Q-Mean auxiliary (Algorithm 1 lines 2 and 6).  A row of d channels sits in d/8 consecutive,
            // aligned lanes; the sum runs in double, where it is exact for any row whose values span fewer
            // than ~40 binades, so its order does not matter.
            const long long row = head * N + (u >> (31 - __clz(upr)));
            double sum = 0.0;
#pragma unroll
            for (int i = 0; i < 8; ++i) sum += (double)v[i];
            for (int off = 1; off < upr; off <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
            if (mu_out) {                                // q_z = round_in(q~ - mu), mu = FP16(mean)
                const float mu = __half2float(__double2half(sum / (double)d));
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] = In16<T>::round_d((double)v[i] - (double)mu);
                if (c0 == 0) mu_out[row] = mu;
            } else if (c0 == 0) {
                ksum_out[row] = __half2float(__double2half(sum));
            }
        }
        uint32_t w[4], mw;
        const uint32_t nib = quantize8(v, threadIdx.x & 7, w, mw);
        reinterpret_cast<uint32_t*>(codes)[t] = nib;
        reinterpret_cast<uint4*>(img)[t] = make_uint4(w[0], w[1], w[2], w[3]);
        if ((threadIdx.x & 7) == 0) meta[t >> 3] = mw;
    }
}

// V: groups of 64 tokens per channel; outputs are stored transposed ([.., d, N]).  One CTA
// transposes a 64-token x 64-channel tile through shared memory.  The tile is kept as 64 rows of
// 8 16-byte chunks, chunk c of row r stored at position c ^ (r >> 3), so that both the row-wise
// 16-byte stores and the column-wise 4-byte reads (a thread reads two adjacent channels of 8
// consecutive tokens) are free of bank conflicts.  256 threads = 32 channel pairs x 8 lanes.
template <typename T>
__device__ __forceinline__ void quantize_tokens_cta(const uint16_t* __restrict__ x, long long bh, int tok0, int ch0,
                                                    int N, int d, uint8_t* __restrict__ codes,
                                                    uint32_t* __restrict__ meta, uint16_t* __restrict__ img)
{
    __shared__ uint4 tile[64 * 8];
    const uint16_t* src = x + (bh * N + tok0) * (long long)d + ch0;
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        const int idx = threadIdx.x + it * QUANT_THREADS;
        const int r = idx >> 3, c8 = idx & 7;
        tile[r * 8 + (c8 ^ (r >> 3))] = __ldg(reinterpret_cast<const uint4*>(src + (long long)r * d) + c8);
    }
    __syncthreads();
    const int cp = threadIdx.x >> 3, j = threadIdx.x & 7;          // channel pair, level-2 unit
    const uint32_t* tw = reinterpret_cast<const uint32_t*>(tile);
    float va[8], vb[8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
        Pair16<T>::unpack(tw[(8 * j + i) * 32 + ((((cp >> 2) ^ j) << 2) | (cp & 3))], va[i], vb[i]);
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        uint32_t w[4], mw;
        const uint32_t nib = quantize8(c ? vb : va, j, w, mw);
        const long long orow = bh * d + ch0 + 2 * cp + c;             // row of the transposed outputs
        reinterpret_cast<uint32_t*>(codes + orow * (N / 2) + tok0 / 2)[j] = nib;
        reinterpret_cast<uint4*>(img + orow * (long long)N + tok0)[j] = make_uint4(w[0], w[1], w[2], w[3]);
        if (j == 0) meta[orow * (N / 64) + tok0 / 64] = mw;
    }
}

template <typename T, int UPT>
__global__ void __launch_bounds__(QUANT_THREADS)
quantize_qkv_kernel(const __grid_constant__ QuantJob job)
{
    // a dependent grid launched with programmatic stream serialization (the attention kernel) may start
    // becoming resident as this grid's CTAs retire; it waits for this grid's completion before it reads
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    unsigned blk = blockIdx.x;
    if (blk < job.q_blocks + job.k_blocks) {
        const bool is_q = blk < job.q_blocks;
        if (!is_q) blk -= job.q_blocks;
        const unsigned head = blk / job.row_blocks_per_head;             // b * H + h
        const unsigned in_head = blk - head * job.row_blocks_per_head;
        if (is_q)
            quantize_rows_cta<T, UPT>(job.q, job.s, job.qmap.kv_of[head % (unsigned)job.Hq], head, in_head, job.N, job.d,
                                 job.q_codes, job.q_meta, job.q_img, job.q_mu, nullptr);
        else
            quantize_rows_cta<T, UPT>(job.k, job.inv_s, (int)(head % (unsigned)job.Hkv), head, in_head, job.N, job.d,
                                 job.k_codes, job.k_meta, job.k_img, nullptr, job.k_sum);
    } else {
        blk -= job.q_blocks + job.k_blocks;
        const unsigned tok_blocks = job.N / 64, ch_blocks = job.d / 64;
        const unsigned tb = blk % tok_blocks, rest = blk / tok_blocks;
        const unsigned cb = rest % ch_blocks, bh = rest / ch_blocks;
        quantize_tokens_cta<T>(job.v, bh, tb * 64, cb * 64, job.N, job.d, job.v_codes, job.v_meta, job.v_img);
    }
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

// s = Kagg^alpha / Qagg^(1-alpha); 1 where degenerate.  The per-sample maxima are combined over the S samples
// by root-mean-square (aggregator 0, the paper's choice), mean (1) or nearest-rank 99th percentile (2).
// gate (optional, device): {alpha, bypass flag} chosen by the applicability gate; overrides the arguments.
__device__ __forceinline__ double percentile99(const float* __restrict__ v, int S, long long stride)
{
    const long long rank = (long long)ceil(0.99 * (double)S) < 1 ? 1 : (long long)ceil(0.99 * (double)S);
    for (int a = 0; a < S; ++a) {                            // selection by counting: S is small
        const float va = v[a * stride];
        long long below = 0, not_above = 0;
        for (int b = 0; b < S; ++b) { const float vb = v[b * stride]; below += vb < va; not_above += vb <= va; }
        if (below < rank && rank <= not_above) return (double)va;
    }
    return 0.0;
}
__global__ void smooth_finalize_kernel(const float* __restrict__ kmax, const float* __restrict__ qmax,
                                       int S, int n, double alpha, int bypass, int aggregator,
                                       const double* __restrict__ gate, float* __restrict__ s, float* __restrict__ inv_s)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    if (gate) { alpha = gate[0]; bypass = gate[1] != 0.0; }
    double kagg, qagg;
    if (aggregator == 2) {
        kagg = percentile99(kmax + i, S, n);
        qagg = percentile99(qmax + i, S, n);
    } else {
        double ks = 0, qs = 0;
        for (int m = 0; m < S; ++m) {
            double a = kmax[(long long)m * n + i], b = qmax[(long long)m * n + i];
            ks += aggregator == 1 ? a : a * a;
            qs += aggregator == 1 ? b : b * b;
        }
        kagg = aggregator == 1 ? ks / S : sqrt(ks / S);
        qagg = aggregator == 1 ? qs / S : sqrt(qs / S);
    }
    double sv = 1.0;
    if (!bypass && kagg > 0 && qagg > 0) sv = pow(kagg, alpha) / pow(qagg, 1.0 - alpha);
    float sf = (float)sv;
    s[i] = sf;
    inv_s[i] = __frcp_rn(sf);
}

// ------------------------------------------------------------------------------- launchers
cudaError_t launch_quantize_qkv(int dtype, const hifa4_shape& sh, const HeadMap& qmap, const void* q,
                                const void* k, const void* v, const float* s, const float* inv_s,
                                const hifa4_qkv& out, cudaStream_t st)
{
    QuantJob job{};
    job.q = (const uint16_t*)q; job.k = (const uint16_t*)k; job.v = (const uint16_t*)v;
    job.s = s; job.inv_s = inv_s;
    job.q_codes = out.q_codes; job.k_codes = out.k_codes; job.v_codes = out.v_codes;
    job.q_meta = out.q_meta; job.k_meta = out.k_meta; job.v_meta = out.v_meta;
    job.q_img = (uint16_t*)out.q_mma; job.k_img = (uint16_t*)out.k_mma; job.v_img = (uint16_t*)out.v_mma;
    job.q_mu = out.q_mu; job.k_sum = out.k_sum;
    job.Hq = sh.Hq; job.Hkv = sh.Hkv; job.N = sh.N; job.d = sh.d;
    const long long head_units = (long long)sh.N * sh.d / 8;
    const int upt = head_units % (QUANT_THREADS * 4) == 0 ? 4 : 2;
    job.row_blocks_per_head = (unsigned)(head_units / (QUANT_THREADS * upt));
    job.q_blocks = q ? (unsigned)sh.B * sh.Hq * job.row_blocks_per_head : 0u;
    job.k_blocks = k ? (unsigned)sh.B * sh.Hkv * job.row_blocks_per_head : 0u;
    const unsigned v_blocks = v ? (unsigned)sh.B * sh.Hkv * (sh.N / 64) * (sh.d / 64) : 0u;
    job.qmap = qmap;
    const unsigned long long total = (unsigned long long)job.q_blocks + job.k_blocks + v_blocks;
    if (total == 0) return cudaSuccess;
    if (total > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
    if (dtype == HIFA4_F16) {
        if (upt == 4) quantize_qkv_kernel<__half, 4><<<(unsigned)total, QUANT_THREADS, 0, st>>>(job);
        else quantize_qkv_kernel<__half, 2><<<(unsigned)total, QUANT_THREADS, 0, st>>>(job);
    } else {
        if (upt == 4) quantize_qkv_kernel<__nv_bfloat16, 4><<<(unsigned)total, QUANT_THREADS, 0, st>>>(job);
        else quantize_qkv_kernel<__nv_bfloat16, 2><<<(unsigned)total, QUANT_THREADS, 0, st>>>(job);
    }
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
                                   int bypass, int aggregator, const double* gate, float* s, float* inv_s,
                                   cudaStream_t st)
{
    smooth_finalize_kernel<<<(n + 127) / 128, 128, 0, st>>>(kmax, qmax, S, n, alpha, bypass, aggregator, gate, s, inv_s);
    count_launch();
    return cudaGetLastError();
}

}  // namespace hifa4
