// Adaptive applicability gate on the GPU ("Adaptive Applicability Gate"): the two statistics
//   rho_K = max|K| / P99(|K|)   (nearest-rank percentile over every element of the calibration K)
//   T_K/Q = max|K| / max|Q|
// and the branch they select (Strong / Mild / Bypass), computed without leaving the device, then the
// Smooth-QK factors for that branch.
//
// |x| of a 16-bit float is a 15-bit pattern whose integer order is the order of the values, so a
// 32768-bin histogram of the patterns is the exact distribution of |K| and the percentile is read off
// its running sum: no sort, no sampling.
#include "hifa4_internal.h"
#include "hifa4_device.cuh"

namespace hifa4 {

constexpr int HIST_BINS = 32768;
constexpr int HIST_THREADS = 512;
constexpr int GATE_THREADS = 1024;

// Every CTA histograms a strided share of x in shared memory (128 KB of counters) and adds its
// non-empty bins to the global histogram.  n_vec = number of 8-element vectors.
__global__ void __launch_bounds__(HIST_THREADS)
abs_hist_kernel(const uint4* __restrict__ x, long long n_vec, uint32_t* __restrict__ hist)
{
    extern __shared__ uint32_t h[];
    for (int i = threadIdx.x; i < HIST_BINS; i += HIST_THREADS) h[i] = 0;
    __syncthreads();
    for (long long v = (long long)blockIdx.x * HIST_THREADS + threadIdx.x; v < n_vec;
         v += (long long)gridDim.x * HIST_THREADS) {
        const uint4 raw = __ldg(x + v);
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            atomicAdd(&h[w[i] & 0x7FFFu], 1u);
            atomicAdd(&h[(w[i] >> 16) & 0x7FFFu], 1u);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < HIST_BINS; i += HIST_THREADS)
        if (h[i]) atomicAdd(&hist[i], h[i]);
}

// One CTA: global maxima from the per-(sample, head, channel) maxima, the percentile from the
// histogram, the gate decision.  gate[0] = alpha, gate[1] = 1 if bypass (doubles, read by the
// finalize kernel); stats[0..3] = rho_K, T_K/Q, branch (0 bypass, 1 strong, 2 mild), alpha (floats).
template <typename T>
__global__ void __launch_bounds__(GATE_THREADS)
gate_kernel(const float* __restrict__ kmax, const float* __restrict__ qmax, int n_max,
            const uint32_t* __restrict__ hist, unsigned long long rank, double* __restrict__ gate,
            float* __restrict__ stats)
{
    __shared__ float s_k[GATE_THREADS / 32], s_q[GATE_THREADS / 32];
    __shared__ unsigned long long s_cnt[GATE_THREADS];
    __shared__ uint32_t s_p99;
    const int tid = threadIdx.x;
    float mk = 0.f, mq = 0.f;
    for (int i = tid; i < n_max; i += GATE_THREADS) {
        mk = fmaxf(mk, kmax[i]);
        mq = fmaxf(mq, qmax[i]);
    }
    for (int o = 16; o; o >>= 1) {
        mk = fmaxf(mk, __shfl_xor_sync(0xffffffffu, mk, o));
        mq = fmaxf(mq, __shfl_xor_sync(0xffffffffu, mq, o));
    }
    if ((tid & 31) == 0) { s_k[tid >> 5] = mk; s_q[tid >> 5] = mq; }
    // running sum of the histogram: thread t owns bins 32t .. 32t+31
    constexpr int PER = HIST_BINS / GATE_THREADS;
    unsigned long long local = 0;
    for (int i = 0; i < PER; ++i) local += hist[tid * PER + i];
    s_cnt[tid] = local;
    if (tid == 0) s_p99 = 0;
    __syncthreads();
    for (int o = 1; o < GATE_THREADS; o <<= 1) {          // inclusive scan (Hillis-Steele)
        unsigned long long add = tid >= o ? s_cnt[tid - o] : 0;
        __syncthreads();
        s_cnt[tid] += add;
        __syncthreads();
    }
    const unsigned long long before = s_cnt[tid] - local;
    if (before < rank && rank <= s_cnt[tid]) {            // exactly one thread: the rank falls in its bins
        unsigned long long c = before;
        for (int i = 0; i < PER; ++i) {
            c += hist[tid * PER + i];
            if (c >= rank) { s_p99 = (uint32_t)(tid * PER + i); break; }
        }
    }
    __syncthreads();
    if (tid == 0) {
        for (int i = 0; i < GATE_THREADS / 32; ++i) { mk = fmaxf(mk, s_k[i]); mq = fmaxf(mq, s_q[i]); }
        const double p99 = (double)In16<T>::to_f((uint16_t)s_p99);
        const double rho = p99 > 0.0 ? (double)mk / p99 : 0.0;
        const double t = mq > 0.f ? (double)mk / (double)mq : 0.0;
        const int branch = (rho >= 6.0 && t >= 2.0) ? (t > 3.0 ? 1 : 2) : 0;
        const double alpha = branch == 1 ? 0.5 : branch == 2 ? 0.25 : 0.0;
        gate[0] = alpha;
        gate[1] = branch == 0 ? 1.0 : 0.0;
        if (stats) {
            stats[0] = (float)rho;
            stats[1] = (float)t;
            stats[2] = (float)branch;
            stats[3] = (float)alpha;
        }
    }
}

cudaError_t launch_gate(int dtype, const void* k_cal, long long nk, const float* kmax, const float* qmax,
                        int n_max, void* gate_ws, float* d_stats, cudaStream_t st)
{
    uint32_t* hist = reinterpret_cast<uint32_t*>(gate_ws);
    double* gate = reinterpret_cast<double*>(reinterpret_cast<char*>(gate_ws) + HIST_BINS * sizeof(uint32_t));
    cudaError_t e = cudaMemsetAsync(hist, 0, HIST_BINS * sizeof(uint32_t), st);
    if (e != cudaSuccess) return e;
    static SmemOptIn opt_in;
    if (!opt_in.ensure(abs_hist_kernel, (int)(HIST_BINS * sizeof(uint32_t)))) return cudaErrorInvalidValue;
    const long long n_vec = nk / 8;
    int sms = 148;
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long want = (n_vec + HIST_THREADS - 1) / HIST_THREADS;
    const unsigned blocks = (unsigned)(want < sms ? (want > 0 ? want : 1) : sms);
    abs_hist_kernel<<<blocks, HIST_THREADS, HIST_BINS * sizeof(uint32_t), st>>>(
        reinterpret_cast<const uint4*>(k_cal), n_vec, hist);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    unsigned long long rank = (unsigned long long)ceil(0.99 * (double)nk);   // nearest-rank percentile
    if (rank < 1) rank = 1;
    if (dtype == HIFA4_F16)
        gate_kernel<__half><<<1, GATE_THREADS, 0, st>>>(kmax, qmax, n_max, hist, rank, gate, d_stats);
    else
        gate_kernel<__nv_bfloat16><<<1, GATE_THREADS, 0, st>>>(kmax, qmax, n_max, hist, rank, gate, d_stats);
    count_launch();
    return cudaGetLastError();
}

const double* gate_result(void* gate_ws)
{
    return reinterpret_cast<const double*>(reinterpret_cast<char*>(gate_ws) + HIST_BINS * sizeof(uint32_t));
}

}  // namespace hifa4
