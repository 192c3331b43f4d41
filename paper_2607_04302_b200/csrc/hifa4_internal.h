// Host-side declarations shared by the translation units of libhifa4.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <mutex>
#include "../../include/hifa4.h"

namespace hifa4 {

struct HeadMap;

void count_launch();

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) holds for one device only: each launcher keeps one of
// these per kernel instantiation and opts in once per device, under a lock (host threads may race).
struct SmemOptIn {
    static constexpr int MAX_DEVICES = 64;
    std::mutex m;
    bool done[MAX_DEVICES] = {};
    template <class Kernel>
    bool ensure(Kernel kern, int bytes)
    {
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return false;
        std::lock_guard<std::mutex> lock(m);
        if (!done[dev]) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
            done[dev] = true;
        }
        return true;
    }
};

// One launch for Q, K and V (null inputs are skipped).  out.q_mu / out.k_sum non-null: Q-Mean
// (subtract the per-row mean of Q and write it; write the per-row channel sum of K).
cudaError_t launch_quantize_qkv(int dtype, const hifa4_shape& sh, const HeadMap& qmap, const void* q,
                                const void* k, const void* v, const float* s, const float* inv_s,
                                const hifa4_qkv& out, cudaStream_t st);
cudaError_t launch_absmax(int dtype, const void* x, const HeadMap& map, int S, int H, int Hkv,
                          int Ncal, int d, float* ws, cudaStream_t st);
// gate: null, or the device {alpha, bypass} pair written by launch_gate (overrides alpha / bypass).
// aggregator: 0 root-mean-square, 1 mean, 2 nearest-rank 99th percentile of the per-sample maxima.
cudaError_t launch_smooth_finalize(const float* kmax, const float* qmax, int S, int n, double alpha,
                                   int bypass, int aggregator, const double* gate, float* s, float* inv_s,
                                   cudaStream_t st);
// Gate statistics and decision on the device.  gate_ws: HIFA4_GATE_WS_BYTES bytes; d_stats: 4 floats or null.
cudaError_t launch_gate(int dtype, const void* k_cal, long long nk, const float* kmax, const float* qmax,
                        int n_max, void* gate_ws, float* d_stats, cudaStream_t st);
const double* gate_result(void* gate_ws);

// Attention forward on the BF16 operand images; returns a hifa4_status.
// q_raw non-null: Q is the raw 16-bit tensor (qkv.q_mma is not read) and is smoothed with q_scale (or not, if null)
// and quantized inside the kernel; see attention_qraw_supported.
// Operands of the kind::f8f6f4 experiment: E4M3 images of element x micro-exponent and the per-group scales S/4.
struct F8Operands {
    const void *q_f8, *k_f8;      // [B,H,N,d] bytes
    const float *q_gs, *k_gs;     // [B,H,N,d/64]
};
// From the packed codes and metadata of Q and K (either may be null).
cudaError_t launch_f8_images(const hifa4_shape& sh, const hifa4_qkv& qkv, void* q_f8, float* q_gs, void* k_f8, float* k_gs,
                             cudaStream_t st);
int launch_attention(const hifa4_shape& shape, const HeadMap& map, const hifa4_qkv& qkv,
                     const hifa4_attn_params& prm, void* out, const hifa4_debug* dbg,
                     const hifa4_mass_stats* stats, int* d_status, cudaStream_t st, bool selftest = false,
                     const void* q_raw = nullptr, const float* q_scale = nullptr, const F8Operands* f8 = nullptr);
// Configurations whose attention kernel can quantize Q itself: the 64-key kernel for d = 128 (256 softmax threads =
// 128 rows x two 64-channel groups) in its default arithmetic or the FP32-P variant, without Q-Mean (the row mean
// needs the whole row before any group is quantized).
bool attention_qraw_supported(const hifa4_shape& shape, const hifa4_attn_params& prm);

}  // namespace hifa4
