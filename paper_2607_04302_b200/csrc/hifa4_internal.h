// Host-side declarations shared by the translation units of libhifa4.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "../../include/hifa4.h"

namespace hifa4 {

struct HeadMap;

void count_launch();

// mu_out: subtract the per-row mean (Q-Mean) and write it; ksum_out: write the per-row channel sum.
cudaError_t launch_quantize_rows(int dtype, const void* x, const float* scale, const HeadMap& map,
                                 int B, int H, int N, int d, uint8_t* codes, uint32_t* meta,
                                 void* img, float* mu_out, float* ksum_out, cudaStream_t st);
cudaError_t launch_quantize_tokens(int dtype, const void* x, int B, int H, int N, int d,
                                   uint8_t* codes, uint32_t* meta, void* img, cudaStream_t st);
cudaError_t launch_absmax(int dtype, const void* x, const HeadMap& map, int S, int H, int Hkv,
                          int Ncal, int d, float* ws, cudaStream_t st);
cudaError_t launch_smooth_finalize(const float* kmax, const float* qmax, int S, int n, double alpha,
                                   int bypass, float* s, float* inv_s, cudaStream_t st);

// Attention forward on the BF16 operand images; returns a hifa4_status.
int launch_attention(const hifa4_shape& shape, const HeadMap& map, const hifa4_qkv& qkv,
                     const hifa4_attn_params& prm, void* out, const hifa4_debug* dbg,
                     int* d_status, cudaStream_t st);

}  // namespace hifa4
