/*
 * hifa4.h -- C ABI of the HiFA4 hot path for NVIDIA B200 (sm_100a).
 *
 * HiFA4 (arxiv 2607.04302) runs both attention GEMMs, Q K^T and P V, on HIF4
 * 4-bit block-floating-point values, keeps the online-softmax state in FP16,
 * rescales post-RoPE Q and K per channel by calibration-static Smooth-QK
 * factors, and takes the softmax normalizer from the quantized P-hat that
 * feeds the PV GEMM (P-Reordering), produced in the same tensor-core pass by a
 * column of ones appended to V (Algorithm 1 "C4V16-Aux").
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller unless a
 *     parameter says "host".  The library allocates no device memory, frees
 *     none and never synchronizes; work is enqueued on `stream`
 *     (a cudaStream_t passed as void*; NULL is the default stream).
 *   - Tensors are contiguous, row-major, in the index order given.
 *   - Return value: a hifa4_status.  No exception crosses this boundary and
 *     there is no CPU fallback: on a device that is not sm_100 every compute
 *     call returns HIFA4_ERR_ARCH.
 *   - `d_status` (optional, may be NULL) is a device int the kernels write a
 *     non-zero hifa4_status into when a bounded wait inside a kernel expires;
 *     the caller zeroes it and reads it after synchronizing.
 */
#ifndef HIFA4_H
#define HIFA4_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    HIFA4_OK = 0,
    HIFA4_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, bad enum          */
    HIFA4_ERR_UNSUPPORTED = 2,   /* shape / flag combination not built                 */
    HIFA4_ERR_WORKSPACE = 3,     /* workspace missing or too small                     */
    HIFA4_ERR_ARCH = 4,          /* current device is not compute capability 10.x      */
    HIFA4_ERR_CUDA = 5,          /* a CUDA runtime/driver call failed                  */
    HIFA4_ERR_TIMEOUT = 6        /* a bounded device-side wait expired (see d_status)  */
} hifa4_status;

typedef enum { HIFA4_F16 = 0, HIFA4_BF16 = 1, HIFA4_F32 = 2 } hifa4_dtype;

enum { HIFA4_Q = 0, HIFA4_K = 1, HIFA4_V = 2 };               /* `which` */
enum { HIFA4_PART_CODES = 0, HIFA4_PART_META = 1, HIFA4_PART_MMA = 2, HIFA4_PART_AUX = 3 }; /* `part` */
enum { HIFA4_MAX_HEADS = 256, HIFA4_MAX_DEBUG_BLOCKS = 16 };
enum { HIFA4_AGG_RMS = 0, HIFA4_AGG_MEAN = 0x100, HIFA4_AGG_P99 = 0x200 };   /* OR-ed into calibration `mode` */
#define HIFA4_STATIC_CALIB_MAX_FLOATS (1u << 20)   /* scratch limit of hifa4_smooth_calibrate_static */

/* Problem shape.  Q is [B,Hq,N,d]; K and V are [B,Hkv,N,d] ("GQA and batch
 * handling", Appendix "Implementation Details").  d in {64,128,256};
 * N a multiple of 64; Hq, Hkv <= HIFA4_MAX_HEADS.  q_to_kv is a HOST array of
 * Hq KV-head indices, or NULL for the usual grouping h / (Hq/Hkv) (then Hq
 * must be a multiple of Hkv).  in_dtype is HIFA4_F16 or HIFA4_BF16. */
typedef struct {
    int B, Hq, Hkv, N, d;
    const int* q_to_kv;
    int in_dtype;
} hifa4_shape;

/* Quantized Q/K/V (Algorithm 1 line 3).  Nine device buffers the caller
 * allocates with the sizes hifa4_quant_bytes() returns.
 *   *_codes : HIF4 element nibbles, two per byte, even element in the low
 *             nibble; nibble = sign<<3 | m, magnitude m/4 (S1P2).
 *   *_meta  : one uint32 per 64-element group: byte 0 the E6M2 level-1 scale
 *             code (S = 2^(e-48) (1+M/4), e = code>>2, M = code&3), byte 1
 *             the 8 level-2 bits (bit u covers elements 8u..8u+7), bytes 2-3
 *             the 16 level-3 bits (bit t covers elements 4t..4t+3).
 *             value_i = +-S * 2^(l2+l3) * m_i / 4      (Background, "HIF4").
 *   *_mma   : the same values, dequantized exactly to BF16 (every HIF4 value
 *             has at most 6 significant bits), in the layout the attention
 *             kernel's TMA loads expect.
 * Groups run along each GEMM's contraction axis: along d for Q and K
 * (codes [B,H,N,d/2], meta [B,H,N,d/64], mma [B,H,N,d]); along tokens for V
 * (codes [B,Hkv,d,N/2], meta [B,Hkv,d,N/64], mma [B,Hkv,d,N], i.e. V is
 * stored transposed).
 * Q-Mean auxiliary (Algorithm 1 lines 2 and 6; "Auxiliary Q-Mean Compensation"): when q_mu and
 * k_sum are both non-NULL, hifa4_quantize_qkv subtracts from every smoothed query token its mean
 * over the d channels before quantizing (the Q buffers then hold Q_z) and writes
 *   q_mu  [B,Hq,N]  floats: the per-token mean mu_i, an FP16 value;
 *   k_sum [B,Hkv,N] floats: sum over channels of the smoothed key, an FP16 value;
 * hifa4_attention_fwd with prm->qmean = 1 adds mu_i * k_sum_j to the raw score accumulators.
 * Leave both NULL for the path without Q-Mean.  (hifa4_quant_bytes: part HIFA4_PART_AUX.) */
typedef struct {
    uint8_t* q_codes; uint32_t* q_meta; void* q_mma;
    uint8_t* k_codes; uint32_t* k_meta; void* k_mma;
    uint8_t* v_codes; uint32_t* v_meta; void* v_mma;
    float* q_mu; float* k_sum;
} hifa4_qkv;

/* Calibration result summary (host memory).  rho_K and T_KQ are the gate
 * statistics of "Adaptive Applicability Gate"; this struct reports them as NaN
 * (hifa4_smooth_calibrate_auto computes them, into device memory).  branch: 0 bypass, 1 strong, 2 mild, 4 caller's alpha. */
typedef struct { float rho_K, T_KQ; int branch; float alpha; } hifa4_calib_stats;

/* Attention parameters.
 *   causal      1: key j contributes to row i only if j <= i.
 *   Br          query rows per CTA; scheduling only, must be 128.
 *   Bc          key-tile width of the online softmax (64 or 128).  It is part
 *               of the result: P is quantized under the running maximum that
 *               holds after each Bc keys (Algorithm 1 lines 7-10).
 *   normalizer  0: consistent (P-Reordering, normalizer = rowsum of P-hat via
 *               the ones column); 1: mismatched, the normalizer is accumulated
 *               from the unquantized FP16 P while PV consumes P-hat (the
 *               "Direct" baseline of "P-Reordering"; Theorem 1's O_mis).  Mode 1
 *               is an ablation: it runs on a one-thread-per-row kernel, several
 *               times slower than mode 0.
 *   qmean       1: add the Q-Mean correction mu_i * k_sum_j to the raw scores (line 6; scaled by the
 *               softmax scale together with them); needs qkv->q_mu and qkv->k_sum filled by
 *               hifa4_quantize_qkv.  0: no correction (the Q buffers must then hold un-centred Q).
 *   p_dtype     HIFA4_F16: exp(S-m) is rounded to FP16 before quantization
 *               ("FP16 operations", Appendix "Implementation Details").
 *               HIFA4_F32: variant that quantizes the FP32 exponential directly (a
 *               different function: it changes a few 1e-4 of the P-hat codes); built
 *               for Bc = 64 with d = 128 or 256 and the consistent normalizer,
 *               HIFA4_ERR_UNSUPPORTED elsewhere.
 *   out_dtype   HIFA4_F16 / HIFA4_BF16 / HIFA4_F32 element type of `out`.
 *   softmax_scale  0 selects 1/sqrt(d). */
typedef struct {
    int causal, Br, Bc;
    int normalizer, qmean, p_dtype, out_dtype;
    float softmax_scale;
} hifa4_attn_params;

/* Optional debug dump of P-hat for up to HIFA4_MAX_DEBUG_BLOCKS 128-row query
 * blocks.  blocks: HOST array of n_blocks triples (b, h, query_block_index).
 * p_codes: device [n_blocks][128][N] bytes, the nibble of every P-hat element
 * (0 where the key tile was skipped by causality); p_step: device
 * [n_blocks][128][N/4] floats, the step of every 4-key subgroup (0 for an all-zero group); l_out, m_out:
 * device [n_blocks][128] floats, the accumulated normalizer and the final
 * running maximum.  Any of the four device pointers may be NULL. */
typedef struct {
    int n_blocks;
    const int* blocks;
    uint8_t* p_codes;
    float* p_step;
    float* l_out;
    float* m_out;
} hifa4_debug;

/* Histogram of the per-tile mass error of P-hat ("P-Reordering", Theorem 1 and the
 * figure of its empirical validation): for every query row and every Bc-key tile whose
 * P is not all zero, eps = sum_j P-hat_j / sum_j P_j - 1 over the keys of the tile, both
 * sums exact.  hist: device array of n_bins + 2 counters that the call ADDS to (clear it
 * first): bin k counts lo + k*w <= eps < lo + (k+1)*w with w = (hi - lo)/n_bins; entry
 * n_bins counts eps < lo, entry n_bins + 1 counts eps >= hi. */
typedef struct {
    unsigned long long* hist;
    int n_bins;
    double lo, hi;
} hifa4_mass_stats;

const char* hifa4_status_string(int status);

/* Self-test of the failure path of the device-side waits (no counterpart in the paper; for deployment
 * checks and for the test-suite).  Launches the Bc = 64, d = 128 attention kernel in an instantiation
 * whose softmax warps withhold the arrival that releases the P V product and whose issuer gives up
 * waiting for it after 2^12 polls (a fraction of a millisecond) instead of 2^20.  When that wait runs out
 * every TMA load has landed and no MMA is in flight; the kernel records HIFA4_ERR_TIMEOUT + 16 * 7 (site 7:
 * the issuer's wait for P V) in *d_status (required, device int, zero on entry), raises the CTA's abort flag,
 * every role leaves through the common exit that frees tensor memory, and the call returns normally.
 * `out` is not written.  Arguments as hifa4_attention_fwd (prm: Bc = 64, no variant flags; shape: d = 128);
 * a one-CTA problem (N <= 128, one head) is what the test-suite uses.  Nothing hangs, faults or traps. */
int hifa4_selftest_wait_timeout(const hifa4_shape* shape, const hifa4_qkv* qkv, const hifa4_attn_params* prm,
                                void* out, int* d_status, void* stream);

/* Calls made so far in this process: out[0] calibrate, out[1] quantize,
 * out[2] attention, out[3] kernels launched (all entry points). */
void hifa4_get_counters(unsigned long long out[4]);

/* Offline Smooth-QK calibration (Eq. "sqk"; "Calibration-Static Deployment").
 *   q_cal [S,Hq,Ncal,d], k_cal [S,Hkv,Ncal,d]: post-RoPE calibration
 *   activations of one layer, S samples of Ncal tokens, element type dt.
 *   Per sample and channel the statistic is the largest magnitude over tokens
 *   (for Q also over the query heads sharing the KV head); samples are
 *   combined by root-mean-square; s = Kagg^alpha / Qagg^(1-alpha), 1 where an
 *   aggregate is zero.  mode: 0 bypass (s = 1), 1 strong (alpha 0.5), 2 mild
 *   (alpha 0.25), 4 caller's alpha; 3 (gate decides) returns
 *   HIFA4_ERR_UNSUPPORTED here: use hifa4_smooth_calibrate_auto, which takes
 *   the extra scratch the gate statistics need.  OR-ing HIFA4_AGG_MEAN or
 *   HIFA4_AGG_P99 into mode replaces the root-mean-square over samples by the
 *   mean or by the nearest-rank 99th percentile of the per-sample maxima (the
 *   two alternatives of the paper's aggregator comparison, table "calib").
 *   Outputs (device): s, inv_s [Hkv,d] floats, inv_s = fl32(1/s).
 *   absmax_ws: device scratch of 2*S*Hkv*d floats; the call clears it.
 *   host_stats: optional HOST struct, filled without synchronizing. */
int hifa4_smooth_calibrate(const void* q_cal, const void* k_cal, int S, int Hq, int Hkv,
                           int Ncal, int d, const int* q_to_kv, int dt, int mode, float alpha,
                           float* s, float* inv_s, float* absmax_ws,
                           hifa4_calib_stats* host_stats, void* stream);

/* Calibration with the applicability gate deciding the branch ("Adaptive Applicability
 * Gate"), entirely on the device:
 *   rho_K = max|K| / P99(|K|), the 99th percentile (nearest rank) over every element of
 *   k_cal, read off an exact histogram of the 15-bit magnitude patterns;
 *   T = max|K| / max|Q| over every element of k_cal and q_cal;
 *   rho_K >= 6 and T >= 2 select Smooth-QK, with alpha = 0.5 (strong) if T > 3 and
 *   alpha = 0.25 (mild) if 2 <= T <= 3; anything else bypasses (s = 1).
 * Arguments as hifa4_smooth_calibrate, plus
 *   gate_ws : device scratch of HIFA4_GATE_WS_BYTES bytes, 8-byte aligned;
 *   d_stats : NULL, or DEVICE array of 4 floats that receives rho_K, T, the branch
 *             (0 bypass, 1 strong, 2 mild) and alpha.  The call does not synchronize: copy
 *             the four floats back after the stream has run if the host wants them.
 * S*Hkv*Ncal*d must be below 2^32 (HIFA4_ERR_UNSUPPORTED otherwise). */
#define HIFA4_GATE_WS_BYTES (32768u * 4u + 64u)
int hifa4_smooth_calibrate_auto(const void* q_cal, const void* k_cal, int S, int Hq, int Hkv,
                                int Ncal, int d, const int* q_to_kv, int dt, float* s,
                                float* inv_s, float* absmax_ws, void* gate_ws, float* d_stats,
                                void* stream);

/* hifa4_smooth_calibrate for callers that cannot allocate device memory.
 * (The paper has no counterpart: this entry point exists for deployment only.)
 *   Who needs it: code that runs where cudaMalloc is off limits -- a serving process whose whole
 *   device memory already belongs to an arena it may not grow, a plug-in called from a runtime
 *   that forbids allocation on its worker threads, a latency-critical section that cannot take
 *   the device-wide synchronization an allocation implies.  Such a caller still owns its inputs
 *   and outputs (q_cal, k_cal, s, inv_s) but has nowhere to get the 2*S*Hkv*d-float scratch from.
 *   What it does: the same computation, with the same kernels, as hifa4_smooth_calibrate; the
 *   scratch is a fixed array of HIFA4_STATIC_CALIB_MAX_FLOATS floats (4 MiB) in device global
 *   memory, which every GPU that loads this library holds until the process exits.  The call
 *   makes no cudaMalloc/cudaFree and uses no allocating library routine.
 *   Limits and rules:
 *   - 2*S*Hkv*d must not exceed HIFA4_STATIC_CALIB_MAX_FLOATS, else HIFA4_ERR_WORKSPACE is
 *     returned and nothing is enqueued (use hifa4_smooth_calibrate with your own workspace).
 *   - The first call on each device looks up the device address of the array (with that device
 *     current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents; each
 *     call clears the part it uses before reducing into it.  Two calls whose kernels may overlap
 *     on the GPU (different streams, no ordering between them) race on it: serialize them.
 *   Arguments and results otherwise as hifa4_smooth_calibrate, minus absmax_ws. */
int hifa4_smooth_calibrate_static(const void* q_cal, const void* k_cal, int S, int Hq, int Hkv,
                                  int Ncal, int d, const int* q_to_kv, int dt, int mode,
                                  float alpha, float* s, float* inv_s,
                                  hifa4_calib_stats* host_stats, void* stream);

/* Bytes of one buffer of hifa4_qkv for this shape; 0 on a bad argument. */
size_t hifa4_quant_bytes(const hifa4_shape* shape, int which, int part);

/* Smooth-QK scaling fused with HIF4 quantization (Algorithm 1 lines 1 and 3).
 *   q~ = round_in(q * s[kv(h)]), k~ = round_in(k * inv_s[g]) with an fp32
 *   multiply rounded to the input dtype; V is quantized as it is.
 *   s, inv_s: [Hkv,d] floats, or both NULL for bypass.  Any of q, k, v may be
 *   NULL to skip that tensor.  Fills the buffers of `out`. */
int hifa4_quantize_qkv(const hifa4_shape* shape, const void* q, const void* k, const void* v,
                       const float* s, const float* inv_s, const hifa4_qkv* out,
                       int* d_status, void* stream);

/* Workspace the attention call needs (may be 0). */
size_t hifa4_attention_workspace_bytes(const hifa4_shape* shape, const hifa4_attn_params* prm);

/* Fused prefill attention forward on quantized operands (Algorithm 1 lines
 * 4-13): S = Q-hat K-hat^T / sqrt(d); FP16 running max and rescale;
 * P = exp(S - m) in FP16; P-hat = HIF4(P) per row and 64 keys;
 * [O | l] += P-hat [V-hat | 1]; out = O / l.
 *   qkv: buffers filled by hifa4_quantize_qkv for the same shape (only the
 *   *_mma images are read).  out: [B,Hq,N,d] of prm->out_dtype.
 *   workspace: at least hifa4_attention_workspace_bytes() bytes (NULL if 0).
 *   dbg: NULL, or a P-hat dump request.
 * Scheduling note: for Bc = 64 the grid is launched with programmatic stream
 * serialization, i.e. its CTAs may become resident while the preceding kernel
 * of the stream is still draining; they read and write no global memory before
 * that kernel has completed, so the usual stream order of results holds. */
int hifa4_attention_fwd(const hifa4_shape* shape, const hifa4_qkv* qkv,
                        const hifa4_attn_params* prm, void* out, void* workspace,
                        const hifa4_debug* dbg, int* d_status, void* stream);

/* hifa4_attention_fwd that also fills the mass-error histogram of P-hat (see
 * hifa4_mass_stats; "P-Reordering", Theorem 1).  Same arguments and result as
 * hifa4_attention_fwd (either normalizer mode); stats must be non-NULL with
 * n_bins >= 1 and lo < hi.  Analysis path: it runs on the one-thread-per-row kernel. */
int hifa4_attention_fwd_stats(const hifa4_shape* shape, const hifa4_qkv* qkv,
                              const hifa4_attn_params* prm, void* out, void* workspace,
                              const hifa4_mass_stats* stats, int* d_status, void* stream);

/* hifa4_attention_fwd with Algorithm 1 line 1 inside the attention kernel: q is
 * the raw post-RoPE Q [B,Hq,N,d] of shape->in_dtype (device), s the Smooth-QK
 * factors of Q [Hkv,d] (device) or NULL; every CTA smooths and HIF4-quantizes
 * its own 128 query rows in shared memory, so Q-hat is never written to device
 * memory (its codes are not produced).  kv: buffers filled by
 * hifa4_quantize_qkv(shape, NULL, k, v, ...) for the same shape (only k_mma
 * and v_mma are read).  The result is bit-identical to hifa4_quantize_qkv on
 * q followed by hifa4_attention_fwd.  Supported for Bc = 64, d = 128,
 * qmean = 0, normalizer = 0; anything else returns HIFA4_ERR_UNSUPPORTED
 * without a launch.  Other arguments, status word and scheduling note as
 * hifa4_attention_fwd. */
int hifa4_attention_fwd_qraw(const hifa4_shape* shape, const void* q, const float* s,
                             const hifa4_qkv* kv, const hifa4_attn_params* prm, void* out,
                             void* workspace, int* d_status, void* stream);

/* Experiment, not a default path: hifa4_attention_fwd with S = Q-hat K-hat^T issued
 * as tcgen05.mma kind::f8f6f4 (the 8-bit MMA kind nearest to the "HIF4 Cube" of
 * Algorithm 1's comments).  Element x micro-exponent (an integer up to 28) is exact
 * in E4M3; the E6M2 group scale is not, so S is accumulated separately per
 * 64-channel group and the two partial sums are combined with the FP32 group
 * scales by the softmax threads (exact products, one rounding).  The call first
 * derives the E4M3 images and group scales of Q and K from qkv's packed codes and
 * metadata into `workspace` (hifa4_f8qk_workspace_bytes(), 256-byte aligned), then
 * runs the attention kernel; P V is unchanged (v_mma is read).  d = 128, Bc = 64,
 * qmean = 0, normalizer = 0, p_dtype = F16; anything else returns
 * HIFA4_ERR_UNSUPPORTED.  The result meets the same bars against the oracle as
 * hifa4_attention_fwd (the scores are the correctly rounded exact sums). */
size_t hifa4_f8qk_workspace_bytes(const hifa4_shape* shape);
int hifa4_attention_fwd_f8qk(const hifa4_shape* shape, const hifa4_qkv* qkv,
                             const hifa4_attn_params* prm, void* out, void* workspace,
                             size_t workspace_bytes, int* d_status, void* stream);

/* Workspace for hifa4_attention_fwd_raw: all hifa4_qkv buffers (each rounded up
 * to 256 bytes; the two Q-Mean vectors only when prm->qmean = 1) plus the
 * attention workspace. */
size_t hifa4_attention_raw_workspace_bytes(const hifa4_shape* shape, const hifa4_attn_params* prm);

/* Algorithm 1 end to end on raw post-RoPE Q/K/V: hifa4_quantize_qkv into
 * `workspace`, then hifa4_attention_fwd; where hifa4_attention_fwd_qraw supports
 * the configuration, only K and V are quantized into the workspace and Q is
 * quantized inside the attention kernel (same result).  s, inv_s as in
 * hifa4_quantize_qkv. */
int hifa4_attention_fwd_raw(const hifa4_shape* shape, const void* q, const void* k, const void* v,
                            const float* s, const float* inv_s, const hifa4_attn_params* prm,
                            void* out, void* workspace, size_t workspace_bytes,
                            int* d_status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HIFA4_H */
