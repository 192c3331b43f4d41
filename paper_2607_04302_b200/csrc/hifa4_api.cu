// C-ABI entry points of libhifa4: argument validation, size queries and launches.
#include <atomic>
#include <cmath>
#include <cstring>

#include "hifa4_internal.h"
#include "hifa4_device.cuh"

namespace hifa4 {

static std::atomic<unsigned long long> g_calls[4];

void count_launch() { g_calls[3].fetch_add(1, std::memory_order_relaxed); }

static int check_arch()
{
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return HIFA4_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return HIFA4_ERR_CUDA;
    return major == 10 ? HIFA4_OK : HIFA4_ERR_ARCH;
}

static int build_map(int Hq, int Hkv, const int* q_to_kv, HeadMap& qmap, HeadMap& kmap)
{
    if (Hq <= 0 || Hkv <= 0 || Hq > HIFA4_MAX_HEADS || Hkv > HIFA4_MAX_HEADS) return HIFA4_ERR_INVALID_ARG;
    if (!q_to_kv && Hq % Hkv) return HIFA4_ERR_INVALID_ARG;
    std::memset(&qmap, 0, sizeof(qmap));
    std::memset(&kmap, 0, sizeof(kmap));
    for (int h = 0; h < Hq; ++h) {
        int g = q_to_kv ? q_to_kv[h] : h / (Hq / Hkv);
        if (g < 0 || g >= Hkv) return HIFA4_ERR_INVALID_ARG;
        qmap.kv_of[h] = (short)g;
    }
    for (int g = 0; g < Hkv; ++g) kmap.kv_of[g] = (short)g;
    return HIFA4_OK;
}

static int check_shape(const hifa4_shape* s)
{
    if (!s) return HIFA4_ERR_INVALID_ARG;
    if (s->B <= 0 || s->N <= 0 || s->d <= 0 || s->Hq <= 0 || s->Hkv <= 0) return HIFA4_ERR_INVALID_ARG;
    if (s->in_dtype != HIFA4_F16 && s->in_dtype != HIFA4_BF16) return HIFA4_ERR_INVALID_ARG;
    if (s->d != 64 && s->d != 128 && s->d != 256) return HIFA4_ERR_UNSUPPORTED;
    if (s->N % 64) return HIFA4_ERR_UNSUPPORTED;
    if ((long long)s->B * s->Hq > 65535 || (long long)s->B * s->Hkv > 65535) return HIFA4_ERR_UNSUPPORTED;
    return HIFA4_OK;
}

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

}  // namespace hifa4

using namespace hifa4;

extern "C" {

const char* hifa4_status_string(int status)
{
    switch (status) {
    case HIFA4_OK: return "ok";
    case HIFA4_ERR_INVALID_ARG: return "invalid argument";
    case HIFA4_ERR_UNSUPPORTED: return "unsupported shape or flag";
    case HIFA4_ERR_WORKSPACE: return "workspace missing or too small";
    case HIFA4_ERR_ARCH: return "device is not sm_100";
    case HIFA4_ERR_CUDA: return "CUDA call failed";
    case HIFA4_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
    }
}

void hifa4_get_counters(unsigned long long out[4])
{
    if (!out) return;
    for (int i = 0; i < 4; ++i) out[i] = g_calls[i].load(std::memory_order_relaxed);
}

int hifa4_smooth_calibrate(const void* q_cal, const void* k_cal, int S, int Hq, int Hkv, int Ncal,
                           int d, const int* q_to_kv, int dt, int mode, float alpha, float* s,
                           float* inv_s, float* absmax_ws, hifa4_calib_stats* host_stats,
                           void* stream)
{
    g_calls[0].fetch_add(1, std::memory_order_relaxed);
    if (!q_cal || !k_cal || !s || !inv_s || !absmax_ws) return HIFA4_ERR_INVALID_ARG;
    if (S <= 0 || Ncal <= 0) return HIFA4_ERR_INVALID_ARG;
    if (dt != HIFA4_F16 && dt != HIFA4_BF16) return HIFA4_ERR_INVALID_ARG;
    if (d != 64 && d != 128 && d != 256) return HIFA4_ERR_UNSUPPORTED;
    if (mode < 0 || (mode & ~0x3FF)) return HIFA4_ERR_INVALID_ARG;
    const int aggregator = mode >> 8;                              // HIFA4_AGG_* flag
    mode &= 0xFF;
    if (aggregator > 2) return HIFA4_ERR_INVALID_ARG;
    if (mode == 3) return HIFA4_ERR_UNSUPPORTED;
    if (mode < 0 || mode > 4) return HIFA4_ERR_INVALID_ARG;
    if (mode == 4 && !(alpha >= 0.f && alpha <= 1.f)) return HIFA4_ERR_INVALID_ARG;
    HeadMap qmap, kmap;
    int rc = build_map(Hq, Hkv, q_to_kv, qmap, kmap);
    if (rc) return rc;
    if ((rc = check_arch())) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    double a = mode == 1 ? 0.5 : mode == 2 ? 0.25 : mode == 4 ? (double)alpha : 0.0;
    size_t n = (size_t)S * Hkv * d;
    float* kmax = absmax_ws;
    float* qmax = absmax_ws + n;
    if (cudaMemsetAsync(absmax_ws, 0, 2 * n * sizeof(float), st) != cudaSuccess) return HIFA4_ERR_CUDA;
    if (mode != 0) {
        if (launch_absmax(dt, k_cal, kmap, S, Hkv, Hkv, Ncal, d, kmax, st) != cudaSuccess) return HIFA4_ERR_CUDA;
        if (launch_absmax(dt, q_cal, qmap, S, Hq, Hkv, Ncal, d, qmax, st) != cudaSuccess) return HIFA4_ERR_CUDA;
    }
    if (launch_smooth_finalize(kmax, qmax, S, Hkv * d, a, mode == 0, aggregator, nullptr, s, inv_s, st) != cudaSuccess)
        return HIFA4_ERR_CUDA;
    if (host_stats) {
        host_stats->rho_K = NAN;
        host_stats->T_KQ = NAN;
        host_stats->branch = mode;
        host_stats->alpha = (float)a;
    }
    return HIFA4_OK;
}

int hifa4_smooth_calibrate_auto(const void* q_cal, const void* k_cal, int S, int Hq, int Hkv, int Ncal,
                                int d, const int* q_to_kv, int dt, float* s, float* inv_s, float* absmax_ws,
                                void* gate_ws, float* d_stats, void* stream)
{
    g_calls[0].fetch_add(1, std::memory_order_relaxed);
    if (!q_cal || !k_cal || !s || !inv_s || !absmax_ws || !gate_ws) return HIFA4_ERR_INVALID_ARG;
    if (S <= 0 || Ncal <= 0) return HIFA4_ERR_INVALID_ARG;
    if (dt != HIFA4_F16 && dt != HIFA4_BF16) return HIFA4_ERR_INVALID_ARG;
    if (d != 64 && d != 128 && d != 256) return HIFA4_ERR_UNSUPPORTED;
    if (((uintptr_t)gate_ws & 7u) != 0) return HIFA4_ERR_INVALID_ARG;
    HeadMap qmap, kmap;
    int rc = build_map(Hq, Hkv, q_to_kv, qmap, kmap);
    if (rc) return rc;
    const long long nk = (long long)S * Hkv * Ncal * d;
    if (nk >= (1ll << 32)) return HIFA4_ERR_UNSUPPORTED;          // 32-bit histogram counters
    if ((rc = check_arch())) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t n = (size_t)S * Hkv * d;
    float* kmax = absmax_ws;
    float* qmax = absmax_ws + n;
    if (cudaMemsetAsync(absmax_ws, 0, 2 * n * sizeof(float), st) != cudaSuccess) return HIFA4_ERR_CUDA;
    if (launch_absmax(dt, k_cal, kmap, S, Hkv, Hkv, Ncal, d, kmax, st) != cudaSuccess) return HIFA4_ERR_CUDA;
    if (launch_absmax(dt, q_cal, qmap, S, Hq, Hkv, Ncal, d, qmax, st) != cudaSuccess) return HIFA4_ERR_CUDA;
    if (launch_gate(dt, k_cal, nk, kmax, qmax, (int)n, gate_ws, d_stats, st) != cudaSuccess) return HIFA4_ERR_CUDA;
    if (launch_smooth_finalize(kmax, qmax, S, Hkv * d, 0.0, 0, 0, gate_result(gate_ws), s, inv_s, st) != cudaSuccess)
        return HIFA4_ERR_CUDA;
    return HIFA4_OK;
}

size_t hifa4_quant_bytes(const hifa4_shape* shape, int which, int part)
{
    if (check_shape(shape) != HIFA4_OK) return 0;
    if (which < HIFA4_Q || which > HIFA4_V || part < HIFA4_PART_CODES || part > HIFA4_PART_AUX) return 0;
    size_t H = which == HIFA4_Q ? shape->Hq : shape->Hkv;
    size_t elems = (size_t)shape->B * H * shape->N * shape->d;
    switch (part) {
    case HIFA4_PART_AUX: return which == HIFA4_V ? 0 : elems / shape->d * sizeof(float);
    case HIFA4_PART_CODES: return elems / 2;
    case HIFA4_PART_META: return elems / 64 * 4;
    default: return elems * 2;
    }
}

int hifa4_quantize_qkv(const hifa4_shape* shape, const void* q, const void* k, const void* v,
                       const float* s, const float* inv_s, const hifa4_qkv* out, int* d_status,
                       void* stream)
{
    (void)d_status;
    g_calls[1].fetch_add(1, std::memory_order_relaxed);
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!out || ((s == nullptr) != (inv_s == nullptr))) return HIFA4_ERR_INVALID_ARG;
    if (q && (!out->q_codes || !out->q_meta || !out->q_mma)) return HIFA4_ERR_INVALID_ARG;
    if (k && (!out->k_codes || !out->k_meta || !out->k_mma)) return HIFA4_ERR_INVALID_ARG;
    if (v && (!out->v_codes || !out->v_meta || !out->v_mma)) return HIFA4_ERR_INVALID_ARG;
    if ((out->q_mu == nullptr) != (out->k_sum == nullptr)) return HIFA4_ERR_INVALID_ARG;
    HeadMap qmap, kmap;
    if ((rc = build_map(shape->Hq, shape->Hkv, shape->q_to_kv, qmap, kmap))) return rc;
    if ((rc = check_arch())) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (launch_quantize_qkv(shape->in_dtype, *shape, qmap, q, k, v, s, inv_s, *out, st) != cudaSuccess)
        return HIFA4_ERR_CUDA;
    return HIFA4_OK;
}

static int check_attn(const hifa4_shape* shape, const hifa4_attn_params* prm)
{
    int rc = check_shape(shape);
    if (rc) return rc;
    if (!prm) return HIFA4_ERR_INVALID_ARG;
    if (prm->out_dtype < HIFA4_F16 || prm->out_dtype > HIFA4_F32) return HIFA4_ERR_INVALID_ARG;
    if (prm->softmax_scale < 0.f || !std::isfinite(prm->softmax_scale)) return HIFA4_ERR_INVALID_ARG;
    if (prm->Br != 128) return HIFA4_ERR_UNSUPPORTED;
    if (prm->Bc != 64 && prm->Bc != 128) return HIFA4_ERR_UNSUPPORTED;
    if (shape->d == 256 && prm->Bc != 64) return HIFA4_ERR_UNSUPPORTED;
    if (prm->qmean != 0 && prm->qmean != 1) return HIFA4_ERR_INVALID_ARG;
    if (prm->normalizer != 0 && prm->normalizer != 1) return HIFA4_ERR_INVALID_ARG;
    if (prm->p_dtype != HIFA4_F16 && prm->p_dtype != HIFA4_F32) return HIFA4_ERR_INVALID_ARG;
    if (prm->p_dtype == HIFA4_F32 && (prm->Bc != 64 || shape->d == 64 || prm->normalizer)) return HIFA4_ERR_UNSUPPORTED;
    return HIFA4_OK;
}

size_t hifa4_attention_workspace_bytes(const hifa4_shape* shape, const hifa4_attn_params* prm)
{
    (void)shape; (void)prm;
    return 0;
}

static int attention_common(const hifa4_shape* shape, const hifa4_qkv* qkv, const hifa4_attn_params* prm,
                            void* out, const hifa4_debug* dbg, const hifa4_mass_stats* stats, int* d_status,
                            void* stream, bool selftest = false, const void* q_raw = nullptr,
                            const float* q_scale = nullptr, const F8Operands* f8 = nullptr)
{
    g_calls[2].fetch_add(1, std::memory_order_relaxed);
    int rc = check_attn(shape, prm);
    if (rc) return rc;
    if (!qkv || !out || (!q_raw && !qkv->q_mma) || !qkv->k_mma || !qkv->v_mma) return HIFA4_ERR_INVALID_ARG;
    if (prm->qmean && (!qkv->q_mu || !qkv->k_sum)) return HIFA4_ERR_INVALID_ARG;
    if (dbg) {
        if (dbg->n_blocks < 0 || dbg->n_blocks > HIFA4_MAX_DEBUG_BLOCKS) return HIFA4_ERR_INVALID_ARG;
        if (dbg->n_blocks > 0 && !dbg->blocks) return HIFA4_ERR_INVALID_ARG;
        for (int i = 0; i < dbg->n_blocks; ++i) {
            const int* t = dbg->blocks + 3 * i;
            if (t[0] < 0 || t[0] >= shape->B || t[1] < 0 || t[1] >= shape->Hq || t[2] < 0 ||
                t[2] >= (shape->N + 127) / 128)
                return HIFA4_ERR_INVALID_ARG;
        }
    }
    HeadMap qmap, kmap;
    if ((rc = build_map(shape->Hq, shape->Hkv, shape->q_to_kv, qmap, kmap))) return rc;
    if ((rc = check_arch())) return rc;
    return launch_attention(*shape, qmap, *qkv, *prm, out, dbg, stats, d_status, (cudaStream_t)stream, selftest,
                            q_raw, q_scale, f8);
}

int hifa4_attention_fwd(const hifa4_shape* shape, const hifa4_qkv* qkv, const hifa4_attn_params* prm,
                        void* out, void* workspace, const hifa4_debug* dbg, int* d_status,
                        void* stream)
{
    (void)workspace;
    return attention_common(shape, qkv, prm, out, dbg, nullptr, d_status, stream);
}

int hifa4_attention_fwd_qraw(const hifa4_shape* shape, const void* q, const float* s, const hifa4_qkv* kv,
                             const hifa4_attn_params* prm, void* out, void* workspace, int* d_status,
                             void* stream)
{
    (void)workspace;
    if (!q) return HIFA4_ERR_INVALID_ARG;
    int rc = check_attn(shape, prm);
    if (rc) return rc;
    if (!attention_qraw_supported(*shape, *prm)) return HIFA4_ERR_UNSUPPORTED;
    return attention_common(shape, kv, prm, out, nullptr, nullptr, d_status, stream, false, q, s);
}

size_t hifa4_f8qk_workspace_bytes(const hifa4_shape* shape)
{
    if (check_shape(shape) != HIFA4_OK || shape->d != 128) return 0;
    const size_t rq = (size_t)shape->B * shape->Hq * shape->N, rk = (size_t)shape->B * shape->Hkv * shape->N;
    return align256(rq * 128) + align256(rk * 128) + align256(rq * 2 * sizeof(float)) + align256(rk * 2 * sizeof(float));
}

int hifa4_attention_fwd_f8qk(const hifa4_shape* shape, const hifa4_qkv* qkv, const hifa4_attn_params* prm, void* out,
                             void* workspace, size_t workspace_bytes, int* d_status, void* stream)
{
    int rc = check_attn(shape, prm);
    if (rc) return rc;
    if (shape->d != 128 || prm->Bc != 64 || prm->qmean || prm->normalizer || prm->p_dtype == HIFA4_F32) return HIFA4_ERR_UNSUPPORTED;
    if (!qkv || !out || !qkv->q_codes || !qkv->q_meta || !qkv->k_codes || !qkv->k_meta || !qkv->v_mma) return HIFA4_ERR_INVALID_ARG;
    const size_t need = hifa4_f8qk_workspace_bytes(shape);
    if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 255)) return HIFA4_ERR_WORKSPACE;
    if ((rc = check_arch())) return rc;
    const size_t rq = (size_t)shape->B * shape->Hq * shape->N, rk = (size_t)shape->B * shape->Hkv * shape->N;
    char* base = (char*)workspace;
    void* q_f8 = base; base += align256(rq * 128);
    void* k_f8 = base; base += align256(rk * 128);
    float* q_gs = (float*)base; base += align256(rq * 2 * sizeof(float));
    float* k_gs = (float*)base;
    if (launch_f8_images(*shape, *qkv, q_f8, q_gs, k_f8, k_gs, (cudaStream_t)stream) != cudaSuccess) return HIFA4_ERR_CUDA;
    const F8Operands f8{q_f8, k_f8, q_gs, k_gs};
    hifa4_qkv tmp = *qkv;
    if (!tmp.q_mma) tmp.q_mma = q_f8;                       // not read by this launch; the common check wants non-null
    if (!tmp.k_mma) tmp.k_mma = k_f8;
    return attention_common(shape, &tmp, prm, out, nullptr, nullptr, d_status, stream, false, nullptr, nullptr, &f8);
}

int hifa4_selftest_wait_timeout(const hifa4_shape* shape, const hifa4_qkv* qkv, const hifa4_attn_params* prm,
                                void* out, int* d_status, void* stream)
{
    if (!d_status) return HIFA4_ERR_INVALID_ARG;
    return attention_common(shape, qkv, prm, out, nullptr, nullptr, d_status, stream, true);
}

int hifa4_attention_fwd_stats(const hifa4_shape* shape, const hifa4_qkv* qkv, const hifa4_attn_params* prm,
                              void* out, void* workspace, const hifa4_mass_stats* stats, int* d_status,
                              void* stream)
{
    (void)workspace;
    if (!stats || !stats->hist || stats->n_bins < 1 || !(stats->lo < stats->hi)) return HIFA4_ERR_INVALID_ARG;
    return attention_common(shape, qkv, prm, out, nullptr, stats, d_status, stream);
}

static size_t qkv_layout(const hifa4_shape* shape, int qmean, char* base, hifa4_qkv* o)
{
    size_t off = 0;
    void** slots[9] = {(void**)&o->q_codes, (void**)&o->q_meta, &o->q_mma,
                       (void**)&o->k_codes, (void**)&o->k_meta, &o->k_mma,
                       (void**)&o->v_codes, (void**)&o->v_meta, &o->v_mma};
    for (int w = 0; w < 3; ++w)
        for (int p = 0; p < 3; ++p) {
            if (o) *slots[3 * w + p] = base + off;
            off += align256(hifa4_quant_bytes(shape, w, p));
        }
    if (o) { o->q_mu = nullptr; o->k_sum = nullptr; }
    if (qmean) {
        if (o) o->q_mu = (float*)(base + off);
        off += align256(hifa4_quant_bytes(shape, HIFA4_Q, HIFA4_PART_AUX));
        if (o) o->k_sum = (float*)(base + off);
        off += align256(hifa4_quant_bytes(shape, HIFA4_K, HIFA4_PART_AUX));
    }
    return off;
}

size_t hifa4_attention_raw_workspace_bytes(const hifa4_shape* shape, const hifa4_attn_params* prm)
{
    if (check_attn(shape, prm) != HIFA4_OK) return 0;
    return qkv_layout(shape, prm->qmean, nullptr, nullptr) + hifa4_attention_workspace_bytes(shape, prm);
}

int hifa4_attention_fwd_raw(const hifa4_shape* shape, const void* q, const void* k, const void* v,
                            const float* s, const float* inv_s, const hifa4_attn_params* prm,
                            void* out, void* workspace, size_t workspace_bytes, int* d_status,
                            void* stream)
{
    int rc = check_attn(shape, prm);
    if (rc) return rc;
    if (!q || !k || !v || !out) return HIFA4_ERR_INVALID_ARG;
    size_t need = hifa4_attention_raw_workspace_bytes(shape, prm);
    if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 255)) return HIFA4_ERR_WORKSPACE;
    hifa4_qkv bufs;
    size_t used = qkv_layout(shape, prm->qmean, (char*)workspace, &bufs);
    if ((s == nullptr) != (inv_s == nullptr)) return HIFA4_ERR_INVALID_ARG;
    // K and V here, Q inside the attention kernel: pays once the Q-hat image (written, then read) is large; measured
    // on B200 at d = 128: -1 to -3 % of the two launches from 64k query rows up, slower below
    if (attention_qraw_supported(*shape, *prm) && (long long)shape->B * shape->Hq * shape->N >= 65536) {
        if ((rc = hifa4_quantize_qkv(shape, nullptr, k, v, s, inv_s, &bufs, d_status, stream))) return rc;
        return hifa4_attention_fwd_qraw(shape, q, s, &bufs, prm, out, (char*)workspace + used, d_status, stream);
    }
    if ((rc = hifa4_quantize_qkv(shape, q, k, v, s, inv_s, &bufs, d_status, stream))) return rc;
    return hifa4_attention_fwd(shape, &bufs, prm, out, (char*)workspace + used, nullptr, d_status, stream);
}

}  // extern "C"
