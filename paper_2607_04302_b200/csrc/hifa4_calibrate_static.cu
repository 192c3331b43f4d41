// hifa4_smooth_calibrate_static: the calibration entry point for callers that cannot give the
// library a scratch buffer.  Its scratch is a fixed array in device global memory that every GPU
// loading the library holds until the process exits.
#include <mutex>

#include "hifa4_internal.h"
#include "hifa4_device.cuh"

namespace hifa4 {

// Per-sample channel maxima of K and Q: 2 * S * Hkv * d floats, at most this many.
// 1 Mi floats = 4 MiB per device, e.g. 64 samples x 8 KV heads x d = 256 eight times over.
constexpr size_t STATIC_SCRATCH_FLOATS = HIFA4_STATIC_CALIB_MAX_FLOATS;
static __device__ __align__(256) float g_calib_scratch[STATIC_SCRATCH_FLOATS];

// In host code the name g_calib_scratch is only a handle for the runtime, not a device address:
// the address each device gave the array is looked up once per device with that device current.
constexpr int MAX_DEVICES = 64;
static float* g_scratch_ptr[MAX_DEVICES];
static std::mutex g_scratch_mutex;

static int scratch_for_current_device(float** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return HIFA4_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
        float* p = nullptr;
        if (cudaGetSymbolAddress((void**)&p, g_calib_scratch) != cudaSuccess || !p) return HIFA4_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return HIFA4_OK;
}

}  // namespace hifa4

using namespace hifa4;

extern "C" int hifa4_smooth_calibrate_static(const void* q_cal, const void* k_cal, int S, int Hq, int Hkv,
                                             int Ncal, int d, const int* q_to_kv, int dt, int mode,
                                             float alpha, float* s, float* inv_s,
                                             hifa4_calib_stats* host_stats, void* stream)
{
    if (S <= 0 || Hkv <= 0 || d <= 0) return HIFA4_ERR_INVALID_ARG;
    const size_t need = 2 * (size_t)S * (size_t)Hkv * (size_t)d;
    if (need > STATIC_SCRATCH_FLOATS) return HIFA4_ERR_WORKSPACE;   // larger sets: hifa4_smooth_calibrate
    float* scratch = nullptr;
    int rc = scratch_for_current_device(&scratch);
    if (rc) return rc;
    // same kernels and the same clearing of the scratch as the entry point that takes a workspace
    return hifa4_smooth_calibrate(q_cal, k_cal, S, Hq, Hkv, Ncal, d, q_to_kv, dt, mode, alpha, s, inv_s,
                                  scratch, host_stats, stream);
}
