// rslrl_gae_scan_static: the GAE scan + normalisation for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc once they are running: a simulator plug-in
// whose device memory was handed over to the simulator's own pool at start-up, a control loop
// with a hard period (cudaMalloc may synchronise the whole device and may fail when memory is
// tight), or a process that has been told to stay within a fixed memory budget.  The normal
// entry point, rslrl_gae_scan, asks such a caller for a scratch buffer it has no way to
// provide.  This variant keeps the scratch (one (count, mean, M2) triple per scan block) in a
// fixed array that is part of the library image, so the call allocates nothing at all.
#include "../../include/rslrl_b200.h"
#include "kernels.h"

#include <mutex>

namespace rslrl { void set_global_error(const char* msg); }

namespace {

constexpr int kStaticMaxEnvs = RSLRL_GAE_STATIC_MAX_ENVS;
constexpr int kStaticBlocks = kStaticMaxEnvs / 128;           // scan blocks of 128 environments
constexpr int kStaticFloats = 3 * kStaticBlocks;              // 96 KiB

// Lives in every GPU that loads the library, until the process exits.
static __device__ __align__(256) float g_gae_scratch[kStaticFloats];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
float* g_scratch_ptr[kMaxDevices] = {};

// In host code `g_gae_scratch` is only a handle for the runtime, not an address the GPU can
// use: the device address has to be asked for, once per device, with that device current.
cudaError_t scratch_for_current_device(float** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_ptr[dev]) {
        float* p = nullptr;
        e = cudaGetSymbolAddress((void**)&p, g_gae_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" rslrl_status rslrl_gae_scan_static(const float* d_rewards, const float* d_values, const uint8_t* d_dones,
                                              const uint8_t* d_timeouts, const float* d_last_values,
                                              float* d_returns, float* d_advantages, int32_t T, int32_t N,
                                              float gamma, float lam, int32_t normalize, int32_t unbiased,
                                              float adv_eps, void* cuda_stream) {
    if (T < 0 || N < 0) return RSLRL_ERR_INVALID_ARG;
    if (N > kStaticMaxEnvs) {
        rslrl::set_global_error("rslrl_gae_scan_static: more than RSLRL_GAE_STATIC_MAX_ENVS environments; "
                                "use rslrl_gae_scan with caller-provided scratch");
        return RSLRL_ERR_UNSUPPORTED;
    }
    // The address lookup comes before the empty-size return on purpose: an empty call (T = 0 or N = 0) at
    // start-up is the way to get the one-time work of a device out of the way (the lookup, and with lazy module
    // loading the loading of the module that holds the array), so that no later call has any left to do.
    float* scratch = nullptr;
    if (scratch_for_current_device(&scratch) != cudaSuccess) {
        rslrl::set_global_error("rslrl_gae_scan_static: cudaGetSymbolAddress failed");
        return RSLRL_ERR_CUDA;
    }
    if (T == 0 || N == 0) return RSLRL_OK;
    if (!d_rewards || !d_values || !d_dones || !d_timeouts || !d_last_values || !d_returns || !d_advantages)
        return RSLRL_ERR_INVALID_ARG;
    if ((long long)T * N >= (1ll << 31)) return RSLRL_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(d_advantages) & 15u) return RSLRL_ERR_ALIGNMENT;
    // Nothing in the array has to start at zero: the scan writes the triple of every block
    // before the normalisation of the same call reads it, and no other slot is read.
    const cudaError_t e = rslrl::launch_gae(d_rewards, d_values, d_dones, d_timeouts, d_last_values, d_returns,
                                            d_advantages, T, N, gamma, lam, normalize, unbiased, adv_eps, scratch,
                                            (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? RSLRL_OK : RSLRL_ERR_CUDA;
}
