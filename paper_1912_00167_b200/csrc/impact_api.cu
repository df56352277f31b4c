// Housekeeping entry points and the host helpers shared by the other translation units.
#include <cuda_runtime.h>

#include <atomic>

#include "impact.h"
#include "impact_internal.h"

namespace impact {

static thread_local int32_t g_last_cuda_error = 0;

int32_t record_cuda_error(cudaError_t e) {
    g_last_cuda_error = (int32_t)e;
    (void)cudaGetLastError();  // clear the sticky-less error so later calls start clean
    return IMPACT_ERR_CUDA;
}

const DeviceInfo* current_device_info() {
    constexpr int kMaxDevices = 64;
    static DeviceInfo infos[kMaxDevices];
    static bool ready[kMaxDevices] = {};
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { record_cuda_error(e); return nullptr; }
    if (dev < 0 || dev >= kMaxDevices) { record_cuda_error(cudaErrorInvalidDevice); return nullptr; }
    if (!ready[dev]) {
        DeviceInfo di;
        di.device = dev;
        e = cudaDeviceGetAttribute(&di.sm_count, cudaDevAttrMultiProcessorCount, dev);
        if (e == cudaSuccess)
            e = cudaDeviceGetAttribute(&di.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
        if (e != cudaSuccess) { record_cuda_error(e); return nullptr; }
        infos[dev] = di;
        ready[dev] = true;
    }
    return &infos[dev];
}

// Launch options: process-wide, read by every loss call at launch time (defaults in the order of IMPACT_OPT_*).
static std::atomic<int64_t> g_options[IMPACT_NUM_OPTIONS] = {
    {1},           // IMPACT_OPT_EARLY_PREFETCH
    {48ll << 20},  // IMPACT_OPT_PREFETCH_BYTES
    {0},           // IMPACT_OPT_WINDOW_BYTES: chosen per launch
};
int64_t option(int32_t which) { return g_options[which].load(std::memory_order_relaxed); }

}  // namespace impact

extern "C" int32_t impact_set_option(int32_t option, int64_t value) {
    if (option < 0 || option >= IMPACT_NUM_OPTIONS || value < 0) return IMPACT_ERR_INVALID_ARG;
    if (option == IMPACT_OPT_WINDOW_BYTES && value != 0 && (value < 16 * 1024 || value > 160 * 1024)) return IMPACT_ERR_INVALID_ARG;
    impact::g_options[option].store(value, std::memory_order_relaxed);
    return IMPACT_OK;
}

extern "C" int64_t impact_get_option(int32_t option) {
    if (option < 0 || option >= IMPACT_NUM_OPTIONS) return -1;
    return impact::option(option);
}

extern "C" int32_t impact_version(void) { return IMPACT_VERSION; }

extern "C" const char* impact_status_string(int32_t status) {
    switch (status) {
        case IMPACT_OK: return "ok";
        case IMPACT_ERR_INVALID_ARG: return "invalid argument";
        case IMPACT_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case IMPACT_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case IMPACT_ERR_EMPTY: return "circular buffer is empty";
        case IMPACT_ERR_FULL: return "circular buffer is full";
        case IMPACT_ERR_CUDA: return "CUDA runtime error";
        default: return "unknown status";
    }
}

extern "C" int32_t impact_last_cuda_error(void) { return impact::g_last_cuda_error; }
