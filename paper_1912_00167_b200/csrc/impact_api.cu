// Housekeeping entry points and the host helpers shared by the other translation units.
#include <cuda_runtime.h>

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

}  // namespace impact

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
