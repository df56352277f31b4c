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
        int mem_khz = 0, bus_bits = 0;
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&mem_khz, cudaDevAttrMemoryClockRate, dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&bus_bits, cudaDevAttrGlobalMemoryBusWidth, dev);
        if (e != cudaSuccess) { record_cuda_error(e); return nullptr; }
        // bytes per ns = 2 transfers per clock x clock in GHz x bus bytes; 8 TB/s / 148 SMs = 55 B/ns on B200
        di.hbm_bytes_per_ns_per_sm = 2.0 * (mem_khz * 1e-6) * (bus_bits / 8.0) / (di.sm_count > 0 ? di.sm_count : 1);
        if (!(di.hbm_bytes_per_ns_per_sm > 1.0)) di.hbm_bytes_per_ns_per_sm = 55.0;
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
