// Host-side helpers shared by the translation units of libimpact (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "impact.h"

namespace impact {

// Records a CUDA failure for impact_last_cuda_error() and maps it to IMPACT_ERR_CUDA.
int32_t record_cuda_error(cudaError_t e);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Properties of the current device, queried once per device.
struct DeviceInfo {
    int device = -1;
    int sm_count = 0;
    int max_smem_optin = 0;
};
// Returns nullptr (and records the error) when no CUDA device is usable.
const DeviceInfo* current_device_info();

}  // namespace impact

#define IMPACT_CUDA_TRY(expr)                                        \
    do {                                                             \
        cudaError_t e_ = (expr);                                     \
        if (e_ != cudaSuccess) return ::impact::record_cuda_error(e_); \
    } while (0)
