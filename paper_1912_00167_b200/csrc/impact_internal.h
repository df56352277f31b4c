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

// Current value of a launch option (IMPACT_OPT_*).
int64_t option(int32_t which);

// Launch with programmatic stream serialization: the grid may be set up on the device while
// the previous kernel of the stream is still running.  Every kernel of this library starts
// with grid_dependency_wait(), which returns only once that previous kernel has completed
// and its writes are visible, so stream order is kept exactly; what is saved is the launch
// latency between consecutive kernels.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_serialized(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                     cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

#ifdef __CUDACC__
// First statement of every kernel: wait for the kernel before this one on the stream (a
// no-op when there is none), then let the kernel after this one begin its own set-up.
__device__ __forceinline__ void grid_dependency_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
#endif

}  // namespace impact

#define IMPACT_CUDA_TRY(expr)                                        \
    do {                                                             \
        cudaError_t e_ = (expr);                                     \
        if (e_ != cudaSuccess) return ::impact::record_cuda_error(e_); \
    } while (0)
