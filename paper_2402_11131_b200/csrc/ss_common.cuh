// Internal helpers shared by the CUDA translation units of libss_msa.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "ss_msa.h"

namespace ss {

// Workspace header: word 0 = device status, the rest of the first 256 bytes is reserved.
constexpr size_t kWsHeaderBytes = 256;

__device__ __forceinline__ void set_status(void* workspace, int32_t code) {
    atomicCAS(reinterpret_cast<int*>(workspace), 0, code);   // keep the first error
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

// Programmatic dependent launch.  A kernel launched with launch_after_previous may be scheduled while the
// previous kernel of the stream drains; it must call wait_for_previous_kernel() before it touches global
// memory, which restores plain stream order for everything after the call.
__device__ __forceinline__ void wait_for_previous_kernel() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_after_previous(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace ss
