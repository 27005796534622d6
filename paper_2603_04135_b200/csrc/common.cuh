// Shared host/device helpers of libdppo (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stdarg.h>
#include <stdio.h>

#include <nvtx3/nvToolsExt.h>

#include "dppo.h"

namespace dppo {

// ---- host: thread-local error message ------------------------------------------------------------
int fail(int code, const char* fmt, ...);          // records the message, returns code
int cuda_fail(cudaError_t e, const char* what);    // DPPO_ERR_CUDA with the CUDA error string
int sm_count();                                    // SMs of the current device (cached per device)

#define DPPO_CHECK_LAUNCH(what)                                        \
    do {                                                               \
        cudaError_t e__ = cudaGetLastError();                          \
        if (e__ != cudaSuccess) return ::dppo::cuda_fail(e__, what);   \
    } while (0)

// ---- host: a named NVTX range around each entry point's host work (its launches show under it in a timeline
// tool; a few nanoseconds when no tool is attached)
struct NvtxRange {
    explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
    NvtxRange(const NvtxRange&) = delete;
    NvtxRange& operator=(const NvtxRange&) = delete;
};

// ---- device: status word ---------------------------------------------------------------------------
__device__ __forceinline__ void set_status(int32_t* status, int32_t code) {
    if (status != nullptr) atomicCAS(status, 0, code);   // first error wins
}

// ---- device: warp / block reductions -----------------------------------------------------------
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

}  // namespace dppo
