// Version, thread-local error text and small host utilities of libdppo.
#include "common.cuh"
#include <string.h>

namespace dppo {

static thread_local char g_err[512] = "";

int fail(int code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

int cuda_fail(cudaError_t e, const char* what) {
    return fail(DPPO_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

int sm_count() {
    static int cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

}  // namespace dppo

extern "C" int dppo_version(void) { return 100; }   // 0.1.0

extern "C" const char* dppo_last_error(void) { return dppo::g_err; }
