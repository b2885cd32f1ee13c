// Status strings, thread-local error text and the architecture gate shared by all entry points.
#include <stdarg.h>
#include <stdio.h>

#include "rdk_common.cuh"

namespace rdk {

static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

int cuda_fail(cudaError_t e, const char* what) {
    set_error("%s: %s (%s)", what, cudaGetErrorName(e), cudaGetErrorString(e));
    return RDK_ERR_CUDA;
}

int check_arch() {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    static thread_local int cached_dev = -1, cached_major = 0;
    if (dev != cached_dev) {
        int major = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
        cached_dev = dev;
        cached_major = major;
    }
    if (cached_major != 10) {
        set_error("device %d has compute capability %d.x; this library contains sm_100a code only", dev, cached_major);
        return RDK_ERR_ARCH;
    }
    return RDK_OK;
}

}  // namespace rdk

extern "C" int rdk_version(void) { return 1 * 1000 + 0; }

extern "C" const char* rdk_status_string(int status) {
    switch (status) {
        case RDK_OK: return "ok";
        case RDK_ERR_INVALID_ARG: return "invalid argument";
        case RDK_ERR_BAD_IDS: return "duplicate kept id";
        case RDK_ERR_EMPTY_INTERSECTION: return "no kept id inside the target vocabulary";
        case RDK_ERR_UNSUPPORTED: return "unsupported request";
        case RDK_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case RDK_ERR_ARCH: return "device is not sm_100";
        case RDK_ERR_CUDA: return "CUDA call failed";
        case RDK_ERR_TIMEOUT: return "bounded device-side wait expired";
        default: return "unknown status";
    }
}

extern "C" const char* rdk_last_error(void) { return rdk::g_err; }
