// Small shared pieces of the C ABI: error strings, architecture check, launch accounting.
#include "internal.h"

namespace ag {
thread_local int g_last_cuda_error = 0;
std::atomic<unsigned long long> g_launch_count{0};

ag_status cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int)e;
    cudaGetLastError();  // clear the sticky-free error state
    return e == cudaErrorMemoryAllocation ? AG_ERR_NOMEM : AG_ERR_CUDA;
}

ag_status check_arch() {
    int dev = 0, major = 0;
    AG_CUDA(cudaGetDevice(&dev));
    AG_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    return major == 10 ? AG_OK : AG_ERR_UNSUPPORTED_ARCH;
}
}  // namespace ag

extern "C" const char* ag_strerror(ag_status s) {
    switch (s) {
        case AG_OK: return "ok";
        case AG_ERR_ARG: return "bad argument";
        case AG_ERR_CUDA: return "CUDA call failed";
        case AG_ERR_UNSUPPORTED_ARCH: return "device is not sm_100";
        case AG_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case AG_ERR_UNMANNED_SM: return "an SM of the set never got a thread block";
        case AG_ERR_NOISY_PROBE: return "latency tiers could not be separated";
        case AG_ERR_STALE_AMAP: return "affinity map does not belong to this buffer";
        case AG_ERR_NOMEM: return "out of memory";
    }
    return "unknown status";
}

extern "C" int ag_last_cuda_error(void) { return ag::g_last_cuda_error; }
extern "C" uint64_t ag_kernel_launch_count(void) { return ag::g_launch_count.load(); }
