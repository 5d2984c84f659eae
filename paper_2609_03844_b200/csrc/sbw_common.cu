// Library-wide host state of the SBW CUDA library: version string, per-thread CUDA error slot,
// cached device properties.
#include "sbw_common.cuh"

#include <mutex>

namespace sbw {

int &last_cuda_error_slot() {
    static thread_local int slot = 0;
    return slot;
}

int current_device_info(DeviceInfo *out) {
    constexpr int kMaxDevices = 64;
    static int sm_counts[kMaxDevices] = {0};
    static std::mutex mu;
    int dev = 0;
    SBW_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SBW_ERR_UNSUPPORTED;
    int sms;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (sm_counts[dev] == 0) {
            int v = 0;
            SBW_CUDA_TRY(cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev));
            sm_counts[dev] = v > 0 ? v : 1;
        }
        sms = sm_counts[dev];
    }
    out->device = dev;
    out->sm_count = sms;
    return SBW_OK;
}

}  // namespace sbw

extern "C" const char *sbw_version(void) { return "sbw-b200 0.1 (SBW-spec v1, sm_100a)"; }

extern "C" int sbw_last_cuda_error(void) { return sbw::last_cuda_error_slot(); }

#ifdef SBW_DEBUG
__device__ unsigned int g_sbw_debug[4];

// Bounds-flag build only: copies the four flag words to `out` (host) and clears them when asked to.
// Synchronises the device.
extern "C" int sbw_debug_flags(unsigned int *out, int clear) {
    SBW_CUDA_TRY(cudaDeviceSynchronize());
    if (out) SBW_CUDA_TRY(cudaMemcpyFromSymbol(out, g_sbw_debug, sizeof(g_sbw_debug)));
    if (clear) {
        const unsigned int zero[4] = {0, 0, 0, 0};
        SBW_CUDA_TRY(cudaMemcpyToSymbol(g_sbw_debug, zero, sizeof(zero)));
    }
    return SBW_OK;
}

// Bounds-flag build only: one check that passes and one that fails (site 31), touching no memory,
// so that a test can see the recording work.
namespace {
__global__ void debug_selftest_kernel(int n) {
    (void)SBW_CHECKED(n >= 0, 30);
    (void)SBW_CHECKED(n < 0, 31);
}
}  // namespace
extern "C" int sbw_debug_selftest(void *stream) {
    debug_selftest_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(1);
    SBW_CUDA_TRY(cudaGetLastError());
    return SBW_OK;
}
#endif
