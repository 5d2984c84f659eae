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
