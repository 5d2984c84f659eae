// Host-side helpers shared by the entry points of the SBW library: argument checks, the
// per-thread CUDA error slot, cached device properties.
#pragma once

#include <cmath>
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/sbw.h"

namespace sbw {

// cudaError_t of the calling thread's last failing runtime call.
int &last_cuda_error_slot();

inline int cuda_fail(cudaError_t e) {
    last_cuda_error_slot() = static_cast<int>(e);
    return SBW_ERR_CUDA;
}

#define SBW_CUDA_TRY(expr)                                  \
    do {                                                    \
        cudaError_t sbw_e_ = (expr);                        \
        if (sbw_e_ != cudaSuccess) return ::sbw::cuda_fail(sbw_e_); \
    } while (0)

struct DeviceInfo {
    int device;
    int sm_count;
};
// Properties of the current device (queried once per device and cached).
int current_device_info(DeviceInfo *out);

// Eq. 1: the integer threshold ceil(gamma * 2^32) lies in [1, 2^32]; the kernels compare
// x <= thr_minus_1 so that it fits 32 bits.
inline uint32_t threshold_minus_one(double gamma) {
    const double t = std::ceil(gamma * 4294967296.0);
    const uint64_t thr = static_cast<uint64_t>(t);
    return static_cast<uint32_t>(thr - 1u);
}

inline bool valid_common(int dtype, int ctx_width, double gamma, int scheme) {
    if (dtype != SBW_DTYPE_F32 && dtype != SBW_DTYPE_BF16) return false;
    if (ctx_width < 1 || ctx_width > SBW_MAX_CTX_WIDTH) return false;
    if (!(gamma > 0.0 && gamma < 1.0)) return false;
    if (scheme != SBW_SCHEME_CONTEXT && scheme != SBW_SCHEME_SELFSALT) return false;
    return true;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Launch with programmatic stream serialisation: the kernel may be scheduled while its
// predecessor in the stream is still draining; it must execute `griddepcontrol.wait` before it
// touches memory that earlier work in the stream may have written.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t stream,
                              Args... args) {
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
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

}  // namespace sbw
