// Host-side helpers shared by the entry points of the SBW library: argument checks, the
// per-thread CUDA error slot, cached device properties.
#pragma once

#include <cmath>
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/sbw.h"

// Bounds-flag build (-DSBW_DEBUG, relocatable device code): every global access of the three core
// kernels is preceded by a check of its row / column / position against the call's sizes.  A
// failed check records its site in a device-side flag word and the access is skipped -- no trap,
// no device assert -- and sbw_debug_flags() reads the words back.  It stands in for a memory
// checker on machines where none can be run; release builds compile the checks away.
#ifdef SBW_DEBUG
extern __device__ unsigned int g_sbw_debug[4];   // [0]: bit mask of failed sites, [1]: failures, [2]: checks passed
#define SBW_CHECKED(ok, site)                                                            \
    ((ok) ? (atomicAdd(&g_sbw_debug[2], 1u), true)                                       \
          : (atomicOr(&g_sbw_debug[0], 1u << (site)), atomicAdd(&g_sbw_debug[1], 1u), false))
#else
#define SBW_CHECKED(ok, site) (true)
#endif
// check sites
#define SBW_SITE_BIAS_VECTOR 0
#define SBW_SITE_BIAS_SCALAR 1
#define SBW_SITE_SAMPLE_LOAD 2
#define SBW_SITE_SAMPLE_WORKSPACE 3
#define SBW_SITE_SAMPLE_OUTPUT 4
#define SBW_SITE_DETECT_TOKEN 5
#define SBW_SITE_DETECT_OUTPUT 6

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
