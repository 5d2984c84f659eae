// Integer-throughput probe: register-only loops of one instruction kind, timed with the SM clock.
// Gives the measured ceiling (thread-operations per clock per SM) for the instruction mix of the
// Philox hash, against which the bias / detect kernels are placed on the roofline.
#include "sbw_common.cuh"
#include "../../include/sbw_probe.h"

namespace sbw {
namespace {

constexpr int kIlp = 8;

template <int KIND>
__global__ void probe_kernel(int steps, int64_t *out_cycles, uint32_t *out_sink) {
    uint32_t x[kIlp], y[kIlp];
    uint64_t p[kIlp];
    float f[kIlp];
#pragma unroll
    for (int i = 0; i < kIlp; ++i) {
        x[i] = threadIdx.x * 2654435761u + i * 40503u + blockIdx.x;
        y[i] = x[i] ^ 0x9E3779B9u;
        p[i] = (static_cast<uint64_t>(x[i]) << 32) | y[i];
        f[i] = __uint_as_float(0x3f800000u | (x[i] & 0xffffu));
    }
    const uint32_t k0 = steps * 0x85EBCA6Bu + 1u, k1 = steps * 0xC2B2AE35u + 3u;
    __syncthreads();
    const long long t0 = clock64();
    for (int s = 0; s < steps; ++s) {
#pragma unroll
        for (int i = 0; i < kIlp; ++i) {
            if constexpr (KIND == SBW_PROBE_MULWIDE) {
                asm volatile("{ .reg .b32 lo, hi; mov.b64 {lo, hi}, %0; mad.wide.u32 %0, lo, %1, %0; }"
                             : "+l"(p[i]) : "r"(0xD2511F53u));
            } else if constexpr (KIND == SBW_PROBE_LOP3) {
                asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[i]) : "r"(y[i]), "r"(k0));
            } else if constexpr (KIND == SBW_PROBE_IADD3) {
                asm volatile("{ .reg .b32 t; add.u32 t, %0, %1; add.u32 %0, t, %2; }"
                             : "+r"(x[i]) : "r"(y[i]), "r"(k0));
            } else if constexpr (KIND == SBW_PROBE_IMAD) {
                asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(x[i]) : "r"(0xCD9E8D57u), "r"(k1));
            } else if constexpr (KIND == SBW_PROBE_PHILOX) {
                const uint64_t a = static_cast<uint64_t>(x[i]) * 0xD2511F53u;
                const uint64_t b = static_cast<uint64_t>(y[i]) * 0xCD9E8D57u;
                const uint32_t nx = static_cast<uint32_t>(b >> 32) ^ static_cast<uint32_t>(a) ^ k0;
                const uint32_t ny = static_cast<uint32_t>(a >> 32) ^ static_cast<uint32_t>(b) ^ k1;
                x[i] = nx;
                y[i] = ny;
            } else if constexpr (KIND == SBW_PROBE_FFMA) {
                asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(f[i]) : "f"(0.99999f), "f"(1e-7f));
            } else if constexpr (KIND == SBW_PROBE_MULHI) {
                asm volatile("mul.hi.u32 %0, %0, %1;" : "+r"(x[i]) : "r"(0xD2511F53u));
            } else if constexpr (KIND == SBW_PROBE_MULWIDE_XOR) {
                asm volatile("{ .reg .b32 lo, hi; .reg .b64 q; mul.wide.u32 q, %0, %1; mov.b64 {lo, hi}, q; "
                             "xor.b32 %0, lo, hi; }" : "+r"(x[i]) : "r"(0xD2511F53u));
            } else if constexpr (KIND == SBW_PROBE_DUAL_FP) {
                asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[i]) : "r"(y[i]), "r"(k0));
                asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(f[i]) : "f"(0.99999f), "f"(1e-7f));
            } else if constexpr (KIND == SBW_PROBE_DUAL_INT) {
                asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[i]) : "r"(y[i]), "r"(k0));
                asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(y[i]) : "r"(0xCD9E8D57u), "r"(k1));
            } else {
                asm volatile("add.u64 %0, %0, %1;" : "+l"(p[i]) : "l"((static_cast<uint64_t>(k1) << 32) | k0));
            }
        }
    }
    const long long t1 = clock64();
    uint32_t acc = 0;
#pragma unroll
    for (int i = 0; i < kIlp; ++i)
        acc ^= x[i] ^ y[i] ^ static_cast<uint32_t>(p[i]) ^ static_cast<uint32_t>(p[i] >> 32) ^ __float_as_uint(f[i]);
    if (acc == 0x12345678u) *out_sink = acc;      // practically never true; keeps the chains live
    if (threadIdx.x == 0) out_cycles[blockIdx.x] = t1 - t0;
}

}  // namespace
}  // namespace sbw

extern "C" int sbw_int_probe(int kind, int steps, int blocks_per_sm, int threads, int64_t *out_cycles,
                             uint32_t *out_sink, void *stream) {
    using namespace sbw;
    if (kind < 0 || kind >= SBW_PROBE_KINDS || steps <= 0 || blocks_per_sm <= 0 || threads <= 0 ||
        threads > 1024 || threads % 32 != 0 || !out_cycles || !out_sink)
        return SBW_ERR_INVALID_ARG;
    DeviceInfo di;
    const int rc = current_device_info(&di);
    if (rc != SBW_OK) return rc;
    const unsigned grid = static_cast<unsigned>(di.sm_count) * blocks_per_sm;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (kind) {
        case SBW_PROBE_MULWIDE: probe_kernel<SBW_PROBE_MULWIDE><<<grid, threads, 0, s>>>(steps, out_cycles, out_sink); break;
        case SBW_PROBE_LOP3: probe_kernel<SBW_PROBE_LOP3><<<grid, threads, 0, s>>>(steps, out_cycles, out_sink); break;
        case SBW_PROBE_IADD3: probe_kernel<SBW_PROBE_IADD3><<<grid, threads, 0, s>>>(steps, out_cycles, out_sink); break;
        case SBW_PROBE_IMAD: probe_kernel<SBW_PROBE_IMAD><<<grid, threads, 0, s>>>(steps, out_cycles, out_sink); break;
        case SBW_PROBE_PHILOX: probe_kernel<SBW_PROBE_PHILOX><<<grid, threads, 0, s>>>(steps, out_cycles, out_sink); break;
        case SBW_PROBE_FFMA: probe_kernel<SBW_PROBE_FFMA><<<grid, threads, 0, s>>>(steps, out_cycles, out_sink); break;
        case SBW_PROBE_MULHI: probe_kernel<SBW_PROBE_MULHI><<<grid, threads, 0, s>>>(steps, out_cycles, out_sink); break;
        case SBW_PROBE_MULWIDE_XOR: probe_kernel<SBW_PROBE_MULWIDE_XOR><<<grid, threads, 0, s>>>(steps, out_cycles, out_sink); break;
        case SBW_PROBE_DUAL_FP: probe_kernel<SBW_PROBE_DUAL_FP><<<grid, threads, 0, s>>>(steps, out_cycles, out_sink); break;
        case SBW_PROBE_DUAL_INT: probe_kernel<SBW_PROBE_DUAL_INT><<<grid, threads, 0, s>>>(steps, out_cycles, out_sink); break;
        default: probe_kernel<SBW_PROBE_ADD64><<<grid, threads, 0, s>>>(steps, out_cycles, out_sink); break;
    }
    SBW_CUDA_TRY(cudaGetLastError());
    return SBW_OK;
}
