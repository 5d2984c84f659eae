// The Gumbel variates of the fused samplers: a fixed fp32 logarithm, so that host and device
// restatements agree bit for bit, applied twice to a uniform made from one Philox word.
#pragma once

#include <cstdint>

namespace sbw {

// ---------------------------------------------------------------------------------------------
// Fixed fp32 natural logarithm for positive normal x; every step is one IEEE operation.
//   ix = bits(x); e = (int)(ix - 0x3f3504f3) >> 23; m = bits^-1(ix - (e << 23)) in [sqrt(1/2), sqrt(2))
//   f = m - 1; r = Horner_{C6..C0}(f); q = fma(r, f, -1/2); t = fma(f*f, q, f)
//   L = fma(e, LN2_HI, fma(e, LN2_LO, t))
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float fixed_log(float x) {
    const uint32_t ix = __float_as_uint(x);
    const int e = static_cast<int>(ix - 0x3f3504f3u) >> 23;
    const float m = __uint_as_float(ix - (static_cast<uint32_t>(e) << 23));
    const float f = __fadd_rn(m, -1.0f);
    float r = 0x1.645de2p-4f;
    r = __fmaf_rn(r, f, -0x1.2432aap-3f);
    r = __fmaf_rn(r, f, 0x1.31747p-3f);
    r = __fmaf_rn(r, f, -0x1.53824cp-3f);
    r = __fmaf_rn(r, f, 0x1.98d7fp-3f);
    r = __fmaf_rn(r, f, -0x1.000382p-2f);
    r = __fmaf_rn(r, f, 0x1.5556d8p-2f);
    const float q = __fmaf_rn(r, f, -0.5f);
    const float t = __fmaf_rn(__fmul_rn(f, f), q, f);
    const float fe = __int2float_rn(e);
    return __fmaf_rn(fe, 0x1.62e43p-1f, __fmaf_rn(fe, -0x1.05c61p-29f, t));
}

// Standard Gumbel variate of a Philox word: u = ((y >> 9) + 1/2) 2^-23 (exact), g = -L(-L(u)).
__device__ __forceinline__ float gumbel_of_word(uint32_t y) {
    const float u = __fmaf_rn(__uint2float_rn(y >> 9), 0x1p-23f, 0x1p-24f);
    return -fixed_log(-fixed_log(u));
}

}  // namespace sbw
