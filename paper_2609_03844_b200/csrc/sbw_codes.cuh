// Order codes of logits: unsigned integers whose order is the total order of the values' bit
// patterns (+NaN > +inf > ... > +0 > -0 > ... > -inf > -NaN).  fp32: 32-bit codes.  bf16: 16-bit
// codes, bits ^ 0xffff for negative values and bits ^ 0x8000 otherwise.  The row passes of the
// top-k kernels take one 16-byte vector at a time: its largest code, then the elements only if
// that reaches the bound.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/sbw.h"

namespace sbw {

__device__ __forceinline__ uint32_t order_code(uint32_t bits) {
    return (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
}
__device__ __forceinline__ uint32_t order_decode(uint32_t code) {
    return (code & 0x80000000u) ? (code & 0x7fffffffu) : ~code;
}

// A signed integer with the order of order_code: signed_key(b) ^ 0x80000000 == order_code(b).
__device__ __forceinline__ int32_t signed_key(uint32_t bits) {
    return static_cast<int32_t>(bits ^ (static_cast<uint32_t>(static_cast<int32_t>(bits) >> 31) & 0x7fffffffu));
}

// The codes of both bf16 halves of a word at once.
__device__ __forceinline__ uint32_t packed_codes(uint32_t w) {
    uint32_t sign;   // 0xffff in each half whose value is negative (selector bit 3: replicate the byte's msb)
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(sign) : "r"(w), "r"(0u), "r"(0xBB99u));
    return w ^ (sign | 0x80008000u);
}

// Largest code among the 4 (fp32) or 8 (bf16) logits of a vector.
template <int DTYPE>
__device__ __forceinline__ uint32_t vector_max_code(const uint4 &w) {
    if constexpr (DTYPE == SBW_DTYPE_F32) {
        // signed keys (the magnitude bits of negative values flipped) cost two operations each; the
        // largest key with its sign bit flipped is the largest code
        const int32_t k = max(max(signed_key(w.x), signed_key(w.y)), max(signed_key(w.z), signed_key(w.w)));
        return static_cast<uint32_t>(k) ^ 0x80000000u;
    } else {
        const uint32_t m = __vmaxu2(__vmaxu2(packed_codes(w.x), packed_codes(w.y)),
                                    __vmaxu2(packed_codes(w.z), packed_codes(w.w)));
        return max(m >> 16, m & 0xffffu);
    }
}

// Code of logit i of a vector.
template <int DTYPE>
__device__ __forceinline__ uint32_t element_code(const uint4 &w, int i) {
    const uint32_t *e = reinterpret_cast<const uint32_t *>(&w);
    if constexpr (DTYPE == SBW_DTYPE_F32) return order_code(e[i]);
    else return (packed_codes(e[i >> 1]) >> (16 * (i & 1))) & 0xffffu;
}

// Code of column `col` of a row in memory.
template <int DTYPE>
__device__ __forceinline__ uint32_t scalar_code(const char *row_ptr, uint32_t col) {
    if constexpr (DTYPE == SBW_DTYPE_F32) return order_code(reinterpret_cast<const uint32_t *>(row_ptr)[col]);
    else return packed_codes(reinterpret_cast<const uint16_t *>(row_ptr)[col]) & 0xffffu;
}

}  // namespace sbw
