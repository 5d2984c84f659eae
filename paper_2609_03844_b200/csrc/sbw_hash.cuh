// Device-side integer hashing for Stateless Bernoulli Watermarking, written for sm_100a.
//
// Everything here lives in registers.  The green test of Eq. 1 needs only word 0 of the
// Philox4x32-10 block whose counter is (v, 0, 0, 0), which lets three of the ten rounds shrink:
//   round 0: c1 = c2 = c3 = 0, so one 32x32->64 product and one xor remain, and the new c0 is
//            just k0;
//   round 1: c0 = k0 does not depend on the candidate, so its product is a per-row constant
//            when the seed is per row (context scheme);
//   rounds 8, 9: only the half-products that reach word 0 are formed.
// The Gumbel stream of the fused sampler needs all four words and uses the plain block.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace sbw {

constexpr uint32_t kPhiloxM0 = 0xD2511F53u;
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u;
constexpr uint32_t kPhiloxW1 = 0xBB67AE85u;

// The Weyl increments of the Philox key schedule, handed to the kernels as launch arguments.
// Adding a 32-bit literal costs two instructions on sm_100; adding a value that sits in a
// register or in the constant bank costs one, and the per-candidate key schedule has 16 adds.
struct Weyl {
    uint32_t w0, w1;
};
inline Weyl make_weyl() { return Weyl{kPhiloxW0, kPhiloxW1}; }

__device__ __forceinline__ void mulhilo(uint32_t a, uint32_t b, uint32_t &hi, uint32_t &lo) {
    const uint64_t p = static_cast<uint64_t>(a) * b;   // one IMAD.WIDE.U32
    hi = static_cast<uint32_t>(p >> 32);
    lo = static_cast<uint32_t>(p);
}

// Section 2.3: Jenkins' six-step 32-bit mix.  a + (a << s) is written as a product so that it
// becomes one integer multiply-add.
__device__ __forceinline__ uint32_t jenkins(uint32_t a) {
    a = a * 4097u + 0x7ed55d16u;
    a = (a ^ 0xc761c23cu) ^ (a >> 19);
    a = a * 33u + 0x165667b1u;
    a = (a + 0xd3a2646cu) ^ (a << 9);
    a = a * 9u + 0xfd7046c5u;
    a = (a ^ 0xb55a4f09u) ^ (a >> 16);
    return a;
}

// One full Philox round on (c0..c3) with round key (k0, k1).
__device__ __forceinline__ void philox_round(uint32_t &c0, uint32_t &c1, uint32_t &c2, uint32_t &c3,
                                             uint32_t k0, uint32_t k1) {
    uint32_t h0, l0, h1, l1;
    mulhilo(kPhiloxM0, c0, h0, l0);
    mulhilo(kPhiloxM1, c2, h1, l1);
    c0 = h1 ^ c1 ^ k0;
    c1 = l1;
    c2 = h0 ^ c3 ^ k1;
    c3 = l0;
}

// Plain Philox4x32-10 block: all four words (used by the Gumbel stream).
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int i = 0; i < 10; ++i)
        philox_round(c0, c1, c2, c3, k0 + static_cast<uint32_t>(i) * kPhiloxW0,
                     k1 + static_cast<uint32_t>(i) * kPhiloxW1);
    return make_uint4(c0, c1, c2, c3);
}

// The same block under round keys prepared by the host (one key for the whole launch).
struct BlockKeys {
    uint32_t k0[10], k1[10];
};
inline BlockKeys make_block_keys(uint32_t k0, uint32_t k1) {
    BlockKeys bk;
    for (int i = 0; i < 10; ++i) {
        bk.k0[i] = k0 + static_cast<uint32_t>(i) * kPhiloxW0;
        bk.k1[i] = k1 + static_cast<uint32_t>(i) * kPhiloxW1;
    }
    return bk;
}
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const BlockKeys &bk) {
#pragma unroll
    for (int i = 0; i < 10; ++i) philox_round(c0, c1, c2, c3, bk.k0[i], bk.k1[i]);
    return make_uint4(c0, c1, c2, c3);
}

// Round keys of a seed that is shared by many candidates (context scheme: one seed per row).
// Everything that does not depend on the candidate is folded in here, once per row.
struct RowKeys {
    uint32_t k0[10];   // k0 + i*W0; entries 1..7 and 9 are read
    uint32_t k1[10];   // k1 + i*W1; entries 0 and 3..8 are read
    uint32_t r1_c2;    // hi(M0*k0) ^ k1[1]: xor-ed with lo(M0*v) it is c2 after round 1
    uint32_t r2_c3k;   // lo(M0*k0) ^ k1[2]: c3 after round 1, pre-mixed with round 2's key
};

__device__ __forceinline__ RowKeys make_row_keys(uint64_t r) {
    RowKeys rk;
    const uint32_t k0 = static_cast<uint32_t>(r), k1 = static_cast<uint32_t>(r >> 32);
#pragma unroll
    for (int i = 0; i < 10; ++i) {
        rk.k0[i] = k0 + static_cast<uint32_t>(i) * kPhiloxW0;
        rk.k1[i] = k1 + static_cast<uint32_t>(i) * kPhiloxW1;
    }
    uint32_t ah, al;
    mulhilo(kPhiloxM0, k0, ah, al);
    rk.r1_c2 = ah ^ rk.k1[1];
    rk.r2_c3k = al ^ rk.k1[2];
    return rk;
}

// Word 0 of Philox4x32-10(counter (v,0,0,0)) under precomputed row keys.
__device__ __forceinline__ uint32_t philox_word0(uint32_t v, const RowKeys &rk) {
    uint32_t h, l, c0, c1, c2, c3;
    // round 0: c0 <- k0, c1 <- 0, c2 <- hi(M0 v) ^ k1, c3 <- lo(M0 v)
    mulhilo(kPhiloxM0, v, h, l);
    c2 = h ^ rk.k1[0];
    // round 1: c0 <- hi(M1 c2) ^ k0', c1 <- lo(M1 c2), c2 <- hi(M0 k0) ^ c3 ^ k1', c3 <- lo(M0 k0)
    uint32_t h1, l1;
    mulhilo(kPhiloxM1, c2, h1, l1);
    c0 = h1 ^ rk.k0[1];
    c1 = l1;
    c2 = l ^ rk.r1_c2;
    // round 2 with c3 = lo(M0 k0) folded into the key
    {
        uint32_t h0, l0;
        mulhilo(kPhiloxM0, c0, h0, l0);
        mulhilo(kPhiloxM1, c2, h1, l1);
        c0 = h1 ^ c1 ^ rk.k0[2];
        c1 = l1;
        c2 = h0 ^ rk.r2_c3k;
        c3 = l0;
    }
#pragma unroll
    for (int i = 3; i < 8; ++i)
        philox_round(c0, c1, c2, c3, rk.k0[i], rk.k1[i]);
    // round 8: only c1 and c2 of the result reach word 0
    const uint32_t n1 = kPhiloxM1 * c2;
    const uint32_t n2 = __umulhi(kPhiloxM0, c0) ^ c3 ^ rk.k1[8];
    // round 9: word 0
    return __umulhi(kPhiloxM1, n2) ^ n1 ^ rk.k0[9];
}

// Word 0 of Philox4x32-10(counter (v,0,0,0), key (lo r, hi r)) for a seed that belongs to one
// candidate only (self-salt scheme, detection).
__device__ __forceinline__ uint32_t philox_word0(uint32_t v, uint64_t r, const Weyl w) {
    uint32_t k0 = static_cast<uint32_t>(r), k1 = static_cast<uint32_t>(r >> 32);
    uint32_t h, l, c0, c1, c2, c3, h0, l0, h1, l1;
    mulhilo(kPhiloxM0, v, h, l);
    c2 = h ^ k1;
    mulhilo(kPhiloxM0, k0, h0, l0);
    mulhilo(kPhiloxM1, c2, h1, l1);
    k0 += w.w0;
    k1 += w.w1;
    c0 = h1 ^ k0;
    c1 = l1;
    c2 = h0 ^ l ^ k1;
    c3 = l0;
#pragma unroll
    for (int i = 2; i < 8; ++i) {
        k0 += w.w0;
        k1 += w.w1;
        philox_round(c0, c1, c2, c3, k0, k1);
    }
    k1 += w.w1;
    k0 += w.w0 + w.w0;
    const uint32_t n1 = kPhiloxM1 * c2;
    const uint32_t n2 = __umulhi(kPhiloxM0, c0) ^ c3 ^ k1;
    return __umulhi(kPhiloxM1, n2) ^ n1 ^ k0;
}

// The same two evaluations for N candidates at once, written round by round so that the N
// dependent multiply/xor chains are interleaved in program order: one warp then keeps the
// multiply pipe busy by itself, whatever the occupancy.
//
// Context scheme, N consecutive ids vbase .. vbase+N-1 (which must not wrap past 2^32): the
// round-0 product M0*(vbase+i) is formed as M0*vbase + M0*i with a 64-bit add, which moves N-1
// multiplies off the multiply pipe.
template <int N>
__device__ __forceinline__ void philox_word0_n(uint32_t vbase, const RowKeys &rk, uint32_t (&out)[N]) {
    uint32_t c0[N], c1[N], c2[N], c3[N];
    const uint64_t p0 = static_cast<uint64_t>(kPhiloxM0) * vbase;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const uint64_t p = p0 + static_cast<uint64_t>(kPhiloxM0) * static_cast<uint32_t>(i);
        c2[i] = static_cast<uint32_t>(p >> 32) ^ rk.k1[0];
        c3[i] = static_cast<uint32_t>(p);
    }
#pragma unroll
    for (int i = 0; i < N; ++i) {
        uint32_t h1, l1;
        mulhilo(kPhiloxM1, c2[i], h1, l1);
        c0[i] = h1 ^ rk.k0[1];
        c1[i] = l1;
        c2[i] = c3[i] ^ rk.r1_c2;
    }
#pragma unroll
    for (int i = 0; i < N; ++i) {
        uint32_t h0, l0, h1, l1;
        mulhilo(kPhiloxM0, c0[i], h0, l0);
        mulhilo(kPhiloxM1, c2[i], h1, l1);
        c0[i] = h1 ^ c1[i] ^ rk.k0[2];
        c1[i] = l1;
        c2[i] = h0 ^ rk.r2_c3k;
        c3[i] = l0;
    }
#pragma unroll
    for (int r = 3; r < 8; ++r) {
#pragma unroll
        for (int i = 0; i < N; ++i) philox_round(c0[i], c1[i], c2[i], c3[i], rk.k0[r], rk.k1[r]);
    }
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const uint32_t n1 = kPhiloxM1 * c2[i];
        const uint32_t n2 = __umulhi(kPhiloxM0, c0[i]) ^ c3[i] ^ rk.k1[8];
        out[i] = __umulhi(kPhiloxM1, n2) ^ n1 ^ rk.k0[9];
    }
}

// Per-candidate seeds r[i] (self-salt scheme, detection), arbitrary ids v[i].
template <int N>
__device__ __forceinline__ void philox_word0_n(const uint32_t (&v)[N], const uint64_t (&r)[N],
                                               uint32_t (&out)[N], const Weyl w) {
    uint32_t c0[N], c1[N], c2[N], c3[N], k0[N], k1[N];
#pragma unroll
    for (int i = 0; i < N; ++i) {
        k0[i] = static_cast<uint32_t>(r[i]);
        k1[i] = static_cast<uint32_t>(r[i] >> 32);
        uint32_t h, l, h0, l0;
        mulhilo(kPhiloxM0, v[i], h, l);
        mulhilo(kPhiloxM0, k0[i], h0, l0);
        c2[i] = h ^ k1[i];           // after round 0
        c1[i] = l;                   // parked: lo(M0 v), consumed by round 1
        c0[i] = h0;                  // parked: hi(M0 k0)
        c3[i] = l0;                  // c3 after round 1
    }
#pragma unroll
    for (int i = 0; i < N; ++i) {
        k0[i] += w.w0;
        k1[i] += w.w1;
        uint32_t h1, l1;
        mulhilo(kPhiloxM1, c2[i], h1, l1);
        c2[i] = c0[i] ^ c1[i] ^ k1[i];
        c0[i] = h1 ^ k0[i];
        c1[i] = l1;
    }
#pragma unroll
    for (int rd = 2; rd < 8; ++rd) {
#pragma unroll
        for (int i = 0; i < N; ++i) {
            k0[i] += w.w0;
            k1[i] += w.w1;
            philox_round(c0[i], c1[i], c2[i], c3[i], k0[i], k1[i]);
        }
    }
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const uint32_t n1 = kPhiloxM1 * c2[i];
        const uint32_t n2 = __umulhi(kPhiloxM0, c0[i]) ^ c3[i] ^ (k1[i] + w.w1);
        out[i] = __umulhi(kPhiloxM1, n2) ^ n1 ^ (k0[i] + w.w0 + w.w0);
    }
}

// Table 12 "additive" PRF: key times the sum of the context ids.
__device__ __forceinline__ uint64_t seed_context(uint64_t key, const int32_t *ctx, int W) {
    uint64_t sigma = 0;
    for (int i = 0; i < W; ++i)
        sigma += static_cast<uint32_t>(ctx[i]);
    return key * sigma;
}

// Table 12 "anchored minhash" PRF.  The window is the context plus the candidate and the anchor
// is the candidate, so min_x J(x)J(v) = J(v) * min(J(v), min_i J(ctx_i)); the inner minimum over
// the context is a per-row constant `jctx_min`.
__device__ __forceinline__ uint64_t seed_selfsalt(uint64_t key, uint32_t jctx_min, uint32_t v) {
    const uint32_t jv = jenkins(v);
    const uint64_t prod = static_cast<uint64_t>(jv) * min(jv, jctx_min);
    return key * prod;
}

__device__ __forceinline__ uint32_t jenkins_min(const int32_t *ctx, int W) {
    uint32_t m = 0xFFFFFFFFu;
    for (int i = 0; i < W; ++i)
        m = min(m, jenkins(static_cast<uint32_t>(ctx[i])));
    return m;
}

}  // namespace sbw
