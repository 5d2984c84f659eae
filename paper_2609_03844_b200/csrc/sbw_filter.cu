// sbw_bias_sample_filtered: bias (Eq. 2 of the paper) + top-k / top-p truncation + Gumbel-max
// sampling (the paper's Appendix F samples with temperature 0.7 and top_p = 0.8).
//
// The biased logits l' are produced once -- the full-vocabulary bias kernel writes a biased copy
// of the rows into the workspace -- and everything after that is memory traffic over that copy,
// one CTA (or one cluster of CTAs) per row:
//   order    candidates are ranked by order-encoded bits, ties by column; with key_m the code of
//            the row maximum, a candidate is the 64-bit composite (key_m - code) << 32 | column,
//            and "kept" is always "composite <= boundary".
//   weights  integers W = trunc(2^(40 + (l' - m) c)) from a fixed fp32 2^f (see nucleus_weight),
//            so sums are exact and the kept set does not depend on the order of addition.
//   select   the boundary is found by a radix descent over the distance key_m - code: a pass
//            histograms the candidates of the current range into 2048 bins (weight and number),
//            a block scan finds the bin in which the running weight crosses the target (top-k: k
//            candidates; top-p: ceil(p32 Z / 2^32) of weight, Z being the total of the first
//            histogram), and the range narrows to that bin.  When the bin holds at most kListCap
//            candidates they are gathered, sorted and scanned in shared memory, which gives the
//            boundary directly; a range of one distance that is still too full is a group of
//            equal logits, cut by column with one ordered counting pass.
//   sample   one last pass draws Gumbel variates for the kept candidates only and takes the
//            arg max of fmaf(l', 1/tau, g), ties to the lowest column.
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include "sbw_codes.cuh"
#include "sbw_common.cuh"
#include "sbw_gumbel.cuh"
#include "sbw_hash.cuh"

namespace sbw {

int bias_logits_impl(void *logits, int dtype, int64_t B, int64_t V, int64_t ld, int64_t vocab_offset,
                     const int32_t *ctx_tokens, int ctx_width, uint64_t key, double gamma, float delta,
                     int scheme, cudaStream_t stream);
int bias_copy_impl(const void *src, int64_t ld_src, void *dst, int dtype, int64_t B, int64_t V, int64_t ld,
                   int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width, uint64_t key, double gamma,
                   float delta, int scheme, cudaStream_t stream, bool *done);

namespace {

constexpr int kFilterThreads = 512;
constexpr int kFilterWarps = kFilterThreads / 32;
constexpr int kBins = 2048;
constexpr int kBinBits = 11;
constexpr int kListCap = 2048;
constexpr int kBigCap = 4096;
constexpr int kLastColumns = 2600;   // what the last retry aims to gather: below kBigCap with room for ties
constexpr uint64_t kAll = ~0ull;

struct FilterArgs {
    const void *biased;    // [B, ld] biased logits, rows 16-byte aligned
    int64_t B, V, ld;
    uint32_t vocab_offset;
    float inv_tau;         // 1 / temperature, fp32 division
    float c;               // (float)(log2(e) / temperature)
    int64_t top_k;         // 0: off
    uint64_t p32;          // floor(top_p 2^32) in [1, 2^32]; 0: top-p off
    uint32_t step_lo, step_hi;
    BlockKeys gkeys;       // Philox round keys of the Gumbel stream
    int32_t *out_tokens;
    int32_t *out_kept;     // nullable
    // candidate path (top_k set): the unbiased rows and what the green test needs; raw = nullptr
    // means `biased` already holds the biased rows
    const void *raw;
    int64_t ld_raw;
    const int32_t *ctx;
    int W;
    int scheme;
    uint64_t key;
    uint32_t thr_m1;
    float delta;           // in the logits' precision, widened
    Weyl weyl;
};

// Weights go into the histogram as four 11-bit limbs, each its own array of 32-bit counters:
// native 32-bit shared-memory adds instead of 64-bit compare-and-swap loops, which crawl when the
// candidates crowd into a few bins (bf16 logits have a few hundred distinct values near the top).
// A limb counter holds up to 2^21 candidates' worth.  The list reuses the histogram's space.
constexpr int kWeightTab = 1280;   // ten binades of bf16 codes
constexpr int kLimbs = 4;
constexpr int kLimbBits = 11;
constexpr int64_t kMaxFilterV = int64_t(1) << 21;

struct FilterShared {
    union {
        struct {
            unsigned int hist_c[kBins];
            unsigned int hist_l[kLimbs][kBins];
        };
        unsigned long long list[kListCap];
        unsigned long long list_big[kBigCap];   // the last retry before the radix descent
        struct {
            unsigned long long list_view[kListCap];
            // bf16 rows, top-p total: the weights of the kWeightTab codes from the row maximum down
            // and of the kWeightTab lowest codes that can have a weight, filled once per row
            unsigned long long wtab[2 * kWeightTab + 1];   // the last entry is 0
        };
    };
    unsigned long long red[kFilterWarps];
    unsigned long long bcast[4];
    unsigned int list_n;
    unsigned int red32[kFilterWarps];
    // what the CTAs of a cluster tell each other about their parts of the row
    unsigned int part_max, part_floor, part_deep, part_last;
    unsigned long long part_z;
};

// Codes are compared in units of one representable value of the logits' type: 32 significant
// bits for fp32, the upper 16 for bf16 (whose lower 16 bits are always zero).
template <int DTYPE>
__device__ __forceinline__ uint32_t code_of_bits(uint32_t bits32) {
    const uint32_t c = order_code(bits32);
    return DTYPE == SBW_DTYPE_F32 ? c : c >> 16;
}
template <int DTYPE>
__device__ __forceinline__ float value_of_code(uint32_t code) {
    if constexpr (DTYPE == SBW_DTYPE_F32) return __uint_as_float(order_decode(code));
    // 16-bit code: undo the order map on 16 bits, then widen (the low 16 bits of the value are 0)
    const uint32_t b16 = (code & 0x8000u) ? (code & 0x7fffu) : (~code & 0xffffu);
    return __uint_as_float(b16 << 16);
}

// The two hot passes work on a cheaper monotone key, a signed integer made from the raw bits in
// two operations (flip the magnitude bits of negative values); for bf16 the bits are the widened
// ones, so the key of a negative value carries 0xFFFF in its low half.  key >= key_of_code(c) is
// code >= c.
__device__ __forceinline__ int32_t order_key(uint32_t bits32) {
    return static_cast<int32_t>(bits32 ^ (static_cast<uint32_t>(static_cast<int32_t>(bits32) >> 31) & 0x7fffffffu));
}
template <int DTYPE>
__device__ __forceinline__ uint32_t code_of_key(int32_t key) {
    const uint32_t c = static_cast<uint32_t>(key) ^ 0x80000000u;
    return DTYPE == SBW_DTYPE_F32 ? c : c >> 16;
}
template <int DTYPE>
__device__ __forceinline__ int32_t key_of_code(uint32_t code) {
    return static_cast<int32_t>((DTYPE == SBW_DTYPE_F32 ? code : code << 16) ^ 0x80000000u);
}

// Integer softmax weight of a candidate at distance `dist` below the maximum code (see the oracle
// of this library for the same steps): 2^40 at the maximum, trunc(2^(40 + (l' - m) c)) below it.
__device__ __forceinline__ unsigned long long nucleus_weight(float l, float m, bool is_max, float c) {
    if (is_max) return 1ull << 40;
    const float d = __fsub_rn(l, m);
    float y = __fmul_rn(d, c);
    if (!(y >= -41.0f)) return 0ull;
    if (y > 0.0f) y = 0.0f;
    const float n = rintf(y);
    const float f = __fsub_rn(y, n);
    float p = 0x1.ffcbfcp-17f;
    p = __fmaf_rn(p, f, 0x1.430912p-13f);
    p = __fmaf_rn(p, f, 0x1.5d87fep-10f);
    p = __fmaf_rn(p, f, 0x1.3b2ab6p-7f);
    p = __fmaf_rn(p, f, 0x1.c6b08ep-5f);
    p = __fmaf_rn(p, f, 0x1.ebfbep-3f);
    p = __fmaf_rn(p, f, 0x1.62e43p-1f);
    p = __fmaf_rn(p, f, 0x1p+0f);
    // p 2^(n + 40): n + 40 lies in [-1, 40], so the scale is a normal power of two and exact
    const float scale = __uint_as_float(static_cast<uint32_t>(static_cast<int>(n) + 40 + 127) << 23);
    return __float2ull_rz(__fmul_rn(p, scale));
}

// The row is padded to whole 16-byte vectors; loads are 16 bytes wide, several in flight.
// The same, out of line, for call sites that are reached rarely inside unrolled loops.
__device__ __noinline__ unsigned long long nucleus_weight_rare(float l, float m, float c) {
    return nucleus_weight(l, m, false, c);
}

template <int DTYPE>
__device__ __forceinline__ uint32_t vectors_of(uint32_t V) {
    return (V + (DTYPE == SBW_DTYPE_F32 ? 4 : 8) - 1) / (DTYPE == SBW_DTYPE_F32 ? 4 : 8);
}

// Calls f(column, code) for the columns of 16-byte vectors [vec_begin, nvec) of the row.
template <int DTYPE, typename F>
__device__ __forceinline__ void for_each(const char *row_ptr, uint32_t V, uint32_t vec_begin, uint32_t nvec, F f) {
    constexpr int VEC = DTYPE == SBW_DTYPE_F32 ? 4 : 8;
    constexpr int kInFlight = 4;
    for (uint32_t j0 = vec_begin + threadIdx.x; j0 < nvec; j0 += kInFlight * kFilterThreads) {
        uint4 w[kInFlight];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            const uint32_t j = j0 + u * kFilterThreads;
            w[u] = j < nvec ? reinterpret_cast<const uint4 *>(row_ptr)[j] : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            const uint32_t j = j0 + u * kFilterThreads;
            if (j >= nvec) break;
            const uint32_t *e = reinterpret_cast<const uint32_t *>(&w[u]);
#pragma unroll
            for (int i = 0; i < VEC; ++i) {
                uint32_t bits;
                if constexpr (DTYPE == SBW_DTYPE_F32) bits = e[i];
                else bits = (i & 1) ? (e[i >> 1] & 0xffff0000u) : (e[i >> 1] << 16);
                const uint32_t col = j * VEC + i;
                if (col < V) f(col, code_of_bits<DTYPE>(bits));
            }
        }
    }
}

template <int DTYPE, typename F>
__device__ __forceinline__ void for_each(const char *row_ptr, uint32_t V, F f) {
    for_each<DTYPE>(row_ptr, V, 0u, vectors_of<DTYPE>(V), f);
}

// The same walk handing out f(column, widened bits, key).  Whole vectors need no column check;
// a ragged last vector is done by one thread afterwards.
template <int DTYPE, typename F>
__device__ __forceinline__ void for_each_key(const char *row_ptr, uint32_t V, uint32_t vec_begin, uint32_t nvec, F f) {
    constexpr int VEC = DTYPE == SBW_DTYPE_F32 ? 4 : 8;
    constexpr int kInFlight = 4;
    const uint32_t nfull = min(nvec, V / VEC);
    for (uint32_t j0 = vec_begin + threadIdx.x; j0 < nfull; j0 += kInFlight * kFilterThreads) {
        uint4 w[kInFlight];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            const uint32_t j = j0 + u * kFilterThreads;
            w[u] = j < nfull ? reinterpret_cast<const uint4 *>(row_ptr)[j] : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            const uint32_t j = j0 + u * kFilterThreads;
            if (j >= nfull) break;
            const uint32_t *e = reinterpret_cast<const uint32_t *>(&w[u]);
#pragma unroll
            for (int i = 0; i < VEC; ++i) {
                uint32_t bits;
                if constexpr (DTYPE == SBW_DTYPE_F32) bits = e[i];
                else bits = (i & 1) ? (e[i >> 1] & 0xffff0000u) : (e[i >> 1] << 16);
                f(j * VEC + i, bits, order_key(bits));
            }
        }
    }
    if (nfull < nvec && nfull >= vec_begin && threadIdx.x == 0) {
        const uint4 w = reinterpret_cast<const uint4 *>(row_ptr)[nfull];
        const uint32_t *e = reinterpret_cast<const uint32_t *>(&w);
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
            uint32_t bits;
            if constexpr (DTYPE == SBW_DTYPE_F32) bits = e[i];
            else bits = (i & 1) ? (e[i >> 1] & 0xffff0000u) : (e[i >> 1] << 16);
            if (nfull * VEC + i < V) f(nfull * VEC + i, bits, order_key(bits));
        }
    }
}

// The walk for passes that only compare: fvec(first column, vector) for whole vectors (each
// thread every kFilterThreads-th), fone(column, code) for the columns of a ragged last vector.
template <int DTYPE, typename FV, typename F1>
__device__ __forceinline__ void for_each_vector(const char *row_ptr, uint32_t V, uint32_t vec_begin, uint32_t nvec,
                                                FV fvec, F1 fone) {
    constexpr int VEC = DTYPE == SBW_DTYPE_F32 ? 4 : 8;
    constexpr int kInFlight = 4;   // eight were measured slower here (the kernel is at its register limit)
    const uint32_t nfull = min(nvec, V / VEC);
    for (uint32_t j0 = vec_begin + threadIdx.x; j0 < nfull; j0 += kInFlight * kFilterThreads) {
        uint4 w[kInFlight];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            const uint32_t j = j0 + u * kFilterThreads;
            w[u] = j < nfull ? reinterpret_cast<const uint4 *>(row_ptr)[j] : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            const uint32_t j = j0 + u * kFilterThreads;
            if (j < nfull) fvec(j * VEC, w[u]);
        }
    }
    if (nfull < nvec && nfull >= vec_begin && threadIdx.x == 0)
        for (uint32_t col = nfull * VEC; col < V; ++col) fone(col, scalar_code<DTYPE>(row_ptr, col));
}

__device__ __forceinline__ unsigned long long warp_sum(unsigned long long x) {
    for (int d = 16; d > 0; d >>= 1) x += __shfl_xor_sync(0xffffffffu, x, d);
    return x;
}

// Sum over the CTA, returned to every thread.  Uses sh.red and sh.bcast[3].
__device__ __forceinline__ unsigned long long block_sum(unsigned long long x, FilterShared &sh) {
    x = warp_sum(x);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh.red[threadIdx.x >> 5] = x;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long t = 0;
        for (int w = 0; w < kFilterWarps; ++w) t += sh.red[w];
        sh.bcast[3] = t;
    }
    __syncthreads();
    return sh.bcast[3];
}

// Exclusive prefix over the CTA in thread order.  Uses sh.red.
__device__ __forceinline__ unsigned long long block_exclusive_scan(unsigned long long x, FilterShared &sh) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long incl = x;
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += up;
    }
    __syncthreads();
    if (lane == 31) sh.red[warp] = incl;
    __syncthreads();
    unsigned long long before = 0;
    for (int w = 0; w < warp; ++w) before += sh.red[w];
    return before + incl - x;
}


enum { kModeCount = 0, kModeMass = 1 };

// Bitonic sort of sh.list[0 .. len), len a power of two >= 2, ascending.
__device__ __forceinline__ void sort_list(unsigned long long *list, int len) {
    for (int k = 2; k <= len; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int t = threadIdx.x; t < len / 2; t += kFilterThreads) {
                const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
                const unsigned long long a = list[i], b = list[i + j];
                if ((a > b) == ((i & k) == 0)) {
                    list[i] = b;
                    list[i + j] = a;
                }
            }
            __syncthreads();
        }
    }
}

// The composite of the last kept candidate: the first one, in the order of the composites, at
// which the running weight reaches the target.  MODE count: every candidate weighs 1 and
// `target` is the number to keep.  MODE mass: candidates weigh nucleus_weight, `target` is p32 and
// the weight to reach is ceil(p32 Z / 2^32), Z being the weight of everything at or below `limit`.
// s0: all candidates with a weight lie at distances below 2^s0.
template <int DTYPE, int MODE>
__device__ unsigned long long select_boundary(const char *row_ptr, uint32_t V, uint32_t key_m, float m, float c,
                                              unsigned long long limit, unsigned long long target, int s0,
                                              FilterShared &sh) {
    auto weight = [&](uint32_t dist) -> unsigned long long {
        if (MODE == kModeCount) return 1ull;
        return nucleus_weight(value_of_code<DTYPE>(key_m - dist), m, dist == 0u, c);
    };
    uint32_t r0 = 0;
    int s = s0;
    unsigned long long acc = 0;
    for (int iter = 0; iter < 5; ++iter) {           // the range loses 11 bits per iteration
        const int sub = s > kBinBits ? s - kBinBits : 0;
        for (int i = threadIdx.x; i < kBins; i += kFilterThreads) {
            sh.hist_c[i] = 0u;
#pragma unroll
            for (int l = 0; l < kLimbs; ++l) sh.hist_l[l][i] = 0u;
        }
        if (threadIdx.x == 0) sh.bcast[0] = kBins;
        __syncthreads();
        for_each<DTYPE>(row_ptr, V, [&](uint32_t col, uint32_t code) {
            const uint32_t dist = key_m - code;
            if (((static_cast<unsigned long long>(dist) << 32) | col) > limit) return;
            const uint32_t rel = dist - r0;           // wraps to a large value below the range
            if (s < 32 && (rel >> s) != 0u) return;
            const unsigned long long w = weight(dist);
            if (w == 0ull) return;
            const uint32_t bin = rel >> sub;
            atomicAdd(&sh.hist_c[bin], 1u);
            if (MODE == kModeMass) {
#pragma unroll
                for (int l = 0; l < kLimbs; ++l) {
                    const unsigned int part = static_cast<unsigned int>(w >> (l * kLimbBits)) & ((1u << kLimbBits) - 1u);
                    if (part) atomicAdd(&sh.hist_l[l][bin], part);
                }
            }
        });
        __syncthreads();
        // every thread owns kBins / kFilterThreads consecutive bins
        constexpr int kOwn = kBins / kFilterThreads;
        unsigned long long own[kOwn], sum = 0;
#pragma unroll
        for (int i = 0; i < kOwn; ++i) {
            const int bin = threadIdx.x * kOwn + i;
            if (MODE == kModeCount) {
                own[i] = sh.hist_c[bin];
            } else {
                own[i] = 0ull;
#pragma unroll
                for (int l = 0; l < kLimbs; ++l)
                    own[i] += static_cast<unsigned long long>(sh.hist_l[l][bin]) << (l * kLimbBits);
            }
            sum += own[i];
        }
        if (MODE == kModeMass && iter == 0) {
            const unsigned long long Z = block_sum(sum, sh);
            const unsigned long long lo = target * Z, hi = __umul64hi(target, Z);
            target = (hi << 32) | (lo >> 32);
            if (lo & 0xffffffffull) target += 1;
        }
        unsigned long long run = acc + block_exclusive_scan(sum, sh);
#pragma unroll
        for (int i = 0; i < kOwn; ++i) {
            if (run < target && run + own[i] >= target) {
                sh.bcast[0] = threadIdx.x * kOwn + i;
                sh.bcast[1] = run;
                sh.bcast[2] = sh.hist_c[threadIdx.x * kOwn + i];
            }
            run += own[i];
        }
        __syncthreads();
        const unsigned long long b = sh.bcast[0];
        if (b >= kBins) return limit;                 // target beyond the total: everything stays
        acc = sh.bcast[1];
        const unsigned long long cnt = sh.bcast[2];
        r0 += static_cast<uint32_t>(b) << sub;
        s = sub;
        __syncthreads();

        if (cnt <= kListCap) {
            // gather the candidates of the range, sort them, walk the weights
            if (threadIdx.x == 0) sh.list_n = 0u;
            __syncthreads();
            for_each<DTYPE>(row_ptr, V, [&](uint32_t col, uint32_t code) {
                const uint32_t dist = key_m - code;
                const unsigned long long comp = (static_cast<unsigned long long>(dist) << 32) | col;
                if (comp > limit) return;
                const uint32_t rel = dist - r0;
                if (s < 32 && (rel >> s) != 0u) return;
                if (weight(dist) == 0ull) return;
                const unsigned idx = atomicAdd(&sh.list_n, 1u);
                if (idx < kListCap) sh.list[idx] = comp;
            });
            __syncthreads();
            const int n = static_cast<int>(min(sh.list_n, static_cast<unsigned>(kListCap)));
            int len = 2;
            while (len < n) len <<= 1;
            for (int i = n + threadIdx.x; i < len; i += kFilterThreads) sh.list[i] = kAll;
            __syncthreads();
            sort_list(sh.list, len);
            constexpr int kPer = kListCap / kFilterThreads;
            unsigned long long w[kPer], mine = 0;
#pragma unroll
            for (int i = 0; i < kPer; ++i) {
                const int idx = threadIdx.x * kPer + i;
                w[i] = idx < n ? weight(static_cast<uint32_t>(sh.list[idx] >> 32)) : 0ull;
                mine += w[i];
            }
            if (threadIdx.x == 0) sh.bcast[0] = limit;
            unsigned long long at = acc + block_exclusive_scan(mine, sh);
#pragma unroll
            for (int i = 0; i < kPer; ++i) {
                if (at < target && at + w[i] >= target) sh.bcast[0] = sh.list[threadIdx.x * kPer + i];
                at += w[i];
            }
            __syncthreads();
            const unsigned long long boundary = sh.bcast[0];
            __syncthreads();
            return boundary;
        }
        if (s == 0) {
            // more equal logits than the list holds: keep the first `need` of them by column
            const unsigned long long wt = weight(r0);
            const unsigned long long need = (target - acc + wt - 1) / wt;     // >= 1
            constexpr int VEC = DTYPE == SBW_DTYPE_F32 ? 4 : 8;
            const uint32_t nvec = (V + VEC - 1) / VEC;
            unsigned long long seen = 0;
            if (threadIdx.x == 0) sh.bcast[0] = limit;
            for (uint32_t base = 0; base < nvec && seen < need; base += kFilterThreads) {
                const uint32_t j = base + threadIdx.x;
                uint32_t match = 0;                    // bit i: column j VEC + i belongs to the group
                if (j < nvec) {
                    const uint4 q = reinterpret_cast<const uint4 *>(row_ptr)[j];
                    const uint32_t *e = reinterpret_cast<const uint32_t *>(&q);
#pragma unroll
                    for (int i = 0; i < VEC; ++i) {
                        uint32_t bits;
                        if constexpr (DTYPE == SBW_DTYPE_F32) bits = e[i];
                        else bits = (i & 1) ? (e[i >> 1] & 0xffff0000u) : (e[i >> 1] << 16);
                        const uint32_t col = j * VEC + i;
                        const uint32_t dist = key_m - code_of_bits<DTYPE>(bits);
                        if (col < V && dist == r0 && ((static_cast<unsigned long long>(dist) << 32) | col) <= limit)
                            match |= 1u << i;
                    }
                }
                const unsigned long long cntm = __popc(match);
                const unsigned long long before = seen + block_exclusive_scan(cntm, sh);
                if (before < need && before + cntm >= need) {
                    uint32_t left = static_cast<uint32_t>(need - before);   // 1-based rank inside `match`
                    uint32_t mm = match;
                    while (left > 1) {
                        mm &= mm - 1;
                        --left;
                    }
                    sh.bcast[0] = (static_cast<unsigned long long>(r0) << 32) | (j * VEC + (__ffs(mm) - 1));
                }
                seen += block_sum(cntm, sh);
            }
            __syncthreads();
            const unsigned long long boundary = sh.bcast[0];
            __syncthreads();
            return boundary;
        }
    }
    return limit;
}

// Gumbel-max score of one candidate, packed for a max-reduction: (order-encoded score << 32) |
// ~column, so that the larger score wins and equal scores go to the lower column.
template <int DTYPE>
__device__ __forceinline__ unsigned long long packed_score(const FilterArgs &a, uint32_t rowb, uint32_t col,
                                                           uint32_t code) {
    const uint32_t v = a.vocab_offset + col;
    const uint4 r = philox4x32_10(v >> 2, rowb, a.step_lo, a.step_hi, a.gkeys);
    const uint32_t k = v & 3u;
    const uint32_t y = k == 0 ? r.x : k == 1 ? r.y : k == 2 ? r.z : r.w;
    const float sc = __fmaf_rn(value_of_code<DTYPE>(code), a.inv_tau, gumbel_of_word(y));
    const uint32_t sb = __float_as_uint(sc);
    const uint32_t enc = (sb & 0x80000000u) ? ~sb : (sb | 0x80000000u);
    return (static_cast<unsigned long long>(enc) << 32) | (0xFFFFFFFFu - col);
}

// ---------------------------------------------------------------------------------------------
// The head of a row's order, in shared memory.  Two passes over the CTA's part of the row: pass A
// finds every thread's largest code; the r-th largest of those maxima is a floor that at least r
// columns reach; pass B gathers every column at or above the floor as (key_m - code) << 32 | column
// (and, when asked, adds up the weights of the part).  In a cluster (CS > 1) every CTA does this on
// its own CS-th of the row with ceil(r / CS) in place of r -- the smallest of the local floors is
// reached by r columns of the row -- the maxima and floors travel through distributed shared
// memory, and CTA 0 pulls the other lists and weight sums.  All CTAs pass the same three cluster
// barriers whatever the data; the others then leave (`leave`), CTA 0 finishes the row alone.
// `slack` > 0 lowers the floor by that much (plus rounding room) in the logits' own units: the
// caller gathers unbiased logits and wants every column that a bias of at most `slack` could lift
// to the floor.  More than `cap` columns (at most kBigCap; kListCap when the weight table shares the
// space) at or above the floor are reported as cap + 1.
// ---------------------------------------------------------------------------------------------
constexpr int kDeepRank = 480;   // of the kFilterThreads thread maxima: about 1400 columns of an ordinary row

struct Head {
    uint32_t key_m;               // largest code of the row
    unsigned gathered;            // entries in sh.list (unsorted), or kListCap + 1
    unsigned long long z_all;     // total weight of the row (want_z)
    uint32_t deep_floor;          // a lower floor (the 480th largest thread maximum) for one retry
    uint32_t last_floor;          // a still lower floor (about kLastColumns columns) for the last retry
    bool leave;
};

template <int DTYPE, int CS>
__device__ __forceinline__ Head gather_head(const FilterArgs &a, FilterShared &sh, const char *src_row, unsigned part,
                                            int want, float slack, bool want_z, unsigned cap) {
    namespace cg = cooperative_groups;
    const uint32_t V = static_cast<uint32_t>(a.V);
    const uint32_t nvec = vectors_of<DTYPE>(V);
    const uint32_t vec_lo = static_cast<uint32_t>(static_cast<uint64_t>(nvec) * part / CS);
    const uint32_t vec_hi = static_cast<uint32_t>(static_cast<uint64_t>(nvec) * (part + 1) / CS);
    Head h;
    h.leave = false;
    // pass A: per-thread maxima, sorted descending (as ~code ascending) in the list area
    uint32_t my_max = 0u;
    for_each_vector<DTYPE>(
        src_row, V, vec_lo, vec_hi,
        [&](uint32_t, const uint4 &w) { my_max = max(my_max, vector_max_code<DTYPE>(w)); },
        [&](uint32_t, uint32_t code) { my_max = max(my_max, code); });
    __syncthreads();
    sh.list[threadIdx.x] = static_cast<unsigned long long>(~my_max);
    if (threadIdx.x == 0) sh.list_n = 0u;
    __syncthreads();
    sort_list(sh.list, kFilterThreads);
    uint32_t key_m = ~static_cast<uint32_t>(sh.list[0]);
    uint32_t floor_code = ~static_cast<uint32_t>(sh.list[(want + CS - 1) / CS - 1]);
    uint32_t deep_floor = ~static_cast<uint32_t>(sh.list[(kDeepRank + CS - 1) / CS - 1]);
    // the floor of the last retry: the thread maximum of the rank that about kLastColumns columns of
    // an ordinary row reach (a thread of this CTA sees V / (CS kFilterThreads) columns)
    const float per_thread = fmaxf(static_cast<float>(V) / static_cast<float>(CS * kFilterThreads), 1.0f);
    const float reach = fminf(static_cast<float>(kLastColumns) / static_cast<float>(V), 0.5f);
    const int last_rank = min(max(static_cast<int>(kFilterThreads * (1.0f - __powf(1.0f - reach, per_thread))), 1),
                              static_cast<int>(kFilterThreads));
    uint32_t last_floor = ~static_cast<uint32_t>(sh.list[last_rank - 1]);
    __syncthreads();
    if constexpr (CS > 1) {
        if (threadIdx.x == 0) {
            sh.part_max = key_m;
            sh.part_floor = floor_code;
            sh.part_deep = deep_floor;
            sh.part_last = last_floor;
        }
        cg::this_cluster().sync();
        for (unsigned r = 0; r < CS; ++r) {
            const FilterShared *other = cg::this_cluster().map_shared_rank(&sh, r);
            key_m = max(key_m, other->part_max);
            floor_code = min(floor_code, other->part_floor);
            deep_floor = min(deep_floor, other->part_deep);
            last_floor = min(last_floor, other->part_last);
        }
    }
    h.key_m = key_m;
    h.deep_floor = deep_floor;
    h.last_floor = last_floor;
    if (slack > 0.0f) {
        const float fl = value_of_code<DTYPE>(floor_code);
        if (fl == fl && fabsf(fl) != __int_as_float(0x7f800000)) {
            // room for the rounding of the biased sum (it may round up to the floor) and of this
            // subtraction: a few units in the last place of the logits' type
            const float eps = DTYPE == SBW_DTYPE_F32 ? 0x1p-20f : 0x1p-5f;
            const float t = __fsub_rn(__fsub_rn(fl, slack), __fmul_rn(__fadd_rn(fabsf(fl), slack), eps));
            const uint32_t c = code_of_bits<DTYPE>(__float_as_uint(t));
            floor_code = min(floor_code, c > 0u ? c - 1u : 0u);
        } else {
            floor_code = 0u;                          // no arithmetic on such a floor: gather all, overflow
        }
    }
    const float m = value_of_code<DTYPE>(key_m);
    // columns with a weight lie within 41 / c of the maximum: code_lo is below all of them
    uint32_t code_lo = key_m;
    if (m == m && fabsf(m) != __int_as_float(0x7f800000))
        code_lo = code_of_bits<DTYPE>(__float_as_uint(__fsub_rn(m, __fdiv_rn(42.0f, a.c))));

    // pass B
    unsigned long long z_local = 0;
    const int32_t floor_key = key_of_code<DTYPE>(floor_code), lo_key = key_of_code<DTYPE>(code_lo);
    if (want_z && DTYPE == SBW_DTYPE_BF16) {
        // A bf16 logit is one of 65536 codes and its weight is a function of the code alone: the
        // weights of the codes that occur in numbers -- the ten binades below the maximum and the
        // ten above the lowest code with a weight -- are computed once per row, the pass looks them
        // up, and only a logit outside both windows (tiny magnitudes) is evaluated on the spot.
        for (int i = threadIdx.x; i < 2 * kWeightTab; i += kFilterThreads) {
            const bool upper = i < kWeightTab;
            const uint32_t code = upper ? key_m - static_cast<uint32_t>(i) : code_lo + static_cast<uint32_t>(i - kWeightTab);
            const bool valid = (upper ? static_cast<uint32_t>(i) <= key_m : code <= key_m) && code >= code_lo;
            sh.wtab[i] = valid ? nucleus_weight(value_of_code<DTYPE>(code), m, code == key_m, a.c) : 0ull;
        }
        if (threadIdx.x == 0) sh.wtab[2 * kWeightTab] = 0ull;
        __syncthreads();
        auto take = [&](uint32_t col, uint32_t code) {
            // one lookup without branches: the upper window, else the lower one, else the zero entry
            const uint32_t down = key_m - code, up = code - code_lo;
            const bool in_upper = down < static_cast<uint32_t>(kWeightTab);
            const bool in_lower = up < static_cast<uint32_t>(kWeightTab);
            const uint32_t slot = in_upper ? down : in_lower ? kWeightTab + up : 2u * kWeightTab;
            z_local += sh.wtab[slot];
            if (!in_upper && !in_lower && code >= code_lo)       // rare: between the windows
                z_local += nucleus_weight_rare(value_of_code<DTYPE>(code), m, a.c);
            if (code >= floor_code && *reinterpret_cast<volatile unsigned int *>(&sh.list_n) <= cap) {
                const unsigned idx = atomicAdd(&sh.list_n, 1u);
                if (idx < cap) sh.list_big[idx] = (static_cast<unsigned long long>(key_m - code) << 32) | col;
            }
        };
        for_each_vector<DTYPE>(
            src_row, V, vec_lo, vec_hi,
            [&](uint32_t col0, const uint4 &w) {
#pragma unroll
                for (int i = 0; i < 8; ++i) take(col0 + i, element_code<DTYPE>(w, i));
            },
            take);
    } else if (!want_z) {
        // gather only: one compare per vector, the elements only where it reaches the floor
        auto take = [&](uint32_t col, uint32_t code) {
            if (code >= floor_code && *reinterpret_cast<volatile unsigned int *>(&sh.list_n) <= cap) {
                const unsigned idx = atomicAdd(&sh.list_n, 1u);
                if (idx < cap) sh.list_big[idx] = (static_cast<unsigned long long>(key_m - code) << 32) | col;
            }
        };
        for_each_vector<DTYPE>(
            src_row, V, vec_lo, vec_hi,
            [&](uint32_t col0, const uint4 &w) {
                if (vector_max_code<DTYPE>(w) < floor_code) return;
#pragma unroll
                for (int i = 0; i < (DTYPE == SBW_DTYPE_F32 ? 4 : 8); ++i) take(col0 + i, element_code<DTYPE>(w, i));
            },
            take);
    } else
    for_each_key<DTYPE>(src_row, V, vec_lo, vec_hi, [&](uint32_t col, uint32_t bits, int32_t key) {
        if (want_z && key >= lo_key)
            z_local += nucleus_weight(__uint_as_float(bits), m, code_of_key<DTYPE>(key) == key_m, a.c);
        if (key >= floor_key && *reinterpret_cast<volatile unsigned int *>(&sh.list_n) <= cap) {
            const unsigned idx = atomicAdd(&sh.list_n, 1u);
            if (idx < cap)
                sh.list_big[idx] = (static_cast<unsigned long long>(key_m - code_of_key<DTYPE>(key)) << 32) | col;
        }
    });
    h.z_all = want_z ? block_sum(z_local, sh) : 0ull;
    __syncthreads();
    unsigned gathered = sh.list_n;
    if constexpr (CS > 1) {
        if (threadIdx.x == 0) sh.part_z = h.z_all;
        cg::this_cluster().sync();
        if (part == 0) {
            for (unsigned r = 1; r < CS; ++r) {
                const FilterShared *other = cg::this_cluster().map_shared_rank(&sh, r);
                const unsigned n_r = other->list_n;
                if (gathered <= cap && n_r <= cap && gathered + n_r <= cap)
                    for (unsigned i = threadIdx.x; i < n_r; i += kFilterThreads) sh.list_big[gathered + i] = other->list_big[i];
                gathered = (gathered > cap || n_r > cap) ? cap + 1 : gathered + n_r;
                h.z_all += other->part_z;
            }
        }
        cg::this_cluster().sync();                   // the other CTAs' shared memory has been read
        h.leave = part != 0;
        __syncthreads();
    }
    h.gathered = gathered > cap ? cap + 1 : gathered;
    return h;
}

// sh.list[0 .. n) holds composites relative to key_m, unsorted.  Sorts them and applies the
// top-k cut and the top-p crossing; returns the number of kept candidates (a prefix of the sorted
// list), or 0 when the list does not reach far enough down the order.
template <int DTYPE, int CAP = kListCap>
__device__ __forceinline__ int cut_list(const FilterArgs &a, FilterShared &sh, unsigned long long *list, int n, uint32_t key_m, bool use_k,
                                        bool use_p, unsigned long long z_all) {
    constexpr int kPer = CAP / kFilterThreads;
    const float m = value_of_code<DTYPE>(key_m);
    int len = 2;
    while (len < n) len <<= 1;
    __syncthreads();
    for (int i = n + threadIdx.x; i < len; i += kFilterThreads) list[i] = kAll;
    __syncthreads();
    sort_list(list, len);
    int n1 = n;
    if (use_k) {
        if (a.top_k > n) return 0;
        n1 = static_cast<int>(a.top_k);
    }
    if (!use_p) return n1;
    unsigned long long w[kPer], mine = 0;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const int idx = threadIdx.x * kPer + i;
        const uint32_t dist = static_cast<uint32_t>(list[idx < len ? idx : 0] >> 32);
        w[i] = idx < n1 ? nucleus_weight(value_of_code<DTYPE>(key_m - dist), m, dist == 0u, a.c) : 0ull;
        mine += w[i];
    }
    const unsigned long long in_list = block_sum(mine, sh);
    const unsigned long long Z = use_k ? in_list : z_all;
    const unsigned long long lo = a.p32 * Z, hi = __umul64hi(a.p32, Z);
    unsigned long long target = (hi << 32) | (lo >> 32);
    if (lo & 0xffffffffull) target += 1;
    if (threadIdx.x == 0) sh.bcast[0] = kAll;
    unsigned long long at = block_exclusive_scan(mine, sh);
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        if (at < target && at + w[i] >= target) sh.bcast[0] = threadIdx.x * kPer + i;
        at += w[i];
    }
    __syncthreads();
    const unsigned long long cross = sh.bcast[0];
    __syncthreads();
    return cross == kAll ? 0 : static_cast<int>(cross) + 1;     // 0: the nucleus reaches below the floor
}

// Arg max of the packed scores over the CTA and the row's outputs.
__device__ __forceinline__ void finish_row(const FilterArgs &a, FilterShared &sh, int64_t row, unsigned long long best,
                                           unsigned long long kept) {
    for (int d = 16; d > 0; d >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xffffffffu, best, d);
        best = o > best ? o : best;
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh.red[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long top = 0;
        for (int w = 0; w < kFilterWarps; ++w) top = sh.red[w] > top ? sh.red[w] : top;
        a.out_tokens[row] = static_cast<int32_t>(0xFFFFFFFFu - static_cast<uint32_t>(top));
    }
    const unsigned long long total = block_sum(kept, sh);
    if (threadIdx.x == 0 && a.out_kept) a.out_kept[row] = static_cast<int32_t>(total);
    __syncthreads();
}

// Draws the sample from the first n2 entries of the sorted list.
template <int DTYPE>
__device__ __forceinline__ void sample_list(const FilterArgs &a, FilterShared &sh, const unsigned long long *list, int64_t row, uint32_t key_m, int n2) {
    unsigned long long best = 0;
    for (int i = threadIdx.x; i < n2; i += kFilterThreads) {
        const unsigned long long comp = list[i];
        const unsigned long long cand = packed_score<DTYPE>(a, static_cast<uint32_t>(row), static_cast<uint32_t>(comp),
                                                            key_m - static_cast<uint32_t>(comp >> 32));
        best = cand > best ? cand : best;
    }
    finish_row(a, sh, row, best, threadIdx.x == 0 ? n2 : 0);
}

// The general path on a biased row: list if it reaches far enough, else the radix descent and one
// more pass over the row.
template <int DTYPE, int CS>
__device__ __forceinline__ bool full_row(const FilterArgs &a, FilterShared &sh, int64_t row, unsigned part) {
    constexpr int ESIZE = DTYPE == SBW_DTYPE_F32 ? 4 : 2;
    constexpr int kCodeBits = DTYPE == SBW_DTYPE_F32 ? 32 : 16;
    const uint32_t V = static_cast<uint32_t>(a.V);
    const bool use_k = a.top_k > 0 && a.top_k < a.V;
    const bool use_p = a.p32 != 0ull;
    const char *row_ptr = static_cast<const char *>(a.biased) + row * a.ld * ESIZE;
    const int want = use_k ? static_cast<int>(min(a.top_k, static_cast<int64_t>(kFilterThreads))) : 384;
    const Head h = gather_head<DTYPE, CS>(a, sh, row_ptr, part, want, 0.0f, use_p && !use_k, kListCap);
    if (h.leave) return false;
    const uint32_t key_m = h.key_m;
    int n2 = 0;
    if ((use_k || use_p) && h.gathered <= kListCap)
        n2 = cut_list<DTYPE>(a, sh, sh.list, static_cast<int>(h.gathered), key_m, use_k, use_p, h.z_all);
    const unsigned long long *kept_list = sh.list;
    if (n2 == 0 && use_p && !use_k && h.gathered <= kListCap) {
        // The nucleus reaches below the floor.  Before the radix descent, which costs several passes
        // on one CTA, gather again with a lower floor: the 480th largest thread maximum (about
        // three times as many columns), then one that about kLastColumns columns reach, with a
        // list of twice the size.
        auto regather = [&](uint32_t floor_code, unsigned long long *list, unsigned cap) -> unsigned {
            __syncthreads();
            if (threadIdx.x == 0) sh.list_n = 0u;
            __syncthreads();
            auto take = [&](uint32_t col, uint32_t code) {
                if (code >= floor_code && *reinterpret_cast<volatile unsigned int *>(&sh.list_n) <= cap) {
                    const unsigned idx = atomicAdd(&sh.list_n, 1u);
                    if (idx < cap) list[idx] = (static_cast<unsigned long long>(key_m - code) << 32) | col;
                }
            };
            for_each_vector<DTYPE>(
                row_ptr, V, 0u, vectors_of<DTYPE>(V),
                [&](uint32_t col0, const uint4 &w) {
                    if (vector_max_code<DTYPE>(w) < floor_code) return;
#pragma unroll
                    for (int i = 0; i < (DTYPE == SBW_DTYPE_F32 ? 4 : 8); ++i) take(col0 + i, element_code<DTYPE>(w, i));
                },
                take);
            __syncthreads();
            return sh.list_n;
        };
        unsigned again = kListCap + 1u;
        if (h.deep_floor < key_m) {
            again = regather(h.deep_floor, sh.list, kListCap);
            if (again <= kListCap)
                n2 = cut_list<DTYPE>(a, sh, sh.list, static_cast<int>(again), key_m, false, true, h.z_all);
        }
        if (n2 == 0 && h.last_floor < h.deep_floor) {
            again = regather(h.last_floor, sh.list_big, kBigCap);
            if (again <= kBigCap) {
                n2 = cut_list<DTYPE, kBigCap>(a, sh, sh.list_big, static_cast<int>(again), key_m, false, true, h.z_all);
                kept_list = sh.list_big;
            }
        }
    }
    if (n2 > 0) {
        sample_list<DTYPE>(a, sh, kept_list, row, key_m, n2);
        return true;
    }
    __syncthreads();
    const float m = value_of_code<DTYPE>(key_m);
    unsigned long long boundary = kAll;
    if (use_k)
        boundary = select_boundary<DTYPE, kModeCount>(row_ptr, V, key_m, m, a.c, kAll,
                                                      static_cast<unsigned long long>(a.top_k), kCodeBits, sh);
    if (use_p) {
        uint32_t code_lo = key_m;
        if (m == m && fabsf(m) != __int_as_float(0x7f800000))
            code_lo = code_of_bits<DTYPE>(__float_as_uint(__fsub_rn(m, __fdiv_rn(42.0f, a.c))));
        const int s0 = 32 - __clz(key_m - code_lo);
        boundary = select_boundary<DTYPE, kModeMass>(row_ptr, V, key_m, m, a.c, boundary, a.p32, s0, sh);
    }
    unsigned long long best = 0, kept = 0;
    for_each<DTYPE>(row_ptr, V, [&](uint32_t col, uint32_t code) {
        const uint32_t dist = key_m - code;
        if (((static_cast<unsigned long long>(dist) << 32) | col) > boundary) return;
        kept += 1;
        const unsigned long long cand = packed_score<DTYPE>(a, static_cast<uint32_t>(row), col, code);
        best = cand > best ? cand : best;
    });
    finish_row(a, sh, row, best, kept);
    return true;
}

// Eq. 1 + Eq. 2 on one logit given as its code; returns the code of the biased logit.
template <int DTYPE>
__device__ __forceinline__ uint32_t biased_code(const FilterArgs &a, uint64_t r_row, uint32_t jmin, uint32_t col,
                                                uint32_t code) {
    const uint32_t v = a.vocab_offset + col;
    const uint64_t r = a.scheme == SBW_SCHEME_CONTEXT ? r_row : seed_selfsalt(a.key, jmin, v);
    if (a.delta == 0.0f || philox_word0(v, r, a.weyl) > a.thr_m1) return code;
    const float l = value_of_code<DTYPE>(code);
    if constexpr (DTYPE == SBW_DTYPE_F32) {
        return code_of_bits<DTYPE>(__float_as_uint(__fadd_rn(l, a.delta)));
    } else {
        // both operands are bf16 values: rounding their fp32 sum once more is the bf16 sum
        const __nv_bfloat16 s = __float2bfloat16_rn(__fadd_rn(l, a.delta));
        return code_of_bits<DTYPE>(static_cast<uint32_t>(__bfloat16_as_ushort(s)) << 16);
    }
}

// With top_k set, the kept candidates can be found without biasing the row.  Let f be the k-th
// largest unbiased logit.  At least k biased logits reach f - max(-delta, 0), so the k-th largest
// biased logit does too, and a column of the biased top-k, whose biased logit is at most
// l + max(delta, 0), has l >= f - |delta| (less the rounding of the sum).  Those columns -- a few
// hundred for ordinary rows -- are gathered from the unbiased row, hashed and biased in shared
// memory, and then cut and sampled like any list.  A row whose candidates do not fit the list is
// biased into the workspace by this CTA and takes the general path.
template <int DTYPE, int CS>
__device__ __forceinline__ bool candidate_row(const FilterArgs &a, FilterShared &sh, int64_t row, unsigned part) {
    constexpr int ESIZE = DTYPE == SBW_DTYPE_F32 ? 4 : 2;
    constexpr int VEC = DTYPE == SBW_DTYPE_F32 ? 4 : 8;
    const uint32_t V = static_cast<uint32_t>(a.V);
    const bool use_p = a.p32 != 0ull;
    const char *raw_row = static_cast<const char *>(a.raw) + row * a.ld_raw * ESIZE;
    const int want = static_cast<int>(min(a.top_k, static_cast<int64_t>(kFilterThreads)));
    // the unbiased candidates may be many when |delta| is large: the list of twice the size
    const Head h = gather_head<DTYPE, CS>(a, sh, raw_row, part, want, fmaxf(fabsf(a.delta), 0x1p-126f), false, kBigCap);
    if (h.leave) return false;
    const int32_t *ctx = a.ctx + row * a.W;
    const uint64_t r_row = a.scheme == SBW_SCHEME_CONTEXT ? seed_context(a.key, ctx, a.W) : 0ull;
    const uint32_t jmin = a.scheme == SBW_SCHEME_SELFSALT ? jenkins_min(ctx, a.W) : 0u;
    if (h.gathered <= kBigCap && static_cast<int64_t>(h.gathered) >= a.top_k) {
        const int n = static_cast<int>(h.gathered);
        unsigned long long *list = sh.list_big;
        // bias the candidates: entries become (biased code << 32 | column), then composites
        // relative to the largest biased code
        uint32_t top = 0;
        for (int i = threadIdx.x; i < n; i += kFilterThreads) {
            const unsigned long long e = list[i];
            const uint32_t col = static_cast<uint32_t>(e);
            const uint32_t code = biased_code<DTYPE>(a, r_row, jmin, col, h.key_m - static_cast<uint32_t>(e >> 32));
            list[i] = (static_cast<unsigned long long>(code) << 32) | col;
            top = max(top, code);
        }
        for (int d = 16; d > 0; d >>= 1) top = max(top, __shfl_xor_sync(0xffffffffu, top, d));
        __syncthreads();
        if ((threadIdx.x & 31) == 0) sh.red32[threadIdx.x >> 5] = top;
        __syncthreads();
        uint32_t key_m = 0;
        for (int w = 0; w < kFilterWarps; ++w) key_m = max(key_m, sh.red32[w]);
        for (int i = threadIdx.x; i < n; i += kFilterThreads) {
            const unsigned long long e = list[i];
            list[i] = (static_cast<unsigned long long>(key_m - static_cast<uint32_t>(e >> 32)) << 32) |
                         static_cast<uint32_t>(e);
        }
        const int n2 = cut_list<DTYPE, kBigCap>(a, sh, list, n, key_m, true, use_p, 0ull);
        if (n2 > 0) {
            sample_list<DTYPE>(a, sh, list, row, key_m, n2);
            return true;
        }
    }
    // the candidates do not fit: bias the whole row into the workspace, then the general path
    __syncthreads();
    char *dst_row = static_cast<char *>(const_cast<void *>(a.biased)) + row * a.ld * ESIZE;
    const uint32_t nvec = vectors_of<DTYPE>(V);
    for (uint32_t j = threadIdx.x; j < nvec; j += kFilterThreads) {
        uint4 w = reinterpret_cast<const uint4 *>(raw_row)[j];
        uint32_t *e = reinterpret_cast<uint32_t *>(&w);
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
            const uint32_t col = j * VEC + i;
            if (col >= V) continue;
            if constexpr (DTYPE == SBW_DTYPE_F32) {
                e[i] = order_decode(biased_code<DTYPE>(a, r_row, jmin, col, code_of_bits<DTYPE>(e[i])));
            } else {
                const uint32_t bits = (i & 1) ? (e[i >> 1] & 0xffff0000u) : (e[i >> 1] << 16);
                const float v = value_of_code<DTYPE>(biased_code<DTYPE>(a, r_row, jmin, col, code_of_bits<DTYPE>(bits)));
                const uint32_t b16 = __float_as_uint(v) >> 16;
                e[i >> 1] = (i & 1) ? ((e[i >> 1] & 0x0000ffffu) | (b16 << 16)) : ((e[i >> 1] & 0xffff0000u) | b16);
            }
        }
        reinterpret_cast<uint4 *>(dst_row)[j] = w;
    }
    __syncthreads();
    return full_row<DTYPE, 1>(a, sh, row, 0u);
}

// One CTA per row (CS = 1, a persistent grid walking the rows), or a cluster of CS CTAs per row
// for small batches.
template <int DTYPE, int CS>
__global__ void __launch_bounds__(kFilterThreads, 2)   // two CTAs per SM: the paths are latency-bound
filter_sample_kernel(const FilterArgs a) {
    __shared__ FilterShared sh;
    const unsigned part = CS > 1 ? blockIdx.x % CS : 0u;          // this CTA's part of the row
    const int64_t first_row = CS > 1 ? blockIdx.x / CS : blockIdx.x;
    const int64_t row_step = CS > 1 ? a.B : gridDim.x;            // a cluster handles exactly one row
    for (int64_t row = first_row; row < a.B; row += row_step) {
        const bool stay = a.raw ? candidate_row<DTYPE, CS>(a, sh, row, part) : full_row<DTYPE, CS>(a, sh, row, part);
        if (!stay) return;
    }
}

template <int DTYPE>
cudaError_t launch_cluster(const FilterArgs &a, int cs, cudaStream_t s) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(a.B * cs));
    cfg.blockDim = dim3(kFilterThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(cs);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    switch (cs) {
        case 8: return cudaLaunchKernelEx(&cfg, filter_sample_kernel<DTYPE, 8>, a);
        case 4: return cudaLaunchKernelEx(&cfg, filter_sample_kernel<DTYPE, 4>, a);
        default: return cudaLaunchKernelEx(&cfg, filter_sample_kernel<DTYPE, 2>, a);
    }
}

}  // namespace
}  // namespace sbw

extern "C" size_t sbw_sample_filtered_workspace_bytes(int dtype, int64_t B, int64_t V) {
    if (B <= 0 || V <= 0 || (dtype != SBW_DTYPE_F32 && dtype != SBW_DTYPE_BF16)) return 0;
    const size_t es = dtype == SBW_DTYPE_F32 ? 4 : 2;
    const size_t vp = sbw::align_up(static_cast<size_t>(V), 8);
    return sbw::align_up(static_cast<size_t>(B) * vp * es, 256);
}

extern "C" int sbw_bias_sample_filtered(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                                        int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width,
                                        uint64_t key, double gamma, float delta, int scheme, float temperature,
                                        int64_t top_k, double top_p, uint64_t rng_seed, uint64_t rng_step,
                                        int32_t *out_tokens, int32_t *out_kept, void *workspace,
                                        size_t workspace_bytes, void *stream) {
    using namespace sbw;
    if (!valid_common(dtype, ctx_width, gamma, scheme)) return SBW_ERR_INVALID_ARG;
    if (B < 0 || V < 1 || ld < V || vocab_offset < 0 || top_k < 0) return SBW_ERR_INVALID_ARG;
    if (!(temperature > 0.0f) || !(top_p > 0.0)) return SBW_ERR_INVALID_ARG;
    if (B == 0) return SBW_OK;
    if (!logits || !ctx_tokens || !out_tokens) return SBW_ERR_INVALID_ARG;
    if (V > kMaxFilterV || B > 0xffffffffLL) return SBW_ERR_UNSUPPORTED;
    const size_t need = sbw_sample_filtered_workspace_bytes(dtype, B, V);
    if (!workspace || workspace_bytes < need || reinterpret_cast<uintptr_t>(workspace) % 256 != 0)
        return SBW_ERR_WORKSPACE;
    DeviceInfo di;
    if (int rc = current_device_info(&di)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t es = dtype == SBW_DTYPE_F32 ? 4 : 2;
    const int64_t vp = static_cast<int64_t>(align_up(static_cast<size_t>(V), 8));

    // With top_k set and 16-byte aligned rows the kernel works on the unbiased rows (candidate
    // path) and no bias pass is launched.  Otherwise l' of Eq. 2, in the logits' precision, goes
    // into the workspace first: one out-of-place pass of the bias kernel when the rows are aligned,
    // else a row copy and the in-place kernel.
    const bool candidates = top_k > 0 && top_k < V && reinterpret_cast<uintptr_t>(logits) % 16 == 0 &&
                            (ld * es) % 16 == 0 && vocab_offset + V <= (int64_t(1) << 32) &&
                            delta == delta && delta - delta == 0.0f;
    if (!candidates) {
        bool fused = false;
        if (int rc = bias_copy_impl(logits, ld, workspace, dtype, B, V, vp, vocab_offset, ctx_tokens, ctx_width, key,
                                    gamma, delta, scheme, s, &fused))
            return rc;
        if (!fused) {
            SBW_CUDA_TRY(cudaMemcpy2DAsync(workspace, vp * es, logits, ld * es, V * es, B, cudaMemcpyDeviceToDevice, s));
            if (int rc = bias_logits_impl(workspace, dtype, B, V, vp, vocab_offset, ctx_tokens, ctx_width, key, gamma,
                                          delta, scheme, s))
                return rc;
        }
    }

    FilterArgs a;
    a.biased = workspace;
    a.B = B;
    a.V = V;
    a.ld = vp;
    a.vocab_offset = static_cast<uint32_t>(vocab_offset);
    a.inv_tau = 1.0f / temperature;
    a.c = static_cast<float>(1.4426950408889634 / static_cast<double>(temperature));
    a.top_k = top_k;
    a.p32 = 0;
    if (top_p < 1.0) {
        const double scaled = std::floor(top_p * 4294967296.0);
        a.p32 = scaled < 1.0 ? 1ull : static_cast<uint64_t>(scaled);
    }
    a.step_lo = static_cast<uint32_t>(rng_step);
    a.step_hi = static_cast<uint32_t>(rng_step >> 32);
    a.gkeys = make_block_keys(static_cast<uint32_t>(rng_seed), static_cast<uint32_t>(rng_seed >> 32));
    a.out_tokens = out_tokens;
    a.out_kept = out_kept;
    a.raw = candidates ? logits : nullptr;
    a.ld_raw = ld;
    a.ctx = ctx_tokens;
    a.W = ctx_width;
    a.scheme = scheme;
    a.key = key;
    a.thr_m1 = threshold_minus_one(gamma);
    a.delta = dtype == SBW_DTYPE_BF16 ? __bfloat162float(__float2bfloat16_rn(delta)) : delta;
    a.weyl = make_weyl();
    // small batches: a cluster of CTAs per row, as many as keeps every SM busy with two CTAs
    const int64_t cap = 2LL * di.sm_count;
    const int cs = B * 8 <= cap ? 8 : B * 4 <= cap ? 4 : B * 2 <= cap ? 2 : 1;
    if (cs == 1) {
        const unsigned grid = static_cast<unsigned>(B < cap ? B : cap);
        if (dtype == SBW_DTYPE_F32) filter_sample_kernel<SBW_DTYPE_F32, 1><<<grid, kFilterThreads, 0, s>>>(a);
        else filter_sample_kernel<SBW_DTYPE_BF16, 1><<<grid, kFilterThreads, 0, s>>>(a);
    } else {
        SBW_CUDA_TRY(dtype == SBW_DTYPE_F32 ? launch_cluster<SBW_DTYPE_F32>(a, cs, s)
                                            : launch_cluster<SBW_DTYPE_BF16>(a, cs, s));
    }
    SBW_CUDA_TRY(cudaGetLastError());
    return SBW_OK;
}
