// sbw_bias_logits_topk: the paper's SBW-ss scheme (Table 1: Bernoulli list, self-salt seeding,
// candidates "top-40") -- per row only the k largest logits are tested and biased, as KGW's
// selfhash does; everything else in the row is left alone.
//
// One CTA per row.  "Largest" is the total order on order-encoded bit patterns with ties to the
// lowest column, expressed as one 64-bit composite (code << 32 | ~column).
//   1. A pass over a prefix of the row (its first 128 KB): every thread keeps the largest code
//      it has seen; groups of four threads give 256 maxima of disjoint column sets.  Their k-th
//      largest value L is a lower bound of the row's k-th largest logit (k distinct columns reach
//      it), and it is known after a fifth (fp32, V = 151936) to a half (bf16, V = 128256) of the row.
//   2. One pass over the whole row: columns with code >= L -- a few hundred for ordinary logits --
//      go into a shared-memory candidate list.  The common path is one compare per 16-byte vector.
//   3. Candidates are ranked by counting larger composites; ranks below k are hashed and biased.
// If the list overflows (rows of equal values, k > 256) the CTA falls back to k rounds of "largest
// composite below the previous one", a block reduction each, and one pass that biases every
// column at or above the k-th composite: slow, but it needs no assumption about the data.
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include "sbw_codes.cuh"
#include "sbw_common.cuh"
#include "sbw_hash.cuh"

namespace sbw {

int bias_logits_impl(void *logits, int dtype, int64_t B, int64_t V, int64_t ld, int64_t vocab_offset,
                     const int32_t *ctx_tokens, int ctx_width, uint64_t key, double gamma, float delta,
                     int scheme, cudaStream_t stream);

namespace {

// CTA size: 1024 threads (one CTA per SM) when there are fewer rows than SMs can take two of,
// 512 threads (two CTAs per SM, twice the rows in flight) for larger batches.
constexpr int kCap = 2048;                  // candidate list entries
constexpr int kHitCap = 2048;                // vectors noted by the gather pass for a closer look
constexpr int kPrefixBytes = 131072;         // leading part of the row read by the pass that finds the bound

struct TopkArgs {
    void *logits;
    int64_t B, V, ld;
    const int32_t *ctx;
    int W;
    uint32_t vocab_offset;
    uint64_t key;
    uint32_t thr_m1;
    float delta;       // in the logits' precision, widened
    Weyl weyl;
    int k;
    bool vector;       // rows start on 16-byte boundaries
};

__device__ __forceinline__ uint64_t composite(uint32_t code, uint32_t col) {
    return (static_cast<uint64_t>(code) << 32) | (0xFFFFFFFFu - col);
}

// Calls f(column, code) for the columns [begin, end) of one row that this thread owns; begin is a
// multiple of 8 columns.
template <int DTYPE, int kTopkThreads, typename F>
__device__ __forceinline__ void for_each_code(const char *row_ptr, uint32_t begin, uint32_t end, bool vector, F f) {
    constexpr int VEC = DTYPE == SBW_DTYPE_F32 ? 4 : 8;
    uint32_t done = begin;
    if (vector) {
        const uint32_t nfull = end / VEC;
        constexpr int kInFlight = 4;   // independent 128-bit loads per thread before the first use
        for (uint32_t j0 = begin / VEC + threadIdx.x; j0 < nfull; j0 += kInFlight * kTopkThreads) {
            uint4 w[kInFlight];
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) {
                const uint32_t j = j0 + u * kTopkThreads;
                // plain loads: the row is written later by this kernel
                w[u] = j < nfull ? reinterpret_cast<const uint4 *>(row_ptr)[j] : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) {
                const uint32_t j = j0 + u * kTopkThreads;
                if (j >= nfull) break;
                const uint32_t *e = reinterpret_cast<const uint32_t *>(&w[u]);
#pragma unroll
                for (int i = 0; i < VEC; ++i) {
                    uint32_t bits;
                    if constexpr (DTYPE == SBW_DTYPE_F32) bits = e[i];
                    else bits = (i & 1) ? (e[i >> 1] & 0xffff0000u) : (e[i >> 1] << 16);
                    f(j * VEC + i, order_code(bits));
                }
            }
        }
        done = max(begin, nfull * VEC);
    }
    for (uint32_t c = done + threadIdx.x; c < end; c += kTopkThreads) {
        uint32_t bits;
        if constexpr (DTYPE == SBW_DTYPE_F32) bits = reinterpret_cast<const uint32_t *>(row_ptr)[c];
        else bits = static_cast<uint32_t>(reinterpret_cast<const uint16_t *>(row_ptr)[c]) << 16;
        f(c, order_code(bits));
    }
}

// Calls fvec(first column, vector) for the aligned 16-byte vectors of the columns [begin, end) that
// this thread owns and fone(column, code) for the columns left over (all of them when the rows
// are not aligned); begin is a multiple of 8 columns.
template <int DTYPE, int kTopkThreads, int kInFlight = 8, typename FV, typename F1>
__device__ __forceinline__ void for_each_vector(const char *row_ptr, uint32_t begin, uint32_t end, bool vector,
                                                FV fvec, F1 fone) {
    constexpr int VEC = DTYPE == SBW_DTYPE_F32 ? 4 : 8;
    uint32_t done = begin;
    if (vector) {
        const uint32_t nfull = end / VEC;
        // kInFlight independent 128-bit loads per thread before the first use
        for (uint32_t j0 = begin / VEC + threadIdx.x; j0 < nfull; j0 += kInFlight * kTopkThreads) {
            uint4 w[kInFlight];
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) {
                const uint32_t j = j0 + u * kTopkThreads;
                // plain loads: the row is written later by this kernel
                w[u] = j < nfull ? reinterpret_cast<const uint4 *>(row_ptr)[j] : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < kInFlight; ++u) {
                const uint32_t j = j0 + u * kTopkThreads;
                if (j < nfull) fvec(j * VEC, w[u]);
            }
        }
        done = max(begin, nfull * VEC);
    }
    for (uint32_t c = done + threadIdx.x; c < end; c += kTopkThreads) fone(c, scalar_code<DTYPE>(row_ptr, c));
}

// What the green test of a row needs from its context tokens: the seed itself (context scheme) or
// the smallest context hash (self-salt).  Read when the row is started, so that the tokens'
// latency hides behind the row's first loads.
template <int SCHEME>
__device__ __forceinline__ uint64_t row_seed_material(const TopkArgs &a, int64_t row) {
    const int32_t *ctx = a.ctx + row * a.W;
    if constexpr (SCHEME == SBW_SCHEME_CONTEXT) return seed_context(a.key, ctx, a.W);
    else return jenkins_min(ctx, a.W);
}

// Eq. 1 + Eq. 2 on one chosen column whose order code is known: the value is rebuilt from the
// code (no second read of the logit) and stored only if the column is green.
template <int DTYPE, int SCHEME>
__device__ __noinline__ void bias_column(const TopkArgs &a, uint64_t material, char *row_ptr, uint32_t col, uint32_t code) {
    const uint32_t v = a.vocab_offset + col;
    uint64_t r;
    if constexpr (SCHEME == SBW_SCHEME_CONTEXT) r = material;
    else r = seed_selfsalt(a.key, static_cast<uint32_t>(material), v);
    if (philox_word0(v, r, a.weyl) > a.thr_m1) return;
    if constexpr (DTYPE == SBW_DTYPE_F32) {
        reinterpret_cast<float *>(row_ptr)[col] = __fadd_rn(__uint_as_float(order_decode(code)), a.delta);
    } else {
        const uint32_t bits = (code & 0x8000u) ? (code ^ 0x8000u) : (code ^ 0xffffu);
        reinterpret_cast<__nv_bfloat16 *>(row_ptr)[col] =
            __float2bfloat16_rn(__fadd_rn(__uint_as_float(bits << 16), a.delta));
    }
}

template <int kTopkWarps>
__device__ __forceinline__ uint64_t block_max_u64(uint64_t x, uint64_t *sh_red, uint64_t *sh_out) {
    for (int d = 16; d > 0; d >>= 1) {
        const uint64_t o = __shfl_xor_sync(0xffffffffu, x, d);
        x = o > x ? o : x;
    }
    if ((threadIdx.x & 31) == 0) sh_red[threadIdx.x >> 5] = x;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint64_t m = sh_red[0];
        for (int w = 1; w < kTopkWarps; ++w) m = sh_red[w] > m ? sh_red[w] : m;
        *sh_out = m;
    }
    __syncthreads();
    return *sh_out;
}

// CS = 1: one CTA per row.  CS > 1 (small batches): a thread-block cluster per row; every CTA runs
// steps 1 and 2 on its CS-th of the row with ceil(k / CS) in place of k (the smallest of the local
// bounds is then reached by at least k columns of the row), the bounds travel through distributed
// shared memory, CTA 0 pulls the other candidate lists and does step 3 (or the fallback) alone.
// Every CTA passes the same three cluster barriers; nothing spins.
template <int DTYPE, int SCHEME, int kTopkThreads, int CS>
__global__ void __launch_bounds__(kTopkThreads)
topk_kernel(const TopkArgs a) {
    constexpr int ESIZE = DTYPE == SBW_DTYPE_F32 ? 4 : 2;
    constexpr int kTopkWarps = kTopkThreads / 32;
    constexpr int kGroups = kTopkThreads / 4;   // maxima of disjoint column sets used for the lower bound
    __shared__ uint32_t sh_max[kGroups];
    __shared__ __align__(16) uint64_t sh_cand[kCap + 2];
    __shared__ __align__(16) uint64_t sh_keep[kCap + 2];
    __shared__ uint32_t sh_hitvec[kHitCap];
    __shared__ unsigned sh_nhit;
    __shared__ unsigned sh_hist[256];
    __shared__ unsigned sh_kept, sh_cut;
    __shared__ uint64_t sh_red[kTopkWarps];
    __shared__ uint64_t sh_best;
    __shared__ uint32_t sh_floor, sh_top;
    __shared__ unsigned sh_count;
    namespace cg = cooperative_groups;
    const uint32_t V = static_cast<uint32_t>(a.V);
    const uint32_t k = static_cast<uint32_t>(a.k);
    const uint32_t k_part = (k + CS - 1) / CS;
    const unsigned part = CS > 1 ? blockIdx.x % CS : 0u;
    const int64_t first_row = CS > 1 ? blockIdx.x / CS : blockIdx.x;
    const int64_t row_step = CS > 1 ? a.B : gridDim.x;           // a cluster handles exactly one row
    // this CTA's columns; part boundaries are multiples of 8 columns
    const uint32_t c_lo = CS > 1 ? static_cast<uint32_t>(static_cast<uint64_t>(V) * part / CS) & ~7u : 0u;
    const uint32_t c_hi = CS > 1 && part + 1 < CS ? static_cast<uint32_t>(static_cast<uint64_t>(V) * (part + 1) / CS) & ~7u : V;

    for (int64_t row = first_row; row < a.B; row += row_step) {
        char *row_ptr = static_cast<char *>(a.logits) + row * a.ld * ESIZE;
        const uint64_t material = row_seed_material<SCHEME>(a, row);

        // 1. lower bound of the k-th largest code from a prefix of the columns
        const uint32_t prefix_end = min(c_hi, c_lo + static_cast<uint32_t>(kPrefixBytes / ESIZE / CS));
        uint32_t mx = 0;
        for_each_vector<DTYPE, kTopkThreads>(
            row_ptr, c_lo, prefix_end, a.vector,
            [&](uint32_t, const uint4 &w) { mx = max(mx, vector_max_code<DTYPE>(w)); },
            [&](uint32_t, uint32_t code) { mx = max(mx, code); });
        mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        if ((threadIdx.x & 3) == 0) sh_max[threadIdx.x >> 2] = mx;
        if (threadIdx.x == 0) {
            sh_floor = 0;            // k_part > kGroups: no bound, everything is a candidate
            sh_top = 0xffffffffu;    // and no largest prefix code either
            sh_count = 0;
            sh_nhit = 0;
        }
        __syncthreads();
        if (k_part <= kGroups && threadIdx.x < kGroups) {
            const uint32_t mine = sh_max[threadIdx.x];
            uint32_t rank = 0;
            for (int u = 0; u < kGroups; ++u) {
                const uint32_t o = sh_max[u];
                rank += (o > mine || (o == mine && u < static_cast<int>(threadIdx.x))) ? 1u : 0u;
            }
            if (rank == k_part - 1) sh_floor = mine;
            if (rank == 0) sh_top = mine;            // the largest code of the prefix
        }
        __syncthreads();
        uint32_t floor_code = sh_floor;
        if constexpr (CS > 1) {
            cg::this_cluster().sync();
            for (unsigned r = 0; r < CS; ++r)
                floor_code = min(floor_code, *cg::this_cluster().map_shared_rank(&sh_floor, r));
        }

        // 2. candidates: every column that reaches the bound
        auto push = [&](uint32_t col, uint32_t code) {
            if (code >= floor_code) {
                const unsigned pos = atomicAdd(&sh_count, 1u);
                if (pos < kCap) sh_cand[pos] = composite(code, col);
            }
        };
        // bf16 (eight logits per vector): a vector that reaches the bound is only noted here (the
        // common case is one compare per vector, the rare one an atomic add and a store) and its
        // logits are looked at afterwards by one thread each, so that no warp walks a vector's
        // elements with a single lane active.  fp32 (four logits) looks at them on the spot: the
        // extra barrier and the second read cost more than they save there.
        if constexpr (DTYPE == SBW_DTYPE_BF16) {
            for_each_vector<DTYPE, kTopkThreads>(
                row_ptr, c_lo, c_hi, a.vector,
                [&](uint32_t col0, const uint4 &w) {
                    if (vector_max_code<DTYPE>(w) < floor_code) return;
                    const unsigned pos = atomicAdd(&sh_nhit, 1u);
                    if (pos < static_cast<unsigned>(kHitCap)) sh_hitvec[pos] = col0;
                },
                push);
            __syncthreads();
            constexpr unsigned kVec = 16 / ESIZE;
            const unsigned nhit = sh_nhit;
            if (nhit <= static_cast<unsigned>(kHitCap)) {
                for (unsigned t = threadIdx.x; t < nhit * kVec; t += kTopkThreads) {
                    const uint32_t col = sh_hitvec[t / kVec] + t % kVec;
                    push(col, scalar_code<DTYPE>(row_ptr, col));
                }
            } else if (threadIdx.x == 0) {
                sh_count = kCap + 1;             // too many to note: the exact fallback takes the row
            }
        } else {
            // ten loads in flight fit the 64 registers that two 512-thread CTAs per SM leave a thread
            // (the cluster variants would spill); bf16, with more work per vector, is faster with eight
            for_each_vector<DTYPE, kTopkThreads, (CS == 1 ? 10 : 8)>(
                row_ptr, c_lo, c_hi, a.vector,
                [&](uint32_t col0, const uint4 &w) {
                    if (vector_max_code<DTYPE>(w) < floor_code) return;   // the common case: one compare per vector
#pragma unroll
                    for (int i = 0; i < 16 / ESIZE; ++i) push(col0 + i, element_code<DTYPE>(w, i));
                },
                push);
        }
        __syncthreads();
        unsigned n = sh_count;
        if constexpr (CS > 1) {
            cg::this_cluster().sync();
            if (part == 0) {
                for (unsigned r = 1; r < CS; ++r) {
                    const unsigned n_r = *cg::this_cluster().map_shared_rank(&sh_count, r);
                    if (n <= kCap && n_r <= kCap && n + n_r <= kCap) {
                        const uint64_t *other = cg::this_cluster().map_shared_rank(&sh_cand[0], r);
                        for (unsigned i = threadIdx.x; i < n_r; i += kTopkThreads) sh_cand[n + i] = other[i];
                    }
                    n = (n > kCap || n_r > kCap) ? kCap + 1 : n + n_r;
                }
            }
            cg::this_cluster().sync();               // the other CTAs' shared memory has been read
            if (part != 0) return;
            __syncthreads();
        }

        if (n <= kCap) {
            uint64_t *list = sh_cand;
            if (n > 2 * k + 64) {
                // Counting costs n^2, so a long list is cut first: a histogram of the codes over
                // [bound, largest code of the prefix] in 256 bins of equal width; the bin in which the count from
                // the top reaches k holds the k-th largest code, and everything in a lower bin has
                // k larger codes above it.
                if (threadIdx.x < 256) sh_hist[threadIdx.x] = 0;
                if (threadIdx.x == 0) {
                    sh_kept = 0;
                    sh_cut = 0;
                }
                __syncthreads();                                  // the histogram is clear
                // bins over [bound, largest code of the prefix]; codes above that share the top bin
                const uint32_t top = sh_top > floor_code ? sh_top : floor_code;
                const uint32_t span = top - floor_code;
                const int shift = span < 256u ? 0 : 32 - __clz(span) - 8;
                auto bin_of = [&](uint64_t e) -> unsigned {
                    const uint32_t b = (static_cast<uint32_t>(e >> 32) - floor_code) >> shift;
                    return b < 255u ? b : 255u;
                };
                for (unsigned i = threadIdx.x; i < n; i += kTopkThreads) atomicAdd(&sh_hist[bin_of(sh_cand[i])], 1u);
                __syncthreads();
                if (threadIdx.x < 32) {
                    unsigned mine = 0;                            // entries in this lane's 8 bins
                    for (int b = 0; b < 8; ++b) mine += sh_hist[threadIdx.x * 8 + b];
                    unsigned above = mine;                        // entries in this lane's bins and all higher ones
                    for (int d = 1; d < 32; d <<= 1) {
                        const unsigned o = __shfl_down_sync(0xffffffffu, above, d);
                        if (threadIdx.x + d < 32) above += o;
                    }
                    if (above >= k && above - mine < k) {         // one lane: the count from the top reaches k in its bins
                        unsigned run = above - mine;
                        int b = 7;
                        for (; b > 0; --b) {
                            run += sh_hist[threadIdx.x * 8 + b];
                            if (run >= k) break;
                        }
                        sh_cut = threadIdx.x * 8 + b;
                    }
                }
                __syncthreads();
                const unsigned cut = sh_cut;
                for (unsigned i = threadIdx.x; i < n; i += kTopkThreads) {
                    const uint64_t e = sh_cand[i];
                    if (bin_of(e) >= cut) sh_keep[atomicAdd(&sh_kept, 1u)] = e;
                }
                __syncthreads();
                list = sh_keep;
                n = sh_kept;
            }
            // 3. rank by counting, bias ranks below k
            if (threadIdx.x == 0 && (n & 1u)) list[n] = 0;         // pad to a pair (kCap is even; 0 ranks below all)
            __syncthreads();
            for (unsigned e = threadIdx.x; e < n; e += kTopkThreads) {
                const uint64_t mine = list[e];
                uint32_t r0 = 0, r1 = 0;
                const ulonglong2 *pairs = reinterpret_cast<const ulonglong2 *>(list);
#pragma unroll 4
                for (unsigned u = 0; u < (n + 1) / 2; ++u) {          // two composites per shared-memory load
                    const ulonglong2 q = pairs[u];
                    r0 += q.x > mine ? 1u : 0u;
                    r1 += q.y > mine ? 1u : 0u;
                }
                if (r0 + r1 < k)
                    bias_column<DTYPE, SCHEME>(a, material, row_ptr, 0xFFFFFFFFu - static_cast<uint32_t>(mine),
                                               static_cast<uint32_t>(mine >> 32));
            }
        } else {
            // fallback: k rounds of "largest composite below the previous one" find the composite
            // of the k-th ranked column without touching the row; one more pass then biases every
            // column at or above it (each column is judged on its own original value).  A real
            // composite is never 0 (its low word is 2^32 - 1 - column >= 2^31), so 0 means "none".
            uint64_t prev = 0;
            const uint32_t rounds = k < V ? k : V;
            for (uint32_t r = 0; r < rounds; ++r) {
                uint64_t best = 0;
                for_each_code<DTYPE, kTopkThreads>(row_ptr, 0u, V, a.vector, [&](uint32_t col, uint32_t code) {
                    const uint64_t c = composite(code, col);
                    if ((r == 0 || c < prev) && c > best) best = c;
                });
                prev = block_max_u64<kTopkWarps>(best, sh_red, &sh_best);
            }
            const uint64_t kth = prev;
            for_each_code<DTYPE, kTopkThreads>(row_ptr, 0u, V, a.vector, [&](uint32_t col, uint32_t code) {
                if (composite(code, col) >= kth)
                    bias_column<DTYPE, SCHEME>(a, material, row_ptr, col, DTYPE == SBW_DTYPE_F32 ? code : code >> 16);
            });
        }
        __syncthreads();             // shared scratch is reused by the next row
    }
}

template <int DTYPE, int SCHEME>
cudaError_t launch_cluster(const TopkArgs &a, int cs, cudaStream_t s) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(a.B * cs));
    cfg.blockDim = dim3(512);
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
        case 8: return cudaLaunchKernelEx(&cfg, topk_kernel<DTYPE, SCHEME, 512, 8>, a);
        case 4: return cudaLaunchKernelEx(&cfg, topk_kernel<DTYPE, SCHEME, 512, 4>, a);
        default: return cudaLaunchKernelEx(&cfg, topk_kernel<DTYPE, SCHEME, 512, 2>, a);
    }
}

template <int DTYPE, int SCHEME>
int launch(const TopkArgs &a, cudaStream_t s) {
    DeviceInfo di;
    const int rc = current_device_info(&di);
    if (rc != SBW_OK) return rc;
    // more rows than SMs: two 512-thread CTAs per SM keep twice as many rows in flight (that
    // kernel has 128 groups, so its fast path needs k <= 128); otherwise one 1024-thread CTA per row
    // small batches: a cluster of 512-thread CTAs per row, as many as keeps two CTAs on every SM
    const int64_t cap = static_cast<int64_t>(di.sm_count) * 2;
    const int cs = a.B * 8 <= cap ? 8 : a.B * 4 <= cap ? 4 : a.B * 2 <= cap ? 2 : 1;
    if (cs > 1 && (a.k + cs - 1) / cs <= 128 && a.V >= 4096) {
        SBW_CUDA_TRY((launch_cluster<DTYPE, SCHEME>(a, cs, s)));
    } else if (a.B > di.sm_count && a.k <= 128) {
        const unsigned grid = static_cast<unsigned>(a.B < cap ? a.B : cap);
        topk_kernel<DTYPE, SCHEME, 512, 1><<<grid, 512, 0, s>>>(a);
    } else {
        const unsigned grid = static_cast<unsigned>(a.B < di.sm_count ? a.B : di.sm_count);
        topk_kernel<DTYPE, SCHEME, 1024, 1><<<grid, 1024, 0, s>>>(a);
    }
    SBW_CUDA_TRY(cudaGetLastError());
    return SBW_OK;
}

}  // namespace
}  // namespace sbw

extern "C" int sbw_bias_logits_topk(void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                                    int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width,
                                    uint64_t key, double gamma, float delta, int scheme, int64_t top_k,
                                    void *stream) {
    using namespace sbw;
    if (!valid_common(dtype, ctx_width, gamma, scheme)) return SBW_ERR_INVALID_ARG;
    if (B < 0 || V <= 0 || ld < V || vocab_offset < 0 || top_k < 1) return SBW_ERR_INVALID_ARG;
    if (V > 0x7fffffffLL || vocab_offset + V > (int64_t(1) << 32)) return SBW_ERR_UNSUPPORTED;
    if (!(delta == delta) || delta - delta != 0.0f) return SBW_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (top_k >= V)   // every column is a candidate: the full-vocabulary kernel
        return bias_logits_impl(logits, dtype, B, V, ld, vocab_offset, ctx_tokens, ctx_width, key, gamma,
                                delta, scheme, s);
    if (B == 0) return SBW_OK;
    if (!logits || !ctx_tokens) return SBW_ERR_INVALID_ARG;

    TopkArgs a;
    a.logits = logits;
    a.B = B; a.V = V; a.ld = ld;
    a.ctx = ctx_tokens;
    a.W = ctx_width;
    a.vocab_offset = static_cast<uint32_t>(vocab_offset);
    a.key = key;
    a.thr_m1 = threshold_minus_one(gamma);
    a.delta = dtype == SBW_DTYPE_BF16 ? __bfloat162float(__float2bfloat16_rn(delta)) : delta;
    a.weyl = make_weyl();
    a.k = static_cast<int>(top_k);
    const int esize = dtype == SBW_DTYPE_F32 ? 4 : 2;
    a.vector = (reinterpret_cast<uintptr_t>(logits) % 16 == 0) && ((ld * esize) % 16 == 0);
    if (a.delta == 0.0f) return SBW_OK;   // the paper's delta = 0 control: no bit changes

    if (dtype == SBW_DTYPE_F32)
        return scheme == SBW_SCHEME_CONTEXT ? launch<SBW_DTYPE_F32, SBW_SCHEME_CONTEXT>(a, s)
                                            : launch<SBW_DTYPE_F32, SBW_SCHEME_SELFSALT>(a, s);
    return scheme == SBW_SCHEME_CONTEXT ? launch<SBW_DTYPE_BF16, SBW_SCHEME_CONTEXT>(a, s)
                                        : launch<SBW_DTYPE_BF16, SBW_SCHEME_SELFSALT>(a, s);
}
