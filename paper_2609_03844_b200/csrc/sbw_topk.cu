// sbw_bias_logits_topk: the paper's SBW-ss scheme (Table 1: Bernoulli list, self-salt seeding,
// candidates "top-40") -- per row only the k largest logits are tested and biased, as KGW's
// selfhash does; everything else in the row is left alone.
//
// One CTA per row.  "Largest" is the total order on order-encoded bit patterns with ties to the
// lowest column, expressed as one 64-bit composite (code << 32 | ~column).
//   1. A pass over a prefix of the row (32 columns per thread): every thread keeps the largest code
//      it has seen; groups of four threads give 256 maxima of disjoint column sets.  Their k-th
//      largest value L is a lower bound of the row's k-th largest logit (k distinct columns reach
//      it), and it is known after a fifth of the row.
//   2. One pass over the whole row: columns with code >= L -- a few hundred for ordinary logits --
//      go into a shared-memory candidate list.  The common path is one compare per 16-byte vector.
//   3. Candidates are ranked by counting larger composites; ranks below k are hashed and biased.
// If the list overflows (rows of equal values, k > 256) the CTA falls back to k rounds of "largest
// composite below the previous one", a block reduction each, and one pass that biases every
// column at or above the k-th composite: slow, but it needs no assumption about the data.
#include <algorithm>
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include "sbw_common.cuh"
#include "sbw_hash.cuh"

namespace sbw {

int bias_logits_impl(void *logits, int dtype, int64_t B, int64_t V, int64_t ld, int64_t vocab_offset,
                     const int32_t *ctx_tokens, int ctx_width, uint64_t key, double gamma, float delta,
                     int scheme, cudaStream_t stream);

// Waits of the bulk-copy pipeline that ran out (see topk_stream_kernel); read by sbw_pipeline_timeouts.
__device__ unsigned long long g_pipeline_timeouts;

namespace {

// CTA size: 1024 threads (one CTA per SM) when there are fewer rows than SMs can take two of,
// 512 threads (two CTAs per SM, twice the rows in flight) for larger batches.
constexpr int kCap = 2048;                  // candidate list entries
constexpr int kPrefixColumns = 32768;        // leading columns read by the pass that finds the bound

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
    // bulk-copy kernel only: bytes of a row that bulk copies take (a multiple of 16), bytes of
    // the prefix pass, and their chunk counts
    uint32_t row_bytes, prefix_bytes, chunks_row, chunks_prefix;
};

__device__ __forceinline__ uint32_t order_code(uint32_t bits) {
    return (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
}
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

// Order codes of the fast paths (steps 1 to 3).  fp32: order_code of the bits.  bf16: the 16-bit analogue,
// bits ^ 0xffff for negative values and bits ^ 0x8000 otherwise, computed for both halves of a word
// at once (a byte permute in sign-replication mode gives each half's sign mask).
__device__ __forceinline__ uint32_t packed_codes(uint32_t w) {
    uint32_t sign;   // 0xffff in each half whose value is negative (selector bit 3: replicate the byte's msb)
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(sign) : "r"(w), "r"(0u), "r"(0xBB99u));
    return w ^ (sign | 0x80008000u);
}
template <int DTYPE>
__device__ __forceinline__ uint32_t vector_max_code(const uint4 &w) {
    if constexpr (DTYPE == SBW_DTYPE_F32) {
        return max(max(order_code(w.x), order_code(w.y)), max(order_code(w.z), order_code(w.w)));
    } else {
        const uint32_t m = __vmaxu2(__vmaxu2(packed_codes(w.x), packed_codes(w.y)),
                                    __vmaxu2(packed_codes(w.z), packed_codes(w.w)));
        return max(m >> 16, m & 0xffffu);
    }
}
template <int DTYPE>
__device__ __forceinline__ uint32_t element_code(const uint4 &w, int i) {
    const uint32_t *e = reinterpret_cast<const uint32_t *>(&w);
    if constexpr (DTYPE == SBW_DTYPE_F32) return order_code(e[i]);
    else return (packed_codes(e[i >> 1]) >> (16 * (i & 1))) & 0xffffu;
}

template <int DTYPE>
__device__ __forceinline__ uint32_t scalar_code(const char *row_ptr, uint32_t col) {
    if constexpr (DTYPE == SBW_DTYPE_F32) return order_code(reinterpret_cast<const uint32_t *>(row_ptr)[col]);
    else return packed_codes(reinterpret_cast<const uint16_t *>(row_ptr)[col]) & 0xffffu;
}

// Calls fvec(first column, vector) for the aligned 16-byte vectors of the columns [begin, end) that
// this thread owns and fone(column, code) for the columns left over (all of them when the rows
// are not aligned); begin is a multiple of 8 columns.
template <int DTYPE, int kTopkThreads, typename FV, typename F1>
__device__ __forceinline__ void for_each_vector(const char *row_ptr, uint32_t begin, uint32_t end, bool vector,
                                                FV fvec, F1 fone) {
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
                if (j < nfull) fvec(j * VEC, w[u]);
            }
        }
        done = max(begin, nfull * VEC);
    }
    for (uint32_t c = done + threadIdx.x; c < end; c += kTopkThreads) fone(c, scalar_code<DTYPE>(row_ptr, c));
}

// Eq. 1 + Eq. 2 on one chosen column.
template <int DTYPE, int SCHEME>
__device__ __noinline__ void bias_column(const TopkArgs &a, int64_t row, char *row_ptr, uint32_t col) {
    const int32_t *ctx = a.ctx + row * a.W;
    const uint32_t v = a.vocab_offset + col;
    uint64_t r;
    if constexpr (SCHEME == SBW_SCHEME_CONTEXT) r = seed_context(a.key, ctx, a.W);
    else r = seed_selfsalt(a.key, jenkins_min(ctx, a.W), v);
    if (philox_word0(v, r, a.weyl) > a.thr_m1) return;
    if constexpr (DTYPE == SBW_DTYPE_F32) {
        float *p = reinterpret_cast<float *>(row_ptr) + col;
        *p = __fadd_rn(*p, a.delta);
    } else {
        __nv_bfloat16 *p = reinterpret_cast<__nv_bfloat16 *>(row_ptr) + col;
        *p = __float2bfloat16_rn(__fadd_rn(__bfloat162float(*p), a.delta));
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
    __shared__ uint64_t sh_cand[kCap];
    __shared__ uint64_t sh_red[kTopkWarps];
    __shared__ uint64_t sh_best;
    __shared__ uint32_t sh_floor;
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

        // 1. lower bound of the k-th largest code from a prefix of the columns
        const uint32_t prefix_end = min(c_hi, c_lo + static_cast<uint32_t>(kPrefixColumns / CS));
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
            sh_count = 0;
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
        for_each_vector<DTYPE, kTopkThreads>(
            row_ptr, c_lo, c_hi, a.vector,
            [&](uint32_t col0, const uint4 &w) {
                if (vector_max_code<DTYPE>(w) < floor_code) return;   // the common case: one compare per vector
#pragma unroll
                for (int i = 0; i < 16 / ESIZE; ++i) push(col0 + i, element_code<DTYPE>(w, i));
            },
            push);
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
            // 3. rank by counting, bias ranks below k
            for (unsigned e = threadIdx.x; e < n; e += kTopkThreads) {
                const uint64_t mine = sh_cand[e];
                uint32_t rank = 0;
                for (unsigned u = 0; u < n; ++u) rank += sh_cand[u] > mine ? 1u : 0u;
                if (rank < k) bias_column<DTYPE, SCHEME>(a, row, row_ptr, 0xFFFFFFFFu - static_cast<uint32_t>(mine));
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
                if (composite(code, col) >= kth) bias_column<DTYPE, SCHEME>(a, row, row_ptr, col);
            });
        }
        __syncthreads();             // shared scratch is reused by the next row
    }
}

// ---------------------------------------------------------------------------------------------
// Large batches: the same three steps with the row staged through shared memory by bulk
// asynchronous copies (cp.async.bulk, completion counted on an mbarrier).  The logits in flight
// sit in a ring of kStages chunks instead of registers, and one thread keeps the ring full across
// the steps and across rows: while a row is ranked and biased, the first chunks of the CTA's next
// row are already on their way.  The order of chunks a CTA consumes is fixed -- per row the
// prefix, then the whole row -- so producer and consumers only count.
//
//   full[s]   completes when the bytes of the chunk in stage s have landed (1 arrival + tx count)
//   empty[s]  completes when all warps are done with the chunk in stage s (kStreamWarps arrivals)
//
// Every wait is bounded (polls and wall time); a wait that runs out marks the CTA dead: it stops
// issuing copies and waiting, writes nothing more, and the count of such events is readable
// through sbw_pipeline_timeouts().
constexpr int kStreamThreads = 512;
constexpr int kStreamWarps = kStreamThreads / 32;
#ifndef SBW_TOPK_CHUNK
#define SBW_TOPK_CHUNK 32768
#endif
#ifndef SBW_TOPK_STAGES
#define SBW_TOPK_STAGES 2
#endif
constexpr uint32_t kChunkBytes = SBW_TOPK_CHUNK;
constexpr int kStages = SBW_TOPK_STAGES;                // a power of two
#ifndef SBW_TOPK_LAG
#define SBW_TOPK_LAG 1
#endif
constexpr uint32_t kRefillLag = SBW_TOPK_LAG;           // 1 <= lag < kStages
constexpr uint32_t kWaitPolls = 1u << 24;
constexpr unsigned long long kWaitNanos = 2000000000ull;

struct StreamShared {
    alignas(128) unsigned char stage[kStages][kChunkBytes];
    uint64_t cand[kCap];
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t red[kStreamWarps];
    uint64_t best;
    uint32_t max4[kStreamThreads / 4];
    uint32_t floor_code;
    unsigned count;
    unsigned dead;
    int64_t next_row;      // thread 0: the next chunk to issue is chunk next_w of this row's sequence
    uint32_t next_w;       //   (prefix chunks, then row chunks),
    uint32_t next_q;       //   chunk next_q of the CTA's whole sequence
};

__device__ __forceinline__ uint32_t shared_address(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(shared_address(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(shared_address(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(shared_address(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(shared_address(bar)), "r"(parity)
        : "memory");
    return ok != 0u;
}
__device__ __forceinline__ unsigned long long global_nanos() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Waits for the phase of `bar` with the given parity; false (and the CTA marked dead) when the
// limits run out.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, StreamShared &sh) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = 0;
    for (uint32_t n = 1; n < kWaitPolls; ++n) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((n & 1023u) == 0u) {
            const unsigned long long now = global_nanos();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitNanos) break;
        }
    }
    *reinterpret_cast<volatile unsigned *>(&sh.dead) = 1u;
    atomicAdd(&g_pipeline_timeouts, 1ull);
    return false;
}
// Source and destination 16-byte aligned, bytes a multiple of 16; this CTA's own shared memory.
__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     shared_address(dst)),
                 "l"(src), "r"(bytes), "r"(shared_address(bar))
                 : "memory");
}

// Thread 0: issue the next chunk of the CTA's sequence, if there is one.  Its position in the
// sequence lives in shared memory (sh.next_*): one thread uses it once per chunk.
template <int ESIZE>
__device__ __forceinline__ void issue_chunk(const TopkArgs &a, StreamShared &sh) {
    const int64_t row = sh.next_row;
    if (row >= a.B) return;
    const uint32_t w = sh.next_w, q = sh.next_q;
    const bool in_prefix = w < a.chunks_prefix;
    const uint32_t c = in_prefix ? w : w - a.chunks_prefix;
    const uint32_t limit = in_prefix ? a.prefix_bytes : a.row_bytes;
    const uint32_t off = c * kChunkBytes;
    const uint32_t bytes = min(kChunkBytes, limit - off);
    const uint32_t st = q % kStages;
    const char *src = static_cast<const char *>(a.logits) + row * a.ld * ESIZE + off;
    mbar_expect_tx(&sh.full[st], bytes);
    bulk_load(sh.stage[st], src, bytes, &sh.full[st]);
    sh.next_q = q + 1;
    if (w + 1 == a.chunks_prefix + a.chunks_row) {
        sh.next_w = 0;
        sh.next_row = row + gridDim.x;
    } else {
        sh.next_w = w + 1;
    }
}

// Consumes `nchunks` chunks covering `limit` bytes from the start of the row; f(first column,
// vector) for every 16-byte vector, each thread taking every kStreamThreads-th.
template <int DTYPE, typename F>
__device__ __forceinline__ void consume_chunks(const TopkArgs &a, StreamShared &sh, uint32_t &q_next, bool &dead,
                                               uint32_t nchunks, uint32_t limit, F f) {
    constexpr int ESIZE = DTYPE == SBW_DTYPE_F32 ? 4 : 2;
    constexpr int VEC = 16 / ESIZE;
    constexpr uint32_t kChunkVectors = kChunkBytes / 16u;
    constexpr int kPer = kChunkVectors / kStreamThreads;
    for (uint32_t c = 0; c < nchunks; ++c) {
        const uint32_t q = q_next;
        const uint32_t st = q % kStages;
        if (threadIdx.x == 0 && q >= kRefillLag && !dead && sh.next_row < a.B) {
            // a stage is refilled once every warp has left it
            const uint32_t qp = q - kRefillLag;
            if (mbar_wait(&sh.empty[qp % kStages], (qp / kStages) & 1u, sh)) issue_chunk<ESIZE>(a, sh);
            else dead = true;
        }
        if (!dead && !mbar_wait(&sh.full[st], (q / kStages) & 1u, sh)) dead = true;
        if (!dead) {
            const uint32_t off = c * kChunkBytes;
            const uint32_t nvec = min(kChunkBytes, limit - off) / 16u;
            const uint4 *src = reinterpret_cast<const uint4 *>(sh.stage[st]);
            const uint32_t vec0 = off / 16u;
            if (nvec == kChunkVectors) {
                uint4 w[kPer];
#pragma unroll
                for (int u = 0; u < kPer; ++u) w[u] = src[threadIdx.x + u * kStreamThreads];
#pragma unroll
                for (int u = 0; u < kPer; ++u) f((vec0 + threadIdx.x + u * kStreamThreads) * VEC, w[u]);
            } else {
                for (uint32_t j = threadIdx.x; j < nvec; j += kStreamThreads) f((vec0 + j) * VEC, src[j]);
            }
        }
        __syncwarp();
        if ((threadIdx.x & 31) == 0) mbar_arrive(&sh.empty[st]);
        q_next = q + 1;
    }
}

template <int DTYPE, int SCHEME>
__global__ void __launch_bounds__(kStreamThreads, 2)
topk_stream_kernel(const TopkArgs a) {
    constexpr int ESIZE = DTYPE == SBW_DTYPE_F32 ? 4 : 2;
    constexpr int kGroups = kStreamThreads / 4;
    extern __shared__ __align__(128) unsigned char stream_smem[];
    StreamShared &sh = *reinterpret_cast<StreamShared *>(stream_smem);
    const uint32_t V = static_cast<uint32_t>(a.V);
    const uint32_t k = static_cast<uint32_t>(a.k);
    uint32_t q_next = 0;     // the chunk of the CTA's sequence this thread consumes next
    bool dead = false;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&sh.full[s], 1u);
            mbar_init(&sh.empty[s], kStreamWarps);
        }
        sh.dead = 0u;
        sh.next_row = blockIdx.x;
        sh.next_w = 0u;
        sh.next_q = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0)
        for (int s = 0; s < kStages; ++s) issue_chunk<ESIZE>(a, sh);

    for (int64_t row = blockIdx.x; row < a.B; row += gridDim.x) {
        char *row_ptr = static_cast<char *>(a.logits) + row * a.ld * ESIZE;

        // 1. lower bound of the k-th largest code from the prefix
        uint32_t mx = 0;
        consume_chunks<DTYPE>(a, sh, q_next, dead, a.chunks_prefix, a.prefix_bytes,
                              [&](uint32_t, const uint4 &w) { mx = max(mx, vector_max_code<DTYPE>(w)); });
        mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        if ((threadIdx.x & 3) == 0) sh.max4[threadIdx.x >> 2] = mx;
        if (threadIdx.x == 0) {
            sh.floor_code = 0;
            sh.count = 0;
        }
        __syncthreads();
        if (threadIdx.x < kGroups) {
            const uint32_t mine = sh.max4[threadIdx.x];
            uint32_t rank = 0;
            for (int u = 0; u < kGroups; ++u) {
                const uint32_t o = sh.max4[u];
                rank += (o > mine || (o == mine && u < static_cast<int>(threadIdx.x))) ? 1u : 0u;
            }
            if (rank == k - 1) sh.floor_code = mine;       // the launch guarantees k <= kGroups
        }
        __syncthreads();
        const uint32_t floor_code = sh.floor_code;

        // 2. candidates: every column that reaches the bound
        auto push = [&](uint32_t col, uint32_t code) {
            if (code >= floor_code) {
                const unsigned pos = atomicAdd(&sh.count, 1u);
                if (pos < kCap) sh.cand[pos] = composite(code, col);
            }
        };
        consume_chunks<DTYPE>(a, sh, q_next, dead, a.chunks_row, a.row_bytes, [&](uint32_t col0, const uint4 &w) {
            if (vector_max_code<DTYPE>(w) < floor_code) return;       // the common case: one compare per vector
#pragma unroll
            for (int i = 0; i < 16 / ESIZE; ++i) push(col0 + i, element_code<DTYPE>(w, i));
        });
        for (uint32_t c = a.row_bytes / ESIZE + threadIdx.x; c < V; c += kStreamThreads) {   // ragged end of the row
            push(c, scalar_code<DTYPE>(row_ptr, c));
        }
        __syncthreads();
        const unsigned n = sh.count;
        const bool row_dead = *reinterpret_cast<volatile unsigned *>(&sh.dead) != 0u;

        if (row_dead) {
            // a wait ran out somewhere in this CTA: the candidates cannot be trusted, nothing is written
        } else if (n <= kCap) {
            // 3. rank by counting, bias ranks below k
            for (unsigned e = threadIdx.x; e < n; e += kStreamThreads) {
                const uint64_t mine = sh.cand[e];
                uint32_t rank = 0;
                for (unsigned u = 0; u < n; ++u) rank += sh.cand[u] > mine ? 1u : 0u;
                if (rank < k) bias_column<DTYPE, SCHEME>(a, row, row_ptr, 0xFFFFFFFFu - static_cast<uint32_t>(mine));
            }
        } else {
            // fallback as in topk_kernel, on the row in global memory
            uint64_t prev = 0;
            const uint32_t rounds = k < V ? k : V;
            for (uint32_t r = 0; r < rounds; ++r) {
                uint64_t best = 0;
                for_each_code<DTYPE, kStreamThreads>(row_ptr, 0u, V, true, [&](uint32_t col, uint32_t code) {
                    const uint64_t c = composite(code, col);
                    if ((r == 0 || c < prev) && c > best) best = c;
                });
                prev = block_max_u64<kStreamWarps>(best, sh.red, &sh.best);
            }
            const uint64_t kth = prev;
            for_each_code<DTYPE, kStreamThreads>(row_ptr, 0u, V, true, [&](uint32_t col, uint32_t code) {
                if (composite(code, col) >= kth) bias_column<DTYPE, SCHEME>(a, row, row_ptr, col);
            });
        }
        __syncthreads();             // shared scratch is reused by the next row
    }

    // Copies that were issued are all consumed above unless the CTA went dead; then wait, within
    // the same limits, for the stages that may still be written before the shared memory is given up.
    if (threadIdx.x == 0 && dead) {
        const uint32_t issued = sh.next_q;
        for (uint32_t back = 1; back <= static_cast<uint32_t>(kStages) && back <= issued; ++back) {
            const uint32_t qi = issued - back;
            mbar_wait(&sh.full[qi % kStages], (qi / kStages) & 1u, sh);
        }
    }
}

template <int DTYPE, int SCHEME>
cudaError_t launch_stream(const TopkArgs &a, unsigned grid, cudaStream_t s) {
    // two CTAs of this size per SM need most of the SM's memory as shared memory
    static const cudaError_t configured = [] {
        const cudaError_t e = cudaFuncSetAttribute(topk_stream_kernel<DTYPE, SCHEME>,
                                                   cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   static_cast<int>(sizeof(StreamShared)));
        if (e != cudaSuccess) return e;
        return cudaFuncSetAttribute(topk_stream_kernel<DTYPE, SCHEME>,
                                    cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    }();
    if (configured != cudaSuccess) return configured;
    topk_stream_kernel<DTYPE, SCHEME><<<grid, kStreamThreads, sizeof(StreamShared), s>>>(a);
    return cudaSuccess;
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
        const int esize = DTYPE == SBW_DTYPE_F32 ? 4 : 2;
        // aligned rows of ordinary width go through the bulk-copy pipeline
        if (a.vector && a.V >= 4096 && a.V * esize < (int64_t(1) << 31)) {
            TopkArgs b = a;
            b.row_bytes = static_cast<uint32_t>(a.V * esize) & ~15u;
            b.prefix_bytes = std::min<uint32_t>(b.row_bytes, kPrefixColumns * esize);
            b.chunks_row = (b.row_bytes + kChunkBytes - 1) / kChunkBytes;
            b.chunks_prefix = (b.prefix_bytes + kChunkBytes - 1) / kChunkBytes;
            SBW_CUDA_TRY((launch_stream<DTYPE, SCHEME>(b, grid, s)));
        }
        else
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
    a.row_bytes = a.prefix_bytes = a.chunks_row = a.chunks_prefix = 0u;
    if (a.delta == 0.0f) return SBW_OK;   // the paper's delta = 0 control: no bit changes

    if (dtype == SBW_DTYPE_F32)
        return scheme == SBW_SCHEME_CONTEXT ? launch<SBW_DTYPE_F32, SBW_SCHEME_CONTEXT>(a, s)
                                            : launch<SBW_DTYPE_F32, SBW_SCHEME_SELFSALT>(a, s);
    return scheme == SBW_SCHEME_CONTEXT ? launch<SBW_DTYPE_BF16, SBW_SCHEME_CONTEXT>(a, s)
                                        : launch<SBW_DTYPE_BF16, SBW_SCHEME_SELFSALT>(a, s);
}

extern "C" int sbw_pipeline_timeouts(unsigned long long *host_count) {
    using namespace sbw;
    if (!host_count) return SBW_ERR_INVALID_ARG;
    SBW_CUDA_TRY(cudaMemcpyFromSymbol(host_count, g_pipeline_timeouts, sizeof(unsigned long long)));
    return SBW_OK;
}
