// sbw_roc_auc: area under the ROC curve of detection scores (Section 4.3 of the paper) as the
// exact pair statistic  AUC = (2 #{z_pos > z_neg} + #{z_pos == z_neg}) / (2 n_pos n_neg).
//
// Three kernels.  split_kernel copies the scores of each class into its own dense array (slot
// allocation by one atomic per warp and class; the order inside a class does not matter to a
// count) and drops NaNs.  sort_tiles_kernel sorts the negatives inside every tile of
// kRocNegTile scores (bitonic network in shared memory).  pairs_kernel walks the (positive
// chunk) x (negative tile) grid with a persistent set of CTAs: the sorted tile sits in shared
// memory and every positive finds #{q < p} and #{q <= p} in it by two branch-free binary
// searches, kRocPerThread positives per thread interleaved -- 2 log2(tile) probes per
// (positive, tile) instead of one compare per pair.  Counts are integers, so the result does not
// depend on the order of anything; the last CTA to finish (atomic ticket) forms the quotient.
#include "sbw_common.cuh"

namespace sbw {
namespace {

constexpr int kRocThreads = 256;
constexpr int kRocPerThread = 8;
constexpr int kRocPosTile = kRocThreads * kRocPerThread;   // positives per work item
constexpr int kRocNegTile = 2048;                          // negatives per sorted tile (16 KiB of shared memory)
constexpr int kRocSortThreads = kRocNegTile / 2;

// counters in the workspace
struct RocCounters {
    unsigned long long n_pos, n_neg, greater, equal;
    unsigned int ticket, pad;
};

__global__ void __launch_bounds__(kRocThreads)
split_kernel(const double *z, const uint8_t *labels, int64_t n, double *pos, double *neg, RocCounters *c) {
    const int lane = threadIdx.x & 31;
    for (int64_t base = (static_cast<int64_t>(blockIdx.x) * kRocThreads + threadIdx.x) - lane; base < n;
         base += static_cast<int64_t>(gridDim.x) * kRocThreads) {
        const int64_t i = base + lane;
        double v = 0.0;
        int cls = -1;                                   // -1: not there or NaN
        if (i < n) {
            v = z[i];
            if (v == v) cls = labels[i] ? 1 : 0;
        }
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const unsigned m = __ballot_sync(0xffffffffu, cls == k);
            if (m == 0u) continue;
            const int leader = __ffs(m) - 1;
            unsigned long long start = 0;
            if (lane == leader) start = atomicAdd(k ? &c->n_pos : &c->n_neg, static_cast<unsigned long long>(__popc(m)));
            start = __shfl_sync(0xffffffffu, start, leader);
            if (cls == k) (k ? pos : neg)[start + __popc(m & ((1u << lane) - 1u))] = v;
        }
    }
}

// Sorts each tile of kRocNegTile negatives in place, ascending; a short last tile is padded with
// +inf in shared memory and only its own entries are written back (they are its smallest).
__global__ void __launch_bounds__(kRocSortThreads)
sort_tiles_kernel(double *neg, const RocCounters *c) {
    __shared__ double s[kRocNegTile];
    const unsigned long long n_neg = c->n_neg;
    const unsigned long long tiles = (n_neg + kRocNegTile - 1) / kRocNegTile;
    const double inf = __longlong_as_double(0x7ff0000000000000LL);
    for (unsigned long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const unsigned long long base = tile * kRocNegTile;
        for (int j = threadIdx.x; j < kRocNegTile; j += kRocSortThreads)
            s[j] = base + j < n_neg ? neg[base + j] : inf;
        __syncthreads();
        for (int k = 2; k <= kRocNegTile; k <<= 1) {
            for (int j = k >> 1; j > 0; j >>= 1) {
                const int t = threadIdx.x;
                const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));     // bit j clear
                const double a = s[i], b = s[i + j];
                const bool ascending = (i & k) == 0;
                if ((a > b) == ascending) {
                    s[i] = b;
                    s[i + j] = a;
                }
                __syncthreads();
            }
        }
        for (int j = threadIdx.x; j < kRocNegTile; j += kRocSortThreads)
            if (base + j < n_neg) neg[base + j] = s[j];
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kRocThreads)
pairs_kernel(const double *pos, const double *neg, RocCounters *c, double *out_auc, uint64_t *out_stats) {
    __shared__ double sneg[kRocNegTile];
    __shared__ unsigned long long red[2][kRocThreads / 32];
    __shared__ bool last;
    const unsigned long long n_pos = c->n_pos, n_neg = c->n_neg;   // written by the split kernel
    const unsigned long long tiles_p = (n_pos + kRocPosTile - 1) / kRocPosTile;
    const unsigned long long tiles_n = (n_neg + kRocNegTile - 1) / kRocNegTile;
    const double nan = __longlong_as_double(0x7ff8000000000000LL);
    const double inf = __longlong_as_double(0x7ff0000000000000LL);

    unsigned long long greater = 0, equal = 0;
    for (unsigned long long item = blockIdx.x; item < tiles_p * tiles_n; item += gridDim.x) {
        const unsigned long long tp = item / tiles_n, tn = item % tiles_n;
        const unsigned long long left = n_neg - tn * kRocNegTile;
        const unsigned m = left < kRocNegTile ? static_cast<unsigned>(left) : kRocNegTile;   // real entries
        double p[kRocPerThread];
#pragma unroll
        for (int r = 0; r < kRocPerThread; ++r) {
            const unsigned long long i = tp * kRocPosTile + r * kRocThreads + threadIdx.x;
            p[r] = i < n_pos ? pos[i] : nan;             // NaN compares false: counts nothing
        }
        __syncthreads();                                 // the previous tile's readers are done
        for (int j = threadIdx.x; j < kRocNegTile; j += kRocThreads)
            sneg[j] = static_cast<unsigned>(j) < m ? neg[tn * kRocNegTile + j] : inf;
        __syncthreads();
        // lt[r] = #{q < p[r]}, le[r] = #{q <= p[r]} over the sorted tile; padding is +inf and
        // sorts last, so clamping to m removes it
        unsigned lt[kRocPerThread], le[kRocPerThread];
#pragma unroll
        for (int r = 0; r < kRocPerThread; ++r) lt[r] = le[r] = 0;
#pragma unroll
        for (int step = kRocNegTile / 2; step > 0; step >>= 1) {
#pragma unroll
            for (int r = 0; r < kRocPerThread; ++r) {
                if (sneg[lt[r] + step - 1] < p[r]) lt[r] += step;
                if (sneg[le[r] + step - 1] <= p[r]) le[r] += step;
            }
        }
        unsigned g = 0, e = 0;
#pragma unroll
        for (int r = 0; r < kRocPerThread; ++r) {
            if (sneg[lt[r]] < p[r]) lt[r] += 1;
            if (sneg[le[r]] <= p[r]) le[r] += 1;
            lt[r] = min(lt[r], m);
            le[r] = min(le[r], m);
            g += lt[r];
            e += le[r] - lt[r];
        }
        greater += g;
        equal += e;
    }
    for (int d = 16; d > 0; d >>= 1) {
        greater += __shfl_down_sync(0xffffffffu, greater, d);
        equal += __shfl_down_sync(0xffffffffu, equal, d);
    }
    if ((threadIdx.x & 31) == 0) {
        red[0][threadIdx.x >> 5] = greater;
        red[1][threadIdx.x >> 5] = equal;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long gs = 0, es = 0;
        for (int w = 0; w < kRocThreads / 32; ++w) {
            gs += red[0][w];
            es += red[1][w];
        }
        if (gs) atomicAdd(&c->greater, gs);
        if (es) atomicAdd(&c->equal, es);
        __threadfence();
        last = atomicAdd(&c->ticket, 1u) == gridDim.x - 1;
        if (last) {
            __threadfence();
            const unsigned long long G = atomicAdd(&c->greater, 0ull), E = atomicAdd(&c->equal, 0ull);
            if (out_stats) {
                out_stats[0] = G;
                out_stats[1] = E;
                out_stats[2] = n_pos;
                out_stats[3] = n_neg;
            }
            *out_auc = (n_pos == 0 || n_neg == 0)
                           ? nan
                           : __ddiv_rn(__ull2double_rn(2ull * G + E), __ull2double_rn(2ull * n_pos * n_neg));
        }
    }
}


// Many independent problems at once (the paper's tables hold one AUC per configuration, each over
// a few hundred texts): one CTA per problem, no workspace.  The problem's scores are walked in
// windows of kRocNegTile; the negatives of a window are compacted into shared memory (their order
// does not matter), padded with +inf and sorted, and every positive of the whole problem is then
// searched in them as in pairs_kernel.
__global__ void __launch_bounds__(kRocSortThreads)
batched_kernel(const double *z, const uint8_t *labels, const int64_t *offsets, int64_t M, double *out_auc,
               uint64_t *out_stats) {
    __shared__ double s[kRocNegTile];
    __shared__ unsigned long long red[3][kRocSortThreads / 32];
    __shared__ unsigned int s_count;
    const double inf = __longlong_as_double(0x7ff0000000000000LL);
    const double nan = __longlong_as_double(0x7ff8000000000000LL);
    for (int64_t prob = blockIdx.x; prob < M; prob += gridDim.x) {
        const int64_t lo = offsets[prob], hi = offsets[prob + 1];
        const int64_t n = hi > lo ? hi - lo : 0;
        const double *zp = z + lo;
        const uint8_t *lp = labels + lo;
        unsigned long long greater = 0, equal = 0, n_pos = 0, n_neg = 0;
        for (int64_t w0 = 0; w0 < n; w0 += kRocNegTile) {
            if (threadIdx.x == 0) s_count = 0u;
            __syncthreads();
            for (int j = threadIdx.x; j < kRocNegTile; j += kRocSortThreads) {
                const int64_t i = w0 + j;
                if (i < n) {
                    const double v = zp[i];
                    if (v == v && !lp[i]) s[atomicAdd(&s_count, 1u)] = v;
                }
            }
            __syncthreads();
            const unsigned m = s_count;
            for (int j = m + threadIdx.x; j < kRocNegTile; j += kRocSortThreads) s[j] = inf;
            __syncthreads();
            for (int k = 2; k <= kRocNegTile; k <<= 1) {
                for (int j = k >> 1; j > 0; j >>= 1) {
                    const int t = threadIdx.x;
                    const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
                    const double a = s[i], b = s[i + j];
                    if ((a > b) == ((i & k) == 0)) {
                        s[i] = b;
                        s[i + j] = a;
                    }
                    __syncthreads();
                }
            }
            if (threadIdx.x == 0) n_neg += m;
            if (m > 0) {
                for (int64_t i = threadIdx.x; i < n; i += kRocSortThreads) {
                    const double p = lp[i] ? zp[i] : nan;          // NaN compares false: counts nothing
                    unsigned lt = 0, le = 0;
#pragma unroll
                    for (int step = kRocNegTile / 2; step > 0; step >>= 1) {
                        if (s[lt + step - 1] < p) lt += step;
                        if (s[le + step - 1] <= p) le += step;
                    }
                    if (s[lt] < p) lt += 1;
                    if (s[le] <= p) le += 1;
                    lt = min(lt, m);
                    le = min(le, m);
                    greater += lt;
                    equal += le - lt;
                }
            }
            __syncthreads();
        }
        for (int64_t i = threadIdx.x; i < n; i += kRocSortThreads) {
            const double v = zp[i];
            if (v == v && lp[i]) n_pos += 1;
        }
        for (int d = 16; d > 0; d >>= 1) {
            greater += __shfl_down_sync(0xffffffffu, greater, d);
            equal += __shfl_down_sync(0xffffffffu, equal, d);
            n_pos += __shfl_down_sync(0xffffffffu, n_pos, d);
        }
        if ((threadIdx.x & 31) == 0) {
            red[0][threadIdx.x >> 5] = greater;
            red[1][threadIdx.x >> 5] = equal;
            red[2][threadIdx.x >> 5] = n_pos;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long G = 0, E = 0, P = 0;
            for (int w = 0; w < kRocSortThreads / 32; ++w) {
                G += red[0][w];
                E += red[1][w];
                P += red[2][w];
            }
            if (out_stats) {
                out_stats[4 * prob + 0] = G;
                out_stats[4 * prob + 1] = E;
                out_stats[4 * prob + 2] = P;
                out_stats[4 * prob + 3] = n_neg;
            }
            out_auc[prob] = (P == 0 || n_neg == 0)
                                ? nan
                                : __ddiv_rn(__ull2double_rn(2ull * G + E), __ull2double_rn(2ull * P * n_neg));
        }
        __syncthreads();
    }
}

}  // namespace
}  // namespace sbw

extern "C" size_t sbw_roc_auc_workspace_bytes(int64_t n) {
    if (n < 0) return 0;
    return 256 + 2 * sbw::align_up(static_cast<size_t>(n) * sizeof(double), 256);
}

extern "C" int sbw_roc_auc(const double *z, const uint8_t *labels, int64_t n, double *out_auc,
                           uint64_t *out_stats, void *workspace, size_t workspace_bytes, void *stream) {
    using namespace sbw;
    if (n < 0 || !out_auc) return SBW_ERR_INVALID_ARG;
    if (n > 0 && (!z || !labels)) return SBW_ERR_INVALID_ARG;
    if (n > (int64_t(1) << 31)) return SBW_ERR_UNSUPPORTED;      // 2 n_pos n_neg must fit 64 bits
    if (!workspace || workspace_bytes < sbw_roc_auc_workspace_bytes(n) ||
        reinterpret_cast<uintptr_t>(workspace) % 256 != 0)
        return SBW_ERR_WORKSPACE;
    DeviceInfo di;
    if (int rc = current_device_info(&di)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    RocCounters *c = static_cast<RocCounters *>(workspace);
    const size_t arr = align_up(static_cast<size_t>(n) * sizeof(double), 256);
    double *pos = reinterpret_cast<double *>(static_cast<char *>(workspace) + 256);
    double *neg = reinterpret_cast<double *>(static_cast<char *>(workspace) + 256 + arr);
    SBW_CUDA_TRY(cudaMemsetAsync(c, 0, sizeof(RocCounters), s));
    if (n > 0) {
        const int64_t blocks = (n + kRocThreads - 1) / kRocThreads;
        const unsigned grid = static_cast<unsigned>(blocks < 8LL * di.sm_count ? blocks : 8LL * di.sm_count);
        split_kernel<<<grid, kRocThreads, 0, s>>>(z, labels, n, pos, neg, c);
        SBW_CUDA_TRY(cudaGetLastError());
    }
    {
        const int64_t tiles = (n + kRocNegTile - 1) / kRocNegTile + 1;
        const int64_t cap = 2LL * di.sm_count;
        sort_tiles_kernel<<<static_cast<unsigned>(tiles < cap ? tiles : cap), kRocSortThreads, 0, s>>>(neg, c);
        SBW_CUDA_TRY(cudaGetLastError());
    }
    // enough CTAs to fill the machine, never more than the largest possible number of tile pairs
    const int64_t max_items = ((n / 2 + kRocPosTile) / kRocPosTile) * ((n / 2 + kRocNegTile) / kRocNegTile) + 1;
    const int64_t cap = 4LL * di.sm_count;
    const unsigned grid = static_cast<unsigned>(max_items < cap ? max_items : cap);
    pairs_kernel<<<grid, kRocThreads, 0, s>>>(pos, neg, c, out_auc, out_stats);
    SBW_CUDA_TRY(cudaGetLastError());
    return SBW_OK;
}

extern "C" int sbw_roc_auc_batched(const double *z, const uint8_t *labels, const int64_t *offsets, int64_t M,
                                   double *out_auc, uint64_t *out_stats, void *stream) {
    using namespace sbw;
    if (M < 0) return SBW_ERR_INVALID_ARG;
    if (M == 0) return SBW_OK;
    if (!offsets || !out_auc || !z || !labels) return SBW_ERR_INVALID_ARG;
    DeviceInfo di;
    if (int rc = current_device_info(&di)) return rc;
    const int64_t cap = 2LL * di.sm_count;
    batched_kernel<<<static_cast<unsigned>(M < cap ? M : cap), kRocSortThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        z, labels, offsets, M, out_auc, out_stats);
    SBW_CUDA_TRY(cudaGetLastError());
    return SBW_OK;
}
