// sbw_roc_auc: area under the ROC curve of detection scores (Section 4.4 of the paper) as the
// exact pair statistic  AUC = (2 #{z_pos > z_neg} + #{z_pos == z_neg}) / (2 n_pos n_neg).
//
// Two kernels.  split_kernel copies the scores of each class into its own dense array (slot
// allocation by one atomic per warp and class; the order inside a class does not matter to a
// count) and drops NaNs.  pairs_kernel walks the (positive tile) x (negative tile) grid with a
// persistent set of CTAs: every thread keeps kRocPerThread positives in registers, the negatives
// of the tile sit in shared memory and are read as warp-wide broadcasts, so a pair costs two
// fp64 compares and two predicated adds.  Counts are integers, so the result does not depend on
// the order of anything; the last CTA to finish (atomic ticket) forms the quotient.
#include "sbw_common.cuh"

namespace sbw {
namespace {

constexpr int kRocThreads = 256;
constexpr int kRocPerThread = 4;
constexpr int kRocPosTile = kRocThreads * kRocPerThread;   // positives per tile
constexpr int kRocNegTile = 1024;                          // negatives per tile (8 KiB of shared memory)

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

__global__ void __launch_bounds__(kRocThreads)
pairs_kernel(const double *pos, const double *neg, RocCounters *c, double *out_auc, uint64_t *out_stats) {
    __shared__ double sneg[kRocNegTile];
    __shared__ unsigned long long red[2][kRocThreads / 32];
    __shared__ bool last;
    const unsigned long long n_pos = c->n_pos, n_neg = c->n_neg;   // written by the previous kernel
    const unsigned long long tiles_p = (n_pos + kRocPosTile - 1) / kRocPosTile;
    const unsigned long long tiles_n = (n_neg + kRocNegTile - 1) / kRocNegTile;
    const double nan = __longlong_as_double(0x7ff8000000000000LL);   // compares false both ways: padding

    unsigned long long greater = 0, equal = 0;
    for (unsigned long long item = blockIdx.x; item < tiles_p * tiles_n; item += gridDim.x) {
        const unsigned long long tp = item / tiles_n, tn = item % tiles_n;
        double p[kRocPerThread];
#pragma unroll
        for (int r = 0; r < kRocPerThread; ++r) {
            const unsigned long long i = tp * kRocPosTile + r * kRocThreads + threadIdx.x;
            p[r] = i < n_pos ? pos[i] : nan;
        }
        __syncthreads();                                 // the previous tile's readers are done
        for (int j = threadIdx.x; j < kRocNegTile; j += kRocThreads) {
            const unsigned long long i = tn * kRocNegTile + j;
            sneg[j] = i < n_neg ? neg[i] : nan;
        }
        __syncthreads();
        unsigned g = 0, e = 0;                           // at most kRocPerThread * kRocNegTile each
#pragma unroll 8
        for (int j = 0; j < kRocNegTile; ++j) {
            const double q = sneg[j];
#pragma unroll
            for (int r = 0; r < kRocPerThread; ++r) {
                g += p[r] > q ? 1u : 0u;
                e += p[r] == q ? 1u : 0u;
            }
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
    // enough CTAs to fill the machine, never more than the largest possible number of tile pairs
    const int64_t max_items = ((n / 2 + kRocPosTile) / kRocPosTile) * ((n / 2 + kRocNegTile) / kRocNegTile) + 1;
    const int64_t cap = 4LL * di.sm_count;
    const unsigned grid = static_cast<unsigned>(max_items < cap ? max_items : cap);
    pairs_kernel<<<grid, kRocThreads, 0, s>>>(pos, neg, c, out_auc, out_stats);
    SBW_CUDA_TRY(cudaGetLastError());
    return SBW_OK;
}
