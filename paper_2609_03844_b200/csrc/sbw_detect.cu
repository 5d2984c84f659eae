// sbw_detect: batch detection -- one membership test per generated token (Section 2.2 of the
// paper, "Detection"), green counts by warp ballot + popcount, z-score of Eq. 5 in fp64.
//
// One warp scores one sequence.  Lanes read consecutive tokens (coalesced 128-byte requests;
// the W predecessors of a token come from the same cache lines), derive the token's seed, run
// one Philox evaluation, and the warp adds popc(ballot(green)) to a warp-uniform counter, so no
// per-lane reduction is needed at the end.  Each lane carries kDetectIlp independent tokens per
// trip, hashed round by round so that the dependent multiply/xor chains overlap; full trips run
// without masks and only the last, ragged trip of a sequence is predicated.
// Sequence starts come from a caller-supplied offsets array or from a two-kernel exclusive scan
// of the lengths into the workspace.
#include "sbw_common.cuh"
#include "sbw_hash.cuh"

namespace sbw {
namespace {

constexpr int kDetectThreads = 128;  // 4 sequences per block: short blocks keep the tail small
constexpr int kDetectIlp = 4;        // tokens per lane in a full trip
constexpr int kScanThreads = 256;
constexpr int kScanItems = 4;        // lengths per thread
constexpr int kScanTile = kScanThreads * kScanItems;

struct DetectArgs {
    const int32_t *tokens;
    const int32_t *lengths;
    const int64_t *offsets;
    int64_t N, total_tokens;
    int W;
    uint64_t key;
    uint32_t thr_m1;
    double gamma;
    int32_t *out_counts;
    int32_t *out_T;
    double *out_z;
    uint32_t *out_bits;   // nullable: per-token green bits, see sbw_detect_bits in sbw.h
    Weyl weyl;   // Philox key-schedule increments (see sbw_hash.cuh)
};

__device__ __forceinline__ int64_t clamp_len(int32_t l) { return l > 0 ? l : 0; }

// Eq. 5, every operation rounded separately; 0 where it is 0/0.
__device__ __forceinline__ double zscore(int G, int T, double gamma) {
    if (T <= 0) return 0.0;
    const double num = __dsub_rn(static_cast<double>(G), __dmul_rn(gamma, static_cast<double>(T)));
    const double var = __dmul_rn(__dmul_rn(static_cast<double>(T), gamma), __dsub_rn(1.0, gamma));
    return __ddiv_rn(num, __dsqrt_rn(var));
}

// ---- exclusive scan of the lengths: tile sums, then per-tile scan with a look-back sum ----
__global__ void __launch_bounds__(kScanThreads)
scan_tile_sums(const int32_t *lengths, int64_t N, int64_t *tile_sums) {
    __shared__ int64_t warp_sums[kScanThreads / 32];
    const int64_t base = static_cast<int64_t>(blockIdx.x) * kScanTile;
    int64_t s = 0;
#pragma unroll
    for (int i = 0; i < kScanItems; ++i) {
        const int64_t idx = base + i * kScanThreads + threadIdx.x;
        if (idx < N) s += clamp_len(lengths[idx]);
    }
    for (int d = 16; d > 0; d >>= 1) s += __shfl_down_sync(0xffffffffu, s, d);
    if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        int64_t t = 0;
        for (int w = 0; w < kScanThreads / 32; ++w) t += warp_sums[w];
        tile_sums[blockIdx.x] = t;
    }
}

__global__ void __launch_bounds__(kScanThreads)
scan_offsets(const int32_t *lengths, int64_t N, const int64_t *tile_sums, int64_t *offsets) {
    __shared__ int64_t warp_sums[kScanThreads / 32];
    __shared__ int64_t tile_base;
    // sum of all earlier tiles
    int64_t s = 0;
    for (int64_t t = threadIdx.x; t < blockIdx.x; t += kScanThreads) s += tile_sums[t];
    for (int d = 16; d > 0; d >>= 1) s += __shfl_down_sync(0xffffffffu, s, d);
    if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        int64_t t = 0;
        for (int w = 0; w < kScanThreads / 32; ++w) t += warp_sums[w];
        tile_base = t;
    }
    __syncthreads();
    // each thread owns kScanItems consecutive lengths
    const int64_t first = static_cast<int64_t>(blockIdx.x) * kScanTile + threadIdx.x * kScanItems;
    int64_t v[kScanItems];
    int64_t mine = 0;
#pragma unroll
    for (int i = 0; i < kScanItems; ++i) {
        v[i] = (first + i < N) ? clamp_len(lengths[first + i]) : 0;
        mine += v[i];
    }
    // inclusive scan of `mine` over the block
    int64_t incl = mine;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int d = 1; d < 32; d <<= 1) {
        const int64_t up = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += up;
    }
    __syncthreads();
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    int64_t before = tile_base;
    for (int w = 0; w < warp; ++w) before += warp_sums[w];
    int64_t run = before + incl - mine;
#pragma unroll
    for (int i = 0; i < kScanItems; ++i) {
        if (first + i < N) offsets[first + i] = run;
        run += v[i];
        if (first + i == N - 1) offsets[N] = run;
    }
}

// ---- the detector ----
// A trip covers the kDetectIlp * 32 positions base + u*32 + lane (u = 0..kDetectIlp-1) of one
// sequence.  TAIL = false: every position is inside the sequence, no masking.  WIDTH > 0 fixes the
// context width at compile time (loops unrolled), WIDTH = 0 reads it from the arguments.
// load_trip reads the tokens and derives their seeds; score_trip hashes them and counts.
template <int SCHEME, int WIDTH, bool TAIL, int ILP = kDetectIlp>
__device__ __forceinline__ void load_trip(const DetectArgs &a, const int32_t *tok, int base, int len, int lane,
                                          uint32_t (&v)[ILP], uint64_t (&r)[ILP], bool (&valid)[ILP]) {
    const int width = WIDTH > 0 ? WIDTH : a.W;
#pragma unroll
    for (int u = 0; u < ILP; ++u) {
        const int t = base + u * 32 + lane;
        valid[u] = !TAIL || static_cast<unsigned>(t) < static_cast<unsigned>(len);
        const int ts = valid[u] ? t : width;      // any readable position; its result is dropped
        (void)SBW_CHECKED(ts >= width && ts < len && (tok - a.tokens) + ts < a.total_tokens && (tok - a.tokens) + ts - width >= 0,
                          SBW_SITE_DETECT_TOKEN);
        v[u] = static_cast<uint32_t>(tok[ts]);
        if constexpr (SCHEME == SBW_SCHEME_CONTEXT) {
            if constexpr (WIDTH == 1) {
                r[u] = a.key * static_cast<uint64_t>(static_cast<uint32_t>(tok[ts - 1]));
            } else {
                uint64_t sigma = 0;
#pragma unroll
                for (int i = 1; i <= (WIDTH > 0 ? WIDTH : SBW_MAX_CTX_WIDTH); ++i)
                    if (i <= width) sigma += static_cast<uint32_t>(tok[ts - i]);
                r[u] = a.key * sigma;
            }
        }
    }
    if constexpr (SCHEME == SBW_SCHEME_SELFSALT) {
        // Every id of the trip is hashed once: a position's context hashes are its neighbours' own
        // hashes, fetched by shuffles (position t - i sits i lanes down, or at the top of the group
        // of 32 before; the group before the trip's first is hashed for the purpose).  A lane whose
        // position is valid only draws on lanes with smaller, hence valid, positions.
        uint32_t jv[ILP + 1];                       // jv[u + 1]: group u; jv[0]: the 32 positions before the trip
        const int before = base - 32 + lane;
        jv[0] = jenkins(static_cast<uint32_t>(tok[before > 0 ? before : 0]));
#pragma unroll
        for (int u = 0; u < ILP; ++u) jv[u + 1] = jenkins(v[u]);
#pragma unroll
        for (int u = 0; u < ILP; ++u) {
            uint32_t jmin = 0xFFFFFFFFu;
#pragma unroll
            for (int i = 1; i <= (WIDTH > 0 ? WIDTH : SBW_MAX_CTX_WIDTH); ++i) {
                if (i <= width) {
                    // lanes 32 - i .. 31 hand over the group before, the others this group
                    const uint32_t give = lane >= 32 - i ? jv[u] : jv[u + 1];
                    jmin = min(jmin, __shfl_sync(0xffffffffu, give, (lane - i) & 31));
                }
            }
            const uint64_t prod = static_cast<uint64_t>(jv[u + 1]) * min(jv[u + 1], jmin);
            r[u] = a.key * prod;
        }
    }
}

// A trip of ILP * 32 positions: ILP = 4 for the bulk of a sequence, 2 and 1 for what is left at its
// end, so that at most 31 lanes idle per sequence.  BITS: also keep the ballots (sbw_detect_bits).
template <int SCHEME, int WIDTH, bool TAIL, bool BITS, int ILP = kDetectIlp>
__device__ __forceinline__ int score_trip(const DetectArgs &a, const int32_t *tok, int base, int len,
                                          int lane, uint32_t *bits) {
    const int width = WIDTH > 0 ? WIDTH : a.W;
    uint32_t v[ILP];
    uint64_t r[ILP];
    bool valid[ILP];
    load_trip<SCHEME, WIDTH, TAIL, ILP>(a, tok, base, len, lane, v, r, valid);
    uint32_t x[ILP];
    philox_word0_n<ILP>(v, r, x, a.weyl);
    int count = 0;
#pragma unroll
    for (int u = 0; u < ILP; ++u) {
        const unsigned greens = __ballot_sync(0xffffffffu, valid[u] && x[u] <= a.thr_m1);
        count += __popc(greens);
        // the ballot is the bit mask of 32 consecutive scored positions: keep it if asked to
        if (BITS && lane == 0 && (!TAIL || base + u * 32 < len)) bits[((base - width) >> 5) + u] = greens;
    }
    return count;
}

// All scored positions of one sequence from `base` on, by one warp.
template <int SCHEME, int WIDTH, bool BITS>
__device__ __forceinline__ int score_sequence(const DetectArgs &a, const int32_t *tok, int base, int len, int lane,
                                              uint32_t *bits) {
    constexpr int kTrip = 32 * kDetectIlp;
    int count = 0;
    // written as differences so that lengths near 2^31 cannot overflow the position
    for (; len - base >= kTrip; base += kTrip)
        count += score_trip<SCHEME, WIDTH, false, BITS>(a, tok, base, len, lane, bits);
    if (len - base >= 64) {
        count += score_trip<SCHEME, WIDTH, false, BITS, 2>(a, tok, base, len, lane, bits);
        base += 64;
    }
    if (len - base >= 32) {
        count += score_trip<SCHEME, WIDTH, false, BITS, 1>(a, tok, base, len, lane, bits);
        base += 32;
    }
    if (base < len) count += score_trip<SCHEME, WIDTH, true, BITS, 1>(a, tok, base, len, lane, bits);
    return count;
}

template <int SCHEME, int WIDTH, bool BITS>
__global__ void __launch_bounds__(kDetectThreads)
detect_kernel(const DetectArgs a) {
    const int lane = threadIdx.x & 31;
    const int64_t seq = static_cast<int64_t>(blockIdx.x) * (kDetectThreads / 32) + (threadIdx.x >> 5);
    if (seq >= a.N) return;
    const int64_t off = a.offsets[seq];
    int64_t L = clamp_len(a.lengths[seq]);
    if (off < 0 || off >= a.total_tokens) L = 0;
    else if (off + L > a.total_tokens) L = a.total_tokens - off;
    const int width = WIDTH > 0 ? WIDTH : a.W;
    const int32_t *tok = a.tokens + off;
    const int len = static_cast<int>(L);
    uint32_t *bits = BITS ? a.out_bits + (off >> 5) + 2 * seq : nullptr;
    const int count = len > width ? score_sequence<SCHEME, WIDTH, BITS>(a, tok, width, len, lane, bits) : 0;

    if (lane == 0) {
        const int T = len > width ? len - width : 0;
        (void)SBW_CHECKED(seq >= 0 && seq < a.N && count >= 0 && count <= T, SBW_SITE_DETECT_OUTPUT);
        a.out_counts[seq] = count;
        if (a.out_T) a.out_T[seq] = T;
        a.out_z[seq] = zscore(count, T, a.gamma);
    }
}

// Few sequences: one CTA per sequence, its warps taking the trips in turn, so that a handful of
// long texts still spreads over the GPU (a warp per sequence would walk each text alone).
template <int SCHEME, int WIDTH, bool BITS>
__global__ void __launch_bounds__(1024)
detect_wide_kernel(const DetectArgs a) {
    __shared__ int sh_count[32];
    __shared__ long long sh_part[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int64_t seq = blockIdx.x;
    int64_t off;
    if (a.offsets) {
        off = a.offsets[seq];
    } else {
        // no offsets given and few sequences: the CTA adds up the lengths before its own
        long long part = 0;
        for (int64_t i = threadIdx.x; i < seq; i += blockDim.x) part += clamp_len(a.lengths[i]);
        for (int d = 16; d > 0; d >>= 1) part += __shfl_xor_sync(0xffffffffu, part, d);
        if (lane == 0) sh_part[warp] = part;
        __syncthreads();
        off = 0;
        for (int w = 0; w < nwarps; ++w) off += sh_part[w];
    }
    int64_t L = clamp_len(a.lengths[seq]);
    if (off < 0 || off >= a.total_tokens) L = 0;
    else if (off + L > a.total_tokens) L = a.total_tokens - off;
    const int width = WIDTH > 0 ? WIDTH : a.W;
    const int32_t *tok = a.tokens + off;
    const int len = static_cast<int>(L);
    constexpr int kTrip = 32 * kDetectIlp;
    uint32_t *bits = BITS ? a.out_bits + (off >> 5) + 2 * seq : nullptr;

    int count = 0;
    const int full = len > width ? (len - width) / kTrip : 0;         // unmasked trips
    for (int i = warp; i < full; i += nwarps)
        count += score_trip<SCHEME, WIDTH, false, BITS>(a, tok, width + i * kTrip, len, lane, bits);
    const int tail_base = width + full * kTrip;
    if (tail_base < len && warp == full % nwarps)
        count += score_trip<SCHEME, WIDTH, true, BITS>(a, tok, tail_base, len, lane, bits);
    if (lane == 0) sh_count[warp] = count;
    __syncthreads();
    if (threadIdx.x == 0) {
        int total = 0;
        for (int w = 0; w < nwarps; ++w) total += sh_count[w];
        const int T = len > width ? len - width : 0;
        a.out_counts[seq] = total;
        if (a.out_T) a.out_T[seq] = T;
        a.out_z[seq] = zscore(total, T, a.gamma);
    }
}

// One warp per sequence fills the GPU from a few thousand sequences on; below that a CTA per
// sequence, the wider the fewer there are.  Returns the CTA size, or 0 for a warp per sequence.
inline int wide_threads(int64_t N, int sm_count) {
    const int64_t resident_warps = static_cast<int64_t>(sm_count) * 64;
    return N * 32 <= resident_warps ? 1024 : N * 16 <= resident_warps ? 512 : N * 8 <= resident_warps ? 256 : 0;
}

template <int SCHEME, bool BITS>
cudaError_t launch_detect(const DetectArgs &a, int sm_count, cudaStream_t s) {
    const int wide = wide_threads(a.N, sm_count);
    if (wide) {
        const unsigned grid = static_cast<unsigned>(a.N);
        switch (a.W) {
            case 1: detect_wide_kernel<SCHEME, 1, BITS><<<grid, wide, 0, s>>>(a); break;
            case 4: detect_wide_kernel<SCHEME, 4, BITS><<<grid, wide, 0, s>>>(a); break;
            default: detect_wide_kernel<SCHEME, 0, BITS><<<grid, wide, 0, s>>>(a); break;
        }
        return cudaGetLastError();
    }
    const unsigned grid = static_cast<unsigned>((a.N + kDetectThreads / 32 - 1) / (kDetectThreads / 32));
    switch (a.W) {
        case 1: detect_kernel<SCHEME, 1, BITS><<<grid, kDetectThreads, 0, s>>>(a); break;
        case 4: detect_kernel<SCHEME, 4, BITS><<<grid, kDetectThreads, 0, s>>>(a); break;
        default: detect_kernel<SCHEME, 0, BITS><<<grid, kDetectThreads, 0, s>>>(a); break;
    }
    return cudaGetLastError();
}

}  // namespace
}  // namespace sbw

extern "C" size_t sbw_detect_workspace_bytes(int64_t N) {
    if (N <= 0) return 0;
    const size_t tiles = static_cast<size_t>((N + sbw::kScanTile - 1) / sbw::kScanTile);
    return sbw::align_up((static_cast<size_t>(N) + 1) * sizeof(int64_t), 256) +
           sbw::align_up(tiles * sizeof(int64_t), 256);
}

namespace sbw {
namespace {
// Exclusive scan of the lengths into the start of `workspace` (int64[N + 1], then the tile sums).
int scan_lengths(const int32_t *lengths, int64_t N, void *workspace, int64_t **out_offsets, cudaStream_t s) {
    int64_t *ws_offsets = static_cast<int64_t *>(workspace);
    int64_t *tile_sums = reinterpret_cast<int64_t *>(
        static_cast<char *>(workspace) + align_up((static_cast<size_t>(N) + 1) * sizeof(int64_t), 256));
    const unsigned tiles = static_cast<unsigned>((N + kScanTile - 1) / kScanTile);
    if (tiles > 1) {                                 // a single tile has no earlier tiles to add up
        scan_tile_sums<<<tiles, kScanThreads, 0, s>>>(lengths, N, tile_sums);
        SBW_CUDA_TRY(cudaGetLastError());
    }
    scan_offsets<<<tiles, kScanThreads, 0, s>>>(lengths, N, tile_sums, ws_offsets);
    SBW_CUDA_TRY(cudaGetLastError());
    *out_offsets = ws_offsets;
    return SBW_OK;
}

int detect_impl(const int32_t *tokens, const int32_t *lengths, const int64_t *offsets, int64_t N,
                int64_t total_tokens, int ctx_width, uint64_t key, double gamma, int scheme,
                int32_t *out_counts, int32_t *out_T, double *out_z, uint32_t *out_bits, void *workspace,
                size_t workspace_bytes, void *stream) {
    if (!valid_common(SBW_DTYPE_F32, ctx_width, gamma, scheme)) return SBW_ERR_INVALID_ARG;
    if (N < 0 || total_tokens < 0) return SBW_ERR_INVALID_ARG;
    if (N == 0) return SBW_OK;
    if (N > (int64_t(1) << 31) * (kDetectThreads / 32) - 1) return SBW_ERR_UNSUPPORTED;
    if (!lengths || !out_counts || !out_z) return SBW_ERR_INVALID_ARG;
    if (!tokens && total_tokens > 0) return SBW_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    DetectArgs a;
    a.tokens = tokens;
    a.lengths = lengths;
    a.offsets = offsets;
    a.N = N;
    a.total_tokens = total_tokens;
    a.W = ctx_width;
    a.key = key;
    a.thr_m1 = threshold_minus_one(gamma);
    a.gamma = gamma;
    a.out_counts = out_counts;
    a.out_T = out_T;
    a.out_z = out_z;
    a.out_bits = out_bits;
    a.weyl = make_weyl();

    if (!offsets) {       // host-side validation first: it must not depend on a device being present
        const size_t need = sbw_detect_workspace_bytes(N);
        if (!workspace || workspace_bytes < need || reinterpret_cast<uintptr_t>(workspace) % 256 != 0)
            return SBW_ERR_WORKSPACE;
    }
    DeviceInfo di;
    if (int rc = current_device_info(&di)) return rc;
    if (!offsets) {
        // the plain detector on few sequences finds its offsets itself (one launch instead of two);
        // with stored bits the offsets stay in the workspace for the calls that read the bits
        if (out_bits || wide_threads(N, di.sm_count) == 0) {
            int64_t *ws_offsets = nullptr;
            const int rc = scan_lengths(lengths, N, workspace, &ws_offsets, s);
            if (rc != SBW_OK) return rc;
            a.offsets = ws_offsets;
        }
    }
    cudaError_t err;
    if (out_bits) {
        err = scheme == SBW_SCHEME_CONTEXT ? launch_detect<SBW_SCHEME_CONTEXT, true>(a, di.sm_count, s)
                                           : launch_detect<SBW_SCHEME_SELFSALT, true>(a, di.sm_count, s);
    } else {
        err = scheme == SBW_SCHEME_CONTEXT ? launch_detect<SBW_SCHEME_CONTEXT, false>(a, di.sm_count, s)
                                           : launch_detect<SBW_SCHEME_SELFSALT, false>(a, di.sm_count, s);
    }
    SBW_CUDA_TRY(err);
    return SBW_OK;
}

// ---- windowed detection on the stored green bits ----
// One warp per sequence.  First the exclusive prefix counts of the sequence's bit words (32 words
// per trip, warp scan, running carry), kept in `prefix` with the layout of the bits; then every
// lane evaluates window starts lane, lane + 32, ...: greens in [start, start + w) is the
// difference of two prefix counts, each one word load, one prefix load and a masked popcount.
__device__ __forceinline__ int greens_before(const uint32_t *bits, const uint32_t *prefix, int p) {
    const int word = p >> 5, bit = p & 31;
    return static_cast<int>(prefix[word]) + (bit ? __popc(bits[word] & ((1u << bit) - 1u)) : 0);
}

__global__ void __launch_bounds__(kDetectThreads)
window_kernel(const uint32_t *all_bits, uint32_t *all_prefix, const int32_t *lengths, const int64_t *offsets,
              int64_t N, int64_t total_tokens, int W, int window, double gamma, int32_t *out_count,
              int32_t *out_start, double *out_z) {
    const int lane = threadIdx.x & 31;
    const int64_t seq = static_cast<int64_t>(blockIdx.x) * (kDetectThreads / 32) + (threadIdx.x >> 5);
    if (seq >= N) return;
    const int64_t off = offsets[seq];
    int64_t L = clamp_len(lengths[seq]);
    if (off < 0 || off >= total_tokens) L = 0;
    else if (off + L > total_tokens) L = total_tokens - off;
    const int T = L > W ? static_cast<int>(L - W) : 0;
    const uint32_t *bits = all_bits + (off >> 5) + 2 * seq;
    uint32_t *prefix = all_prefix + (off >> 5) + 2 * seq;
    const int nwords = (T + 31) >> 5;
    // the region of a sequence has a word to spare: prefix[nwords] is written too, so that a
    // window ending exactly at T needs no special case
    unsigned carry = 0;
    for (int k0 = 0; k0 <= nwords; k0 += 32) {
        const int k = k0 + lane;
        const unsigned c = k < nwords ? __popc(bits[k]) : 0u;
        unsigned incl = c;
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        if (k <= nwords) prefix[k] = carry + incl - c;
        carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    __syncwarp();
    const int w = window < T ? window : T;
    int best = 0, best_start = 0;
    if (w > 0) {
        for (int start = lane; start + w <= T; start += 32) {
            const int g = greens_before(bits, prefix, start + w) - greens_before(bits, prefix, start);
            if (g > best) { best = g; best_start = start; }       // strict: earliest start per lane
        }
        for (int d = 16; d > 0; d >>= 1) {
            const int og = __shfl_down_sync(0xffffffffu, best, d);
            const int os = __shfl_down_sync(0xffffffffu, best_start, d);
            if (og > best || (og == best && os < best_start)) { best = og; best_start = os; }
        }
    }
    if (lane == 0) {
        out_count[seq] = best;
        out_start[seq] = best > 0 ? best_start : 0;
        out_z[seq] = zscore(best, w, gamma);
    }
}


// ---- detection on truncated text: popcount of the first kept bits ----
__global__ void __launch_bounds__(kDetectThreads)
prefix_kernel(const uint32_t *all_bits, const int32_t *lengths, const int64_t *offsets, const int32_t *keep,
              int64_t N, int64_t total_tokens, int W, double gamma, int32_t *out_count, int32_t *out_T,
              double *out_z) {
    const int lane = threadIdx.x & 31;
    const int64_t seq = static_cast<int64_t>(blockIdx.x) * (kDetectThreads / 32) + (threadIdx.x >> 5);
    if (seq >= N) return;
    const int64_t off = offsets[seq];
    int64_t L = clamp_len(lengths[seq]);
    if (off < 0 || off >= total_tokens) L = 0;
    else if (off + L > total_tokens) L = total_tokens - off;
    int64_t K = clamp_len(keep[seq]);
    if (K > L) K = L;
    const int T = K > W ? static_cast<int>(K - W) : 0;
    const uint32_t *bits = all_bits + (off >> 5) + 2 * seq;
    const int nfull = T >> 5, rem = T & 31;
    int count = 0;
    for (int k = lane; k < nfull; k += 32) count += __popc(bits[k]);
    if (lane == 0 && rem) count += __popc(bits[nfull] & ((1u << rem) - 1u));
    for (int d = 16; d > 0; d >>= 1) count += __shfl_down_sync(0xffffffffu, count, d);
    if (lane == 0) {
        out_count[seq] = count;
        if (out_T) out_T[seq] = T;
        out_z[seq] = zscore(count, T, gamma);
    }
}

// ---- detection over the distinct (context, token) tuples of a sequence ----
// One warp per sequence, as in detect_kernel, plus a hash set of the tuples seen so far: open
// addressing with linear probing over a power-of-two table of token positions (0 = empty; scored
// positions start at W >= 1).  A lane claims a slot with one compare-and-swap; a lane that finds
// the slot taken compares its tuple with the tuple at the stored position and either stops
// (duplicate) or probes on.  Entries are never removed, so concurrent inserts by the lanes of
// the warp are safe: whichever lane claims a tuple first, every other occurrence meets it on its
// probe path.  Which occurrence represents a tuple does not matter -- equal tuples have equal
// green bits -- so counts are deterministic.  The table lives in shared memory (kUniqueSlots
// slots per warp) for sequences with at most kUniqueSmemMaxT scored tokens, otherwise in the
// caller's workspace at 4 * offset (the smallest power of two >= 2T is below 4T slots).  The
// compare-and-swap insert below serves the workspace tables; shared-memory tables use the
// atomic-free scheme of insert_trip_shared.
constexpr int kUniqueSlots = 4096;
constexpr int kUniqueSmemMaxT = 1536;
static_assert(kUniqueSmemMaxT + SBW_MAX_CTX_WIDTH < 2048, "positions on the shared path must fit 11 bits");

template <int WIDTH>
__device__ __forceinline__ uint32_t tuple_hash(const int32_t *tok, int t, int width) {
    uint32_t h = static_cast<uint32_t>(tok[t]) * 0x9E3779B1u;
#pragma unroll
    for (int i = 1; i <= (WIDTH > 0 ? WIDTH : SBW_MAX_CTX_WIDTH); ++i)
        if (i <= width) h = (h + static_cast<uint32_t>(tok[t - i])) * 0x85EBCA77u;
    return (h ^ (h >> 15)) * 0x9E3779B1u;
}

template <int WIDTH>
__device__ __forceinline__ bool same_tuple(const int32_t *tok, int p, int q, int width) {
    bool same = true;
#pragma unroll
    for (int i = 0; i <= (WIDTH > 0 ? WIDTH : SBW_MAX_CTX_WIDTH); ++i)
        if (i <= width) same = same && tok[p - i] == tok[q - i];
    return same;
}

// true if position t is the one that enters its tuple into the set
template <int WIDTH>
__device__ __forceinline__ bool insert_tuple(uint32_t *table, uint32_t mask, int shift, const int32_t *tok,
                                             int t, int width) {
    uint32_t slot = tuple_hash<WIDTH>(tok, t, width) >> shift;
    for (uint32_t n = 0; n <= mask; ++n) {           // bounded: the table always has a free slot
        const uint32_t prev = atomicCAS(&table[slot], 0u, static_cast<uint32_t>(t));
        if (prev == 0u) return true;
        if (same_tuple<WIDTH>(tok, static_cast<int>(prev), t, width)) return false;
        slot = (slot + 1u) & mask;
    }
    return true;
}

// The shared-memory table is filled without atomics.  An entry is 16 bits, (fingerprint << 11) |
// position: the low 5 bits of the tuple's hash and the token position (below 2048 on this path),
// so most foreign entries are told apart without touching the tokens, and kUniqueSlots of them
// keep the load factor at or below 3/8.  The warp inserts the positions of
// a trip in rounds of three phases separated by __syncwarp: (1) every pending position walks its
// probe path over the table as the last round left it, until it meets its own tuple (duplicate,
// done) or an empty slot; (2) those at an empty slot store their entry -- several may hit the
// same slot, one store lands; (3) each reads the slot back: the one that finds its own entry has
// entered the tuple, the others stay pending and meet the winner in the next round.  Equal
// tuples of one trip walk the same path over the same table state, so they always collide in
// phase 2 and exactly one of them wins.
constexpr int kUniquePosBits = 11;

template <int WIDTH, bool TAIL>
__device__ __forceinline__ void insert_trip_shared(volatile uint16_t *table, uint32_t mask, int shift,
                                                   const int32_t *tok, int base, int lane, int width,
                                                   bool (&first)[kDetectIlp]) {
    uint32_t slot[kDetectIlp], mine[kDetectIlp];
    bool pending[kDetectIlp], writer[kDetectIlp];
#pragma unroll
    for (int u = 0; u < kDetectIlp; ++u) {
        const int t = base + u * 32 + lane;
        pending[u] = first[u];                           // on entry: the position exists
        const uint32_t h = tuple_hash<WIDTH>(tok, pending[u] ? t : width, width);
        slot[u] = h >> shift;
        mine[u] = ((h << kUniquePosBits) | static_cast<uint32_t>(t)) & 0xFFFFu;
    }
    for (int round = 0; round < 32 * kDetectIlp + 1; ++round) {   // every round settles a position
#pragma unroll
        for (int u = 0; u < kDetectIlp; ++u) {
            writer[u] = false;
            if (!pending[u]) continue;
            const int t = base + u * 32 + lane;
            for (uint32_t n = 0; n <= mask; ++n) {       // bounded: the table always has a free slot
                const uint32_t e = table[slot[u]];
                if (e == 0u) {
                    writer[u] = true;
                    break;
                }
                if (((e ^ mine[u]) >> kUniquePosBits) == 0u &&
                    same_tuple<WIDTH>(tok, static_cast<int>(e & ((1u << kUniquePosBits) - 1u)), t, width)) {
                    pending[u] = false;
                    first[u] = false;
                    break;
                }
                slot[u] = (slot[u] + 1u) & mask;
            }
        }
        __syncwarp();
#pragma unroll
        for (int u = 0; u < kDetectIlp; ++u)
            if (writer[u]) table[slot[u]] = static_cast<uint16_t>(mine[u]);
        __syncwarp();
        bool more = false;
#pragma unroll
        for (int u = 0; u < kDetectIlp; ++u) {
            if (writer[u] && table[slot[u]] == mine[u]) pending[u] = false;
            more = more || pending[u];
        }
        if (!__any_sync(0xffffffffu, more)) break;
    }
}

template <int SCHEME, int WIDTH, bool TAIL, bool SHARED>
__device__ __forceinline__ void unique_trip(const DetectArgs &a, const int32_t *tok, int base, int len, int lane,
                                            void *table, uint32_t mask, int shift, int &count, int &distinct) {
    const int width = WIDTH > 0 ? WIDTH : a.W;
    uint32_t v[kDetectIlp];
    uint64_t r[kDetectIlp];
    bool first[kDetectIlp];
    load_trip<SCHEME, WIDTH, TAIL>(a, tok, base, len, lane, v, r, first);
    if constexpr (SHARED) {
        insert_trip_shared<WIDTH, TAIL>(static_cast<uint16_t *>(table), mask, shift, tok, base, lane, width, first);
    } else {
#pragma unroll
        for (int u = 0; u < kDetectIlp; ++u)
            first[u] = first[u] && insert_tuple<WIDTH>(static_cast<uint32_t *>(table), mask, shift, tok,
                                                       base + u * 32 + lane, width);
    }
    uint32_t x[kDetectIlp];
    philox_word0_n<kDetectIlp>(v, r, x, a.weyl);
#pragma unroll
    for (int u = 0; u < kDetectIlp; ++u) {
        distinct += __popc(__ballot_sync(0xffffffffu, first[u]));
        count += __popc(__ballot_sync(0xffffffffu, first[u] && x[u] <= a.thr_m1));
    }
}

template <int SCHEME, int WIDTH, bool SHARED>
__device__ __forceinline__ void unique_sequence(const DetectArgs &a, const int32_t *tok, int len, int lane,
                                                void *table, uint32_t slots, int &count, int &distinct) {
    const int width = WIDTH > 0 ? WIDTH : a.W;
    constexpr int kTrip = 32 * kDetectIlp;
    const uint32_t mask = slots - 1u;
    const int shift = __clz(slots) + 1;               // 32 - log2(slots)
    const uint32_t bytes = slots * (SHARED ? 2u : 4u);   // a multiple of 128 (slots >= 64)
    for (uint32_t i = lane * 16u; i < bytes; i += 512u)
        *reinterpret_cast<uint4 *>(static_cast<char *>(table) + i) = make_uint4(0u, 0u, 0u, 0u);
    __syncwarp();
    int base = width;
    for (; len - base >= kTrip; base += kTrip)
        unique_trip<SCHEME, WIDTH, false, SHARED>(a, tok, base, len, lane, table, mask, shift, count, distinct);
    if (base < len)
        unique_trip<SCHEME, WIDTH, true, SHARED>(a, tok, base, len, lane, table, mask, shift, count, distinct);
}

// Persistent warps: sequences differ in length by an order of magnitude and a warp's table pins
// 8 KiB of shared memory, so each warp takes its next sequence from a counter instead of leaving
// its slot idle until the longest sequence of its CTA is done.
template <int SCHEME, int WIDTH>
__global__ void __launch_bounds__(kDetectThreads)
detect_unique_kernel(const DetectArgs a, uint32_t *global_tables, unsigned long long *next_sequence) {
    __shared__ __align__(16) uint16_t smem_tables[kDetectThreads / 32][kUniqueSlots];
    const int lane = threadIdx.x & 31;
    const int width = WIDTH > 0 ? WIDTH : a.W;
    for (;;) {
        unsigned long long ticket = 0;
        if (lane == 0) ticket = atomicAdd(next_sequence, 1ull);
        const int64_t seq = static_cast<int64_t>(__shfl_sync(0xffffffffu, ticket, 0));
        if (seq >= a.N) return;
        const int64_t off = a.offsets[seq];
        int64_t L = clamp_len(a.lengths[seq]);
        if (off < 0 || off >= a.total_tokens) L = 0;
        else if (off + L > a.total_tokens) L = a.total_tokens - off;
        const int32_t *tok = a.tokens + off;
        const int len = static_cast<int>(L);
        const int T = len > width ? len - width : 0;

        int count = 0, distinct = 0;
        uint32_t slots = 64;
        if (T <= kUniqueSmemMaxT) {
            while (slots < 4u * static_cast<uint32_t>(T) && slots < kUniqueSlots) slots <<= 1;
            unique_sequence<SCHEME, WIDTH, true>(a, tok, len, lane, smem_tables[threadIdx.x >> 5], slots, count, distinct);
        } else if (global_tables) {
            while (slots < 2u * static_cast<uint32_t>(T)) slots <<= 1;
            unique_sequence<SCHEME, WIDTH, false>(a, tok, len, lane, global_tables + 4 * off, slots, count, distinct);
        } else {                                     // longer than the caller said any sequence is
            count = distinct = -1;
        }
        if (lane == 0) {
            a.out_counts[seq] = count;
            if (a.out_T) a.out_T[seq] = distinct;
            a.out_z[seq] =
                distinct < 0 ? __longlong_as_double(0x7ff8000000000000LL) : zscore(count, distinct, a.gamma);
        }
        __syncwarp();                                // the table is reused by the next sequence
    }
}

template <int SCHEME>
cudaError_t launch_detect_unique(const DetectArgs &a, uint32_t *tables, unsigned long long *next,
                                 unsigned grid, cudaStream_t s) {
    switch (a.W) {
        case 1: detect_unique_kernel<SCHEME, 1><<<grid, kDetectThreads, 0, s>>>(a, tables, next); break;
        case 4: detect_unique_kernel<SCHEME, 4><<<grid, kDetectThreads, 0, s>>>(a, tables, next); break;
        default: detect_unique_kernel<SCHEME, 0><<<grid, kDetectThreads, 0, s>>>(a, tables, next); break;
    }
    return cudaGetLastError();
}

}  // namespace
}  // namespace sbw

extern "C" int sbw_detect(const int32_t *tokens, const int32_t *lengths, const int64_t *offsets,
                          int64_t N, int64_t total_tokens, int ctx_width, uint64_t key, double gamma,
                          int scheme, int32_t *out_counts, int32_t *out_T, double *out_z,
                          void *workspace, size_t workspace_bytes, void *stream) {
    return sbw::detect_impl(tokens, lengths, offsets, N, total_tokens, ctx_width, key, gamma, scheme,
                            out_counts, out_T, out_z, nullptr, workspace, workspace_bytes, stream);
}

extern "C" size_t sbw_detect_bits_words(int64_t N, int64_t total_tokens) {
    if (N <= 0 || total_tokens < 0) return 0;
    return static_cast<size_t>(total_tokens / 32 + 2 * N + 2);
}

extern "C" int sbw_detect_bits(const int32_t *tokens, const int32_t *lengths, const int64_t *offsets,
                               int64_t N, int64_t total_tokens, int ctx_width, uint64_t key, double gamma,
                               int scheme, int32_t *out_counts, int32_t *out_T, double *out_z,
                               uint32_t *out_bits, void *workspace, size_t workspace_bytes, void *stream) {
    if (N > 0 && !out_bits) return SBW_ERR_INVALID_ARG;
    return sbw::detect_impl(tokens, lengths, offsets, N, total_tokens, ctx_width, key, gamma, scheme,
                            out_counts, out_T, out_z, out_bits, workspace, workspace_bytes, stream);
}

extern "C" int sbw_window_z(const uint32_t *bits, const int32_t *lengths, const int64_t *offsets, int64_t N,
                            int64_t total_tokens, int ctx_width, int64_t window, double gamma,
                            uint32_t *prefix_scratch, int32_t *out_count, int32_t *out_start, double *out_z,
                            void *stream) {
    using namespace sbw;
    if (ctx_width < 1 || ctx_width > SBW_MAX_CTX_WIDTH || !(gamma > 0.0 && gamma < 1.0)) return SBW_ERR_INVALID_ARG;
    if (N < 0 || total_tokens < 0 || window < 1) return SBW_ERR_INVALID_ARG;
    if (N == 0) return SBW_OK;
    if (!bits || !lengths || !offsets || !prefix_scratch || !out_count || !out_start || !out_z)
        return SBW_ERR_INVALID_ARG;
    const int w = window > 0x7fffffffLL ? 0x7fffffff : static_cast<int>(window);
    const unsigned grid = static_cast<unsigned>((N + kDetectThreads / 32 - 1) / (kDetectThreads / 32));
    window_kernel<<<grid, kDetectThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        bits, prefix_scratch, lengths, offsets, N, total_tokens, ctx_width, w, gamma, out_count, out_start, out_z);
    SBW_CUDA_TRY(cudaGetLastError());
    return SBW_OK;
}

extern "C" int sbw_prefix_z(const uint32_t *bits, const int32_t *lengths, const int64_t *offsets,
                            const int32_t *keep, int64_t N, int64_t total_tokens, int ctx_width, double gamma,
                            int32_t *out_counts, int32_t *out_T, double *out_z, void *stream) {
    using namespace sbw;
    if (ctx_width < 1 || ctx_width > SBW_MAX_CTX_WIDTH || !(gamma > 0.0 && gamma < 1.0)) return SBW_ERR_INVALID_ARG;
    if (N < 0 || total_tokens < 0) return SBW_ERR_INVALID_ARG;
    if (N == 0) return SBW_OK;
    if (!bits || !lengths || !offsets || !keep || !out_counts || !out_z) return SBW_ERR_INVALID_ARG;
    const unsigned grid = static_cast<unsigned>((N + kDetectThreads / 32 - 1) / (kDetectThreads / 32));
    prefix_kernel<<<grid, kDetectThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        bits, lengths, offsets, keep, N, total_tokens, ctx_width, gamma, out_counts, out_T, out_z);
    SBW_CUDA_TRY(cudaGetLastError());
    return SBW_OK;
}

extern "C" size_t sbw_detect_unique_workspace_bytes(int64_t N, int64_t total_tokens, int64_t max_length) {
    if (N <= 0 || total_tokens < 0) return 0;
    size_t bytes = sbw::align_up(sbw_detect_workspace_bytes(N), 256) + 256;   // offsets, sequence counter
    if (max_length - 1 > sbw::kUniqueSmemMaxT) bytes += 16 * static_cast<size_t>(total_tokens);
    return bytes;
}

extern "C" int sbw_detect_unique(const int32_t *tokens, const int32_t *lengths, const int64_t *offsets, int64_t N,
                                 int64_t total_tokens, int64_t max_length, int ctx_width, uint64_t key,
                                 double gamma, int scheme, int32_t *out_counts, int32_t *out_T, double *out_z,
                                 void *workspace, size_t workspace_bytes, void *stream) {
    using namespace sbw;
    if (!valid_common(SBW_DTYPE_F32, ctx_width, gamma, scheme)) return SBW_ERR_INVALID_ARG;
    if (N < 0 || total_tokens < 0 || max_length < 0) return SBW_ERR_INVALID_ARG;
    if (N == 0) return SBW_OK;
    if (N > (int64_t(1) << 31) * (kDetectThreads / 32) - 1) return SBW_ERR_UNSUPPORTED;
    if (!lengths || !out_counts || !out_z) return SBW_ERR_INVALID_ARG;
    if (!tokens && total_tokens > 0) return SBW_ERR_INVALID_ARG;
    const size_t need = sbw_detect_unique_workspace_bytes(N, total_tokens, max_length);
    if (!workspace || workspace_bytes < need || reinterpret_cast<uintptr_t>(workspace) % 256 != 0)
        return SBW_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t scan_bytes = align_up(sbw_detect_workspace_bytes(N), 256);
    unsigned long long *next = reinterpret_cast<unsigned long long *>(static_cast<char *>(workspace) + scan_bytes);
    uint32_t *tables = max_length - 1 > kUniqueSmemMaxT
                           ? reinterpret_cast<uint32_t *>(static_cast<char *>(workspace) + scan_bytes + 256)
                           : nullptr;
    DeviceInfo di;
    if (int rc = current_device_info(&di)) return rc;
    SBW_CUDA_TRY(cudaMemsetAsync(next, 0, sizeof(unsigned long long), s));

    DetectArgs a;
    a.tokens = tokens;
    a.lengths = lengths;
    a.offsets = offsets;
    a.N = N;
    a.total_tokens = total_tokens;
    a.W = ctx_width;
    a.key = key;
    a.thr_m1 = threshold_minus_one(gamma);
    a.gamma = gamma;
    a.out_counts = out_counts;
    a.out_T = out_T;
    a.out_z = out_z;
    a.out_bits = nullptr;
    a.weyl = make_weyl();
    if (!offsets) {
        int64_t *ws_offsets = nullptr;
        const int rc = scan_lengths(lengths, N, workspace, &ws_offsets, s);
        if (rc != SBW_OK) return rc;
        a.offsets = ws_offsets;
    }
    const int64_t blocks = (N + kDetectThreads / 32 - 1) / (kDetectThreads / 32);
    const int64_t resident = 8LL * di.sm_count;       // more CTAs than fit: the counter balances them
    const unsigned grid = static_cast<unsigned>(blocks < resident ? blocks : resident);
    SBW_CUDA_TRY(scheme == SBW_SCHEME_CONTEXT ? launch_detect_unique<SBW_SCHEME_CONTEXT>(a, tables, next, grid, s)
                                              : launch_detect_unique<SBW_SCHEME_SELFSALT>(a, tables, next, grid, s));
    return SBW_OK;
}
