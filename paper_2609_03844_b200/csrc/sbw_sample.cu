// sbw_bias_sample: the bias of Eq. 1 + Eq. 2 fused with temperature softmax statistics and
// Gumbel-max sampling, in one read-only pass over the [B, V] logits.  The paper leaves sampling
// to the serving engine; this kernel is the "absorbed into existing logit post-processing" form
// that Section 5.1 points at.
//
// Work layout.  A row is cut into 16-byte slots as in the bias kernel and, further, into `split`
// column chunks; the B*split (row, chunk) items are spread over the warps of a persistent grid,
// with `split` chosen so that the item count is close to a multiple of the number of resident
// warps.  A warp works alone on an item -- no shared memory, no block barrier: its lanes keep an
// online-softmax pair (running max m, sum of exp2((l' - m) c)) and their best Gumbel score in
// registers, the warp reduces them with shuffles and leaves a partial in the workspace.  The last
// warp to take a row's ticket (an atomic, nobody waits) merges that row's partials in index
// order.
//
// Numerics.  The sampled id must be reproducible bit for bit, so everything that feeds it is an
// exactly rounded fp32 operation spelled with intrinsics: the Gumbel variate is -L(-L(u)) with L
// the fixed logarithm below, and the score is fmaf(l', 1/tau, g).  Most candidates cannot win,
// and the two logarithms are the most expensive part of a candidate, so each warp first applies
// a conservative test on the raw Philox word (see word_floor) and evaluates the exact score only
// for slots in which some candidate might reach the warp's best score so far; the result is the
// same argmax as evaluating every candidate.  The softmax sum only has to be accurate (1e-6
// relative): exponent arguments are formed as a rounded product plus its exact rounding error,
// exp2 of the rounded part comes from the SFU (2 ulp), and the error term is applied to first
// order.  The per-row finish (merging chunk partials, p = exp(.)/Z) is fp64.
#include <cuda_bf16.h>

#include <atomic>
#include <cfloat>
#include <climits>
#include <mutex>

#include "sbw_common.cuh"
#include "sbw_hash.cuh"
#include "sbw_gumbel.cuh"

namespace sbw {
namespace {

// Block shape.  With statistics: one block of 16 warps per SM at about 110 registers (3 % ahead of
// two blocks of 8 warps, as in the bias kernel).  Ids only: the kernel waits on its loads and does
// best with three blocks of 8 warps (85 registers).
__host__ __device__ constexpr int sample_threads(bool stats) { return stats ? 512 : 256; }
__host__ __device__ constexpr int sample_min_blocks(bool stats) { return stats ? 1 : 3; }
constexpr int kMaxSplit = 512;         // chunks per row at most
constexpr int kMinSlotsPerItem = 32;   // one full trip of a warp at least
constexpr int kMaxExtraParts = 40960;  // partials beyond one per row never needed: ~16 waves of warps

struct __align__(32) Partial {
    float m;      // max of l' over the chunk
    float z;      // sum of exp((l' - m)/tau) over the chunk
    float s;      // best Gumbel score
    int id;       // its column (INT_MAX: none)
    float l;      // its biased logit
    float pad[3];
};

struct SampleArgs {
    const void *logits;
    int64_t B, V, ld;
    int64_t n_items;      // B * split
    uint32_t nslot, slots_per_chunk;
    int split;
    const int32_t *ctx;
    int W;
    uint32_t vocab_offset;
    uint64_t key;
    uint32_t thr_m1;
    float delta;          // in the logits' precision, widened
    uint32_t delta_bf16;  // bf16 bits of delta
    float slack;          // max(delta, 0): the most a bias can add
    float inv_tau;        // 1/tau rounded once to fp32 (feeds the score)
    float c2_hi, c2_lo;   // log2(e)/tau as an fp32 pair (feeds the softmax sum)
    double tau;
    uint32_t step_lo, step_hi;   // Gumbel stream: counter words 2 and 3
    BlockKeys gkeys;             // its ten round keys
    Weyl weyl;                   // key-schedule increments of the green hash
    int32_t *out_tokens;
    float *out_max, *out_sumexp, *out_prob;
    float *out_shard;     // [B, 8] or NULL: (m, Z, best score, global id bits, its biased logit, 0, 0, 0)
    bool shard_ids_only;  // the summary is wanted for the ids alone: m = -inf, Z = 0 in it
    uint32_t row_offset;  // global index of row 0 (enters the Gumbel counter)
    Partial *partials;    // [B * split]
    unsigned *tickets;    // [B], zero before the launch
    unsigned *bounds;     // [B], zero before the launch: best exact score per row, order-encoded
    double2 *rowstats;    // [B] (m, Z) for the optional probabilities pass
};

// Monotone map float -> unsigned (larger float, larger code); code 0 decodes to a NaN, which the
// screen treats as "no bound yet", so a zeroed array needs no other initialisation.
__device__ __forceinline__ unsigned encode_score(float f) {
    const unsigned b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float decode_score(unsigned c) {
    return __uint_as_float((c & 0x80000000u) ? (c & 0x7fffffffu) : ~c);
}

__device__ __forceinline__ uint32_t add_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// The same with results below 2^-126 flushed to zero (one instruction instead of a scaled
// sequence): for terms of a sum whose largest term is 1.
__device__ __forceinline__ float ex2_approx_ftz(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// exp2(d * c) for d <= 0 with c = c_hi + c_lo: returns e = exp2(round(d c_hi)) and the residual
// `lo` such that the true value is e * 2^lo ~ e * (1 + lo ln 2).
__device__ __forceinline__ float exp2_split(float d, float c_hi, float c_lo, float &lo) {
    d = fmaxf(d, -1e15f);                       // keeps -inf logits finite below
    const float hi = __fmul_rn(d, c_hi);
    lo = __fmaf_rn(d, c_lo, __fmaf_rn(d, c_hi, -hi));
    return ex2_approx_ftz(hi);
}
__device__ __forceinline__ float exp2_scaled(float d, float c_hi, float c_lo) {
    float lo;
    const float e = exp2_split(d, c_hi, c_lo, lo);
    return __fmaf_rn(e, lo * 0.693147180559945f, e);
}

// Conservative screen for the Gumbel-max.  A candidate of a slot whose largest biased logit is
// `vmax` can reach the score `bound` only if its Gumbel variate g is at least
// T = bound - vmax/tau.  g = -ln(-ln u) increases with u, so that requires
// u >= exp(-exp(-T)), i.e. a Philox word of at least about 2^32 exp(-exp(-T)).  The value
// returned here is a lower bound of that word: T is lowered by a margin that covers the error
// of the fixed logarithm (|g - g_exact| < 4e-6) and every fp32 rounding on the way, the inner
// exponential is rounded up and the outer one down by 1e-4 relative (SFU error 2^-22 plus the
// rounding of their arguments), and 1024 is subtracted to cover the 9 dropped bits of the word
// and the float-to-integer step.  Words below the returned value provably lose; everything
// else is scored exactly.  bound = -inf (nothing scored yet) returns 0: nobody is screened out.
__device__ __forceinline__ uint32_t word_floor(float bound, float vmax, float inv_tau) {
    const float T = __fmaf_rn(-vmax, inv_tau, bound);
    const float Tm = T - (1e-3f + 1e-5f * (fabsf(T) + fabsf(bound)));
    const float E = ex2_approx(Tm * -1.4426950408889634f) * 1.0001f;      // >= exp(-Tm)
    const float U = ex2_approx(E * -1.4426950408889634f) * 0.9999f;       // <= exp(-exp(-Tm))
    const uint32_t k = __float2uint_rd(U * 4294967296.0f);                // NaN -> 0
    return k > 1024u ? k - 1024u : 0u;
}

struct Best {
    float s;
    int id;
    float l;
};
__device__ __forceinline__ bool better(float s1, int id1, float s2, int id2) {
    return s1 > s2 || (s1 == s2 && id1 < id2);
}

template <int SCHEME>
struct RowSeedS;
template <>
struct RowSeedS<SBW_SCHEME_CONTEXT> {
    RowKeys rk;
    __device__ __forceinline__ void init(uint64_t key, const int32_t *ctx, int W) {
        rk = make_row_keys(seed_context(key, ctx, W));
    }
    __device__ __forceinline__ uint32_t word0(uint32_t v, uint64_t, const Weyl) const {
        return philox_word0(v, rk);
    }
    template <int N>
    __device__ __forceinline__ void word0_n(uint32_t vg, uint64_t, const Weyl, uint32_t (&x)[N]) const {
        philox_word0_n<N>(vg, rk, x);
    }
};
template <>
struct RowSeedS<SBW_SCHEME_SELFSALT> {
    uint32_t jmin;
    __device__ __forceinline__ void init(uint64_t, const int32_t *ctx, int W) { jmin = jenkins_min(ctx, W); }
    __device__ __forceinline__ uint32_t word0(uint32_t v, uint64_t key, const Weyl w) const {
        return philox_word0(v, seed_selfsalt(key, jmin, v), w);
    }
    template <int N>
    __device__ __forceinline__ void word0_n(uint32_t vg, uint64_t key, const Weyl w, uint32_t (&x)[N]) const {
        uint32_t v[N];
        uint64_t r[N];
#pragma unroll
        for (int i = 0; i < N; ++i) {
            v[i] = vg + i;
            r[i] = seed_selfsalt(key, jmin, v[i]);
        }
        philox_word0_n<N>(v, r, x, w);
    }
};

// Biased logit of one element, widened to fp32 (Eq. 2 in the logits' own precision).
template <int DTYPE>
__device__ __forceinline__ float biased(uint32_t raw, bool green, float delta) {
    if constexpr (DTYPE == SBW_DTYPE_F32) {
        const float x = __uint_as_float(raw);
        return green ? __fadd_rn(x, delta) : x;
    } else {
        const float x = __uint_as_float(raw << 16);
        // fp32 sum of two bf16 values, rounded once more to bf16 = correctly rounded bf16 sum
        return green ? __bfloat162float(__float2bfloat16_rn(__fadd_rn(x, delta))) : x;
    }
}

// Final per-row merge of `n` partials by one warp.  Two passes over the partials (they sit in
// L2): the row maximum first, then every partial's sum rescaled to it -- one independent fp32
// exp2 per partial (the partial that holds the maximum is scaled by exactly 1), accumulated in
// fp64 in index order per lane.  The sampled probability is one fp64 exp per row.
// Ids only: one pass, best score and its column.
__device__ void finish_row_ids(const SampleArgs &a, int64_t row, const Partial *parts, int n) {
    const int lane = threadIdx.x & 31;
    float s = -INFINITY;
    int id = INT_MAX;
    for (int i = lane; i < n; i += 32) {
        const float4 q0 = __ldcg(reinterpret_cast<const float4 *>(parts + i));
        if (better(q0.z, __float_as_int(q0.w), s, id)) { s = q0.z; id = __float_as_int(q0.w); }
    }
    for (int d = 16; d > 0; d >>= 1) {
        const float os = __shfl_down_sync(0xffffffffu, s, d);
        const int oid = __shfl_down_sync(0xffffffffu, id, d);
        if (better(os, oid, s, id)) { s = os; id = oid; }
    }
    if (lane == 0) {
        if (id == INT_MAX) id = 0;                       // every score was -inf: lowest id
        a.out_tokens[row] = id;
        if (a.out_shard) {
            float4 *o = reinterpret_cast<float4 *>(a.out_shard + row * 8);
            o[0] = make_float4(-INFINITY, 0.0f, s, __int_as_float(static_cast<int>(a.vocab_offset) + id));
            o[1] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        }
    }
}

// The loads of a pass are issued eight at a time per lane before any is used.
__device__ void finish_row(const SampleArgs &a, int64_t row, const Partial *parts, int n) {
    constexpr int kBatch = 8;
    const int lane = threadIdx.x & 31;
    float m = -INFINITY;
    for (int i0 = lane; i0 < n; i0 += 32 * kBatch) {
        float pm[kBatch];
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
            const int i = i0 + 32 * k;
            pm[k] = i < n ? __ldcg(&parts[i].m) : -INFINITY;
        }
#pragma unroll
        for (int k = 0; k < kBatch; ++k) m = fmaxf(m, pm[k]);
    }
    for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
    double Z = 0.0;
    float s = -INFINITY, l = -INFINITY;
    int id = INT_MAX;
    for (int i0 = lane; i0 < n; i0 += 32 * kBatch) {
        // L2 loads: the partials were written by other SMs during this launch
        float4 q[kBatch];
        float pl[kBatch];
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {
            const int i = i0 + 32 * k;
            q[k] = make_float4(-INFINITY, 0.0f, -INFINITY, __int_as_float(INT_MAX));
            pl[k] = -INFINITY;
            if (i < n) {
                q[k] = __ldcg(reinterpret_cast<const float4 *>(parts + i));
                pl[k] = __ldcg(&parts[i].l);
            }
        }
#pragma unroll
        for (int k = 0; k < kBatch; ++k) {                  // index order per lane
            const float pm = q[k].x, pz = q[k].y, ps = q[k].z;
            const int pid = __float_as_int(q[k].w);
            if (pm > -INFINITY) Z += static_cast<double>(pz * exp2_scaled(pm - m, a.c2_hi, a.c2_lo));
            if (better(ps, pid, s, id)) { s = ps; id = pid; l = pl[k]; }
        }
    }
    for (int d = 16; d > 0; d >>= 1) {
        Z += __shfl_down_sync(0xffffffffu, Z, d);
        const float os = __shfl_down_sync(0xffffffffu, s, d);
        const int oid = __shfl_down_sync(0xffffffffu, id, d);
        const float ol = __shfl_down_sync(0xffffffffu, l, d);
        if (better(os, oid, s, id)) { s = os; id = oid; l = ol; }
    }
    if (lane == 0) {
        if (id == INT_MAX) id = 0;                       // every score was -inf: lowest id
        const double md = static_cast<double>(m);
        (void)SBW_CHECKED(row >= 0 && row < a.B && id >= 0 && id < a.V, SBW_SITE_SAMPLE_OUTPUT);
        a.out_tokens[row] = id;
        if (a.out_max) a.out_max[row] = m;
        if (a.out_sumexp) a.out_sumexp[row] = static_cast<float>(Z);
        if (a.out_prob) a.out_prob[row] = static_cast<float>(exp((static_cast<double>(l) - md) / a.tau) / Z);
        a.rowstats[row] = make_double2(md, Z);
        if (a.out_shard) {
            float4 *o = reinterpret_cast<float4 *>(a.out_shard + row * 8);
            o[0] = make_float4(m, static_cast<float>(Z), s, __int_as_float(static_cast<int>(a.vocab_offset) + id));
            o[1] = make_float4(l, 0.0f, 0.0f, 0.0f);
        }
    }
}

// Biased logits lp[0..VEC) of slot j (columns cb .. cb+VEC-1); columns at or beyond V give -inf.
template <int DTYPE, int SCHEME, bool VECTOR, int VEC>
__device__ __forceinline__ void load_biased(const SampleArgs &a, const RowSeedS<SCHEME> &rs, const char *row_ptr,
                                            uint32_t j, uint32_t cb, uint32_t V, float (&lp)[VEC]) {
    const uint32_t vg = a.vocab_offset + cb;
    if (VECTOR && cb + VEC <= V) {
        (void)SBW_CHECKED(static_cast<uint64_t>(j) * VEC + VEC <= static_cast<uint64_t>(a.V), SBW_SITE_SAMPLE_LOAD);
        const uint4 w = __ldg(reinterpret_cast<const uint4 *>(row_ptr) + j);
        const uint32_t *e = reinterpret_cast<const uint32_t *>(&w);
        uint32_t x[VEC];
        rs.template word0_n<VEC>(vg, a.key, a.weyl, x);
        if constexpr (DTYPE == SBW_DTYPE_F32) {
#pragma unroll
            for (int i = 0; i < VEC; ++i) {
                const float v = __uint_as_float(e[i]);
                lp[i] = x[i] <= a.thr_m1 ? __fadd_rn(v, a.delta) : v;
            }
        } else {
            // one packed bf16 add per pair with {delta or -0.0} per half, then widen
            const uint32_t dlo = a.delta_bf16, dhi = a.delta_bf16 << 16;
#pragma unroll
            for (int i = 0; i < VEC / 2; ++i) {
                const uint32_t d = (x[2 * i] <= a.thr_m1 ? dlo : 0x8000u) |
                                   (x[2 * i + 1] <= a.thr_m1 ? dhi : 0x80000000u);
                const uint32_t b = add_bf16x2(e[i], d);
                lp[2 * i] = __uint_as_float(b << 16);
                lp[2 * i + 1] = __uint_as_float(b & 0xffff0000u);
            }
        }
    } else {
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
            lp[i] = -INFINITY;
            if (cb + i < V) {
                uint32_t raw;
                if constexpr (DTYPE == SBW_DTYPE_F32) raw = reinterpret_cast<const uint32_t *>(row_ptr)[cb + i];
                else raw = reinterpret_cast<const uint16_t *>(row_ptr)[cb + i];
                lp[i] = biased<DTYPE>(raw, rs.word0(vg + i, a.key, a.weyl) <= a.thr_m1, a.delta);
            }
        }
    }
}

// Unbiased logits of slot j as raw bit patterns (fp32 bits, or bf16 bits in the low half) and
// widened values; columns at or beyond V give -inf.
template <int DTYPE, bool VECTOR, int VEC>
__device__ __forceinline__ void load_raw(const char *row_ptr, uint32_t j, uint32_t cb, uint32_t V, uint32_t (&raw)[VEC],
                                         float (&lr)[VEC]) {
    if (VECTOR && cb + VEC <= V) {
        const uint4 w = __ldg(reinterpret_cast<const uint4 *>(row_ptr) + j);
        const uint32_t *e = reinterpret_cast<const uint32_t *>(&w);
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
            if constexpr (DTYPE == SBW_DTYPE_F32) raw[i] = e[i];
            else raw[i] = (i & 1) ? e[i >> 1] >> 16 : e[i >> 1] & 0xffffu;
        }
    } else {
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
            raw[i] = DTYPE == SBW_DTYPE_F32 ? 0xff800000u : 0xff80u;        // -inf
            if (cb + i < V) {
                if constexpr (DTYPE == SBW_DTYPE_F32) raw[i] = reinterpret_cast<const uint32_t *>(row_ptr)[cb + i];
                else raw[i] = reinterpret_cast<const uint16_t *>(row_ptr)[cb + i];
            }
        }
    }
#pragma unroll
    for (int i = 0; i < VEC; ++i) lr[i] = __uint_as_float(DTYPE == SBW_DTYPE_F32 ? raw[i] : raw[i] << 16);
}

// Philox words of the Gumbel stream for the VEC candidates starting at global id vg:
// candidate v uses word v & 3 of block v >> 2.
template <int VEC>
__device__ __forceinline__ void gumbel_words(const SampleArgs &a, uint32_t vg, uint32_t rowb, uint32_t (&y)[VEC]) {
    if (VEC >= 4 && (vg & 3u) == 0) {
#pragma unroll
        for (int b = 0; b < (VEC >= 4 ? VEC / 4 : 1); ++b) {
            const uint4 r = philox4x32_10((vg >> 2) + b, rowb, a.step_lo, a.step_hi, a.gkeys);
            if (4 * b + 0 < VEC) y[4 * b + 0] = r.x;
            if (4 * b + 1 < VEC) y[4 * b + 1] = r.y;
            if (4 * b + 2 < VEC) y[4 * b + 2] = r.z;
            if (4 * b + 3 < VEC) y[4 * b + 3] = r.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
            const uint32_t v = vg + i;
            const uint4 r = philox4x32_10(v >> 2, rowb, a.step_lo, a.step_hi, a.gkeys);
            const uint32_t k = v & 3u;
            y[i] = k == 0 ? r.x : k == 1 ? r.y : k == 2 ? r.z : r.w;
        }
    }
}

// STATS = false serves callers that want the sampled ids only (no maximum, softmax sum,
// probability or shard summary).  Then a logit's green test is needed only if the logit could
// win: the Gumbel word of every candidate is drawn first (a quarter of a Philox block each), the
// screen assumes the largest bias the candidate could get, l + max(delta, 0), and the green hash
// -- four fifths of the multiplies of the full pass -- runs for the few candidates that survive.
// The ids are the same: a candidate that fails the screen with the largest possible bias fails it
// with its true one.
__global__ void __launch_bounds__(1024) clear_kernel(unsigned *p, unsigned n) {
    asm volatile("griddepcontrol.launch_dependents;");
    const unsigned i = blockIdx.x * 1024u + threadIdx.x;
    if (i < n) p[i] = 0u;
}

template <int DTYPE, int SCHEME, bool VECTOR, bool STATS>
__global__ void __launch_bounds__(sample_threads(STATS), sample_min_blocks(STATS))
sample_kernel(const SampleArgs a) {
    constexpr int kSampleWarps = sample_threads(STATS) / 32;
    constexpr int VEC = VECTOR ? (DTYPE == SBW_DTYPE_F32 ? 4 : 8) : 1;
    constexpr int ESIZE = DTYPE == SBW_DTYPE_F32 ? 4 : 2;
    const int lane = threadIdx.x & 31;
    // warp w of block b takes items b + w * gridDim.x, ...: consecutive items go to different blocks, so
    // a small batch (fewer items than warps) spreads over all SMs instead of filling a few
    const int64_t warp_id = static_cast<int64_t>(threadIdx.x >> 5) * gridDim.x + blockIdx.x;
    const int64_t n_warps = static_cast<int64_t>(gridDim.x) * kSampleWarps;
    const uint32_t V = static_cast<uint32_t>(a.V);
    // the kernel that clears tickets and bounds may still be running (see launch_one)
    asm volatile("griddepcontrol.wait;" ::: "memory");

    for (int64_t item = warp_id; item < a.n_items; item += n_warps) {
        const int64_t row = item / a.split;
        const int chunk = static_cast<int>(item - row * a.split);
        const uint32_t j_begin = chunk * a.slots_per_chunk;
        const uint32_t j_end = min(a.nslot, j_begin + a.slots_per_chunk);
        const uint32_t rowb = a.row_offset + static_cast<uint32_t>(row);
        const char *row_ptr = static_cast<const char *>(a.logits) + row * a.ld * ESIZE;

        RowSeedS<SCHEME> rs;
        rs.init(a.key, a.ctx + row * a.W, a.W);

        float m_t = -INFINITY, z1 = 0.0f, z2 = 0.0f;
        Best best = {-INFINITY, INT_MAX, -INFINITY};
        // best exact score seen so far: by this warp, and (through the workspace) by every warp
        // that works on the same row -- a lower bound of the row's final best score
        float bound = -INFINITY;

        // warp-uniform trip count: lanes past the end of the chunk carry an empty slot
        for (uint32_t jb = j_begin; jb < j_end; jb += 32) {
            const unsigned shared_bound = __ldcg(a.bounds + row);
            const uint32_t j = jb + lane;
            const bool live = j < j_end;
            const uint32_t cb = j * VEC;
            if constexpr (!STATS) {
                // this path waits on its loads: ask for the next trip's logits now
                if (VECTOR && j + 32 < j_end)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const uint4 *>(row_ptr) + j + 32));
                uint32_t raw[VEC], y[VEC];
                float lr[VEC];
                if (live) {
                    load_raw<DTYPE, VECTOR, VEC>(row_ptr, j, cb, V, raw, lr);
                    gumbel_words<VEC>(a, a.vocab_offset + cb, rowb, y);
                } else {
#pragma unroll
                    for (int i = 0; i < VEC; ++i) { raw[i] = 0u; lr[i] = -INFINITY; y[i] = 0u; }
                }
                float vmax = lr[0];
#pragma unroll
                for (int i = 1; i < VEC; ++i) vmax = fmaxf(vmax, lr[i]);
                // the largest biased value any of these logits could take, rounding included
                float upper = vmax + a.slack;
                upper += fabsf(upper) * (DTYPE == SBW_DTYPE_F32 ? 0x1p-22f : 0x1p-7f);
                bound = fmaxf(bound, decode_score(shared_bound));
                const uint32_t floor_word = word_floor(bound, upper, a.inv_tau);
                bool maybe = false;
#pragma unroll
                for (int i = 0; i < VEC; ++i) maybe |= y[i] >= floor_word;
                maybe &= live;
                if (__any_sync(0xffffffffu, maybe)) {
#pragma unroll
                    for (int i = 0; i < VEC; ++i) {
                        if (live && cb + i < V && y[i] >= floor_word) {
                            const bool green = rs.word0(a.vocab_offset + cb + i, a.key, a.weyl) <= a.thr_m1;
                            const float lp = biased<DTYPE>(raw[i], green, a.delta);
                            const float s = __fmaf_rn(lp, a.inv_tau, gumbel_of_word(y[i]));
                            if (s > best.s) { best.s = s; best.id = static_cast<int>(cb + i); best.l = lp; }
                        }
                    }
                    float b = best.s;
                    for (int d = 16; d > 0; d >>= 1) b = fmaxf(b, __shfl_xor_sync(0xffffffffu, b, d));
                    if (b > bound) {
                        bound = b;
                        if (lane == 0) atomicMax(a.bounds + row, encode_score(b));
                    }
                }
                continue;
            }
            float lp[VEC];
            uint32_t y[VEC];
            if (live) {
                load_biased<DTYPE, SCHEME, VECTOR, VEC>(a, rs, row_ptr, j, cb, V, lp);
                gumbel_words<VEC>(a, a.vocab_offset + cb, rowb, y);
            } else {
#pragma unroll
                for (int i = 0; i < VEC; ++i) { lp[i] = -INFINITY; y[i] = 0u; }
            }
            // online softmax
            float vmax = lp[0];
#pragma unroll
            for (int i = 1; i < VEC; ++i) vmax = fmaxf(vmax, lp[i]);
            if (vmax > m_t) {
                const float f = exp2_scaled(m_t - vmax, a.c2_hi, a.c2_lo);   // 0 when m_t = -inf
                z1 *= f;
                z2 *= f;
                m_t = vmax;
            }
            if (m_t > -INFINITY) {
#pragma unroll
                for (int i = 0; i < VEC; ++i) {
                    float lo;
                    const float e = exp2_split(lp[i] - m_t, a.c2_hi, a.c2_lo, lo);
                    z1 += e;
                    z2 = fmaf(e, lo, z2);
                }
            }
            // Gumbel-max: screen on the raw words, score exactly only where somebody might win
            bound = fmaxf(bound, decode_score(shared_bound));     // fmaxf drops the NaN of "none yet"
            const uint32_t floor_word = word_floor(bound, vmax, a.inv_tau);
            bool maybe = false;
#pragma unroll
            for (int i = 0; i < VEC; ++i) maybe |= y[i] >= floor_word;
            maybe &= live;
            if (__any_sync(0xffffffffu, maybe)) {
                if (live) {
#pragma unroll
                    for (int i = 0; i < VEC; ++i) {
                        if (cb + i < V) {
                            const float s = __fmaf_rn(lp[i], a.inv_tau, gumbel_of_word(y[i]));
                            if (s > best.s) { best.s = s; best.id = static_cast<int>(cb + i); best.l = lp[i]; }
                        }
                    }
                }
                float b = best.s;
                for (int d = 16; d > 0; d >>= 1) b = fmaxf(b, __shfl_xor_sync(0xffffffffu, b, d));
                if (b > bound) {
                    bound = b;
                    if (lane == 0) atomicMax(a.bounds + row, encode_score(b));
                }
            }
        }

        // ---- warp reduction: max, then rescaled sums, then lexicographic argmax ----
        float m_w = m_t;
        for (int d = 16; d > 0; d >>= 1) m_w = fmaxf(m_w, __shfl_xor_sync(0xffffffffu, m_w, d));
        float z_t = 0.0f;
        if (m_t > -INFINITY) z_t = (z1 + 0.693147180559945f * z2) * exp2_scaled(m_t - m_w, a.c2_hi, a.c2_lo);
        for (int d = 16; d > 0; d >>= 1) z_t += __shfl_down_sync(0xffffffffu, z_t, d);
        for (int d = 16; d > 0; d >>= 1) {
            const float os = __shfl_down_sync(0xffffffffu, best.s, d);
            const int oid = __shfl_down_sync(0xffffffffu, best.id, d);
            const float ol = __shfl_down_sync(0xffffffffu, best.l, d);
            if (better(os, oid, best.s, best.id)) { best.s = os; best.id = oid; best.l = ol; }
        }
        unsigned ticket = 0;
        if (lane == 0) {
            Partial p;
            p.m = m_w; p.z = z_t; p.s = best.s; p.id = best.id; p.l = best.l;
            p.pad[0] = p.pad[1] = p.pad[2] = 0.0f;
            if (SBW_CHECKED(item >= 0 && item < a.n_items && row < a.B, SBW_SITE_SAMPLE_WORKSPACE)) a.partials[item] = p;
            __threadfence();                           // partial visible before the ticket is taken
            if (a.split > 1) ticket = atomicAdd(&a.tickets[row], 1u);
        }
        ticket = __shfl_sync(0xffffffffu, ticket, 0);
        if (a.split == 1 || ticket == static_cast<unsigned>(a.split - 1)) {
            __threadfence();                           // the other warps' partials are visible now
            // ids only and many partials (small batches): the single-pass merge
            if (!STATS && a.split > 16) finish_row_ids(a, row, a.partials + row * a.split, a.split);
            else finish_row(a, row, a.partials + row * a.split, a.split);
            if (lane == 0 && a.split > 1) a.tickets[row] = 0;
        }
    }
}

// Optional second pass: the full softmax of the biased logits, fp64 per element.
template <int DTYPE, int SCHEME>
__global__ void __launch_bounds__(256)
probs_kernel(const SampleArgs a, float *out_probs) {
    constexpr int ESIZE = DTYPE == SBW_DTYPE_F32 ? 4 : 2;
    for (int64_t row = blockIdx.y; row < a.B; row += gridDim.y) {
        RowSeedS<SCHEME> rs;
        rs.init(a.key, a.ctx + row * a.W, a.W);
        const double2 st = a.rowstats[row];
        const char *row_ptr = static_cast<const char *>(a.logits) + row * a.ld * ESIZE;
        for (int64_t c = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; c < a.V;
             c += static_cast<int64_t>(gridDim.x) * blockDim.x) {
            uint32_t raw;
            if constexpr (DTYPE == SBW_DTYPE_F32) raw = reinterpret_cast<const uint32_t *>(row_ptr)[c];
            else raw = reinterpret_cast<const uint16_t *>(row_ptr)[c];
            const uint32_t v = a.vocab_offset + static_cast<uint32_t>(c);
            const bool green = rs.word0(v, a.key, a.weyl) <= a.thr_m1;
            const double lp = biased<DTYPE>(raw, green, a.delta);
            out_probs[row * a.V + c] = static_cast<float>(exp((lp - st.x) / a.tau) / st.y);
        }
    }
}

struct Workspace {
    double2 *rowstats;
    unsigned *tickets;
    unsigned *bounds;
    Partial *partials;
    size_t fixed_bytes;   // everything but the partials
};
Workspace carve(void *base, int64_t B) {
    Workspace w;
    char *p = static_cast<char *>(base);
    size_t off = 0;
    w.rowstats = reinterpret_cast<double2 *>(p + off);
    off += align_up(static_cast<size_t>(B) * sizeof(double2), 256);
    w.tickets = reinterpret_cast<unsigned *>(p + off);                 // tickets and bounds are
    w.bounds = w.tickets + B;                                           // cleared by one memset
    off += align_up(2 * static_cast<size_t>(B) * sizeof(unsigned), 256);
    w.partials = reinterpret_cast<Partial *>(p + off);
    w.fixed_bytes = off;
    return w;
}
// Bytes every call needs (one partial per row) and bytes that let the library split rows freely.
size_t workspace_min_bytes(int64_t B) {
    return carve(nullptr, B).fixed_bytes + align_up(static_cast<size_t>(B) * sizeof(Partial), 256);
}
size_t workspace_full_bytes(int64_t B) {
    // B * split partials with split <= kMaxSplit, but items beyond a dozen waves of resident warps
    // bring nothing, so the count is capped at one per row plus kMaxExtraParts
    const int64_t parts = B * kMaxSplit < B + kMaxExtraParts ? B * kMaxSplit : B + kMaxExtraParts;
    return carve(nullptr, B).fixed_bytes + align_up(static_cast<size_t>(parts) * sizeof(Partial), 256);
}

// Chunks per row: the smallest split whose item count B*split fills whole waves of `ctas`
// resident warps to 95 %, else the fullest one; bounded by the row length and by the workspace.
int choose_split(int64_t B, int64_t nslot, int64_t ctas, int64_t max_parts) {
    int64_t max_split = nslot / kMinSlotsPerItem;
    if (max_split > kMaxSplit) max_split = kMaxSplit;
    if (max_split > max_parts / B) max_split = max_parts / B;
    if (max_split < 1) max_split = 1;
    int best = 1;
    double best_eff = 0.0;
    for (int64_t s = 1; s <= max_split; ++s) {
        const int64_t items = B * s;
        const int64_t waves = (items + ctas - 1) / ctas;
        const double eff = static_cast<double>(items) / static_cast<double>(waves * ctas);
        if (eff > best_eff + 1e-9) { best_eff = eff; best = static_cast<int>(s); }
        if (eff >= 0.95) return static_cast<int>(s);
    }
    return best;
}

template <int DTYPE, int SCHEME, bool VECTOR, bool STATS>
int launch_one(SampleArgs &a, int64_t nslot, size_t partial_bytes, cudaStream_t s) {
    DeviceInfo di;
    const int rc = current_device_info(&di);
    if (rc != SBW_OK) return rc;
    constexpr int kSampleThreads = sample_threads(STATS), kSampleWarps = kSampleThreads / 32;
    static std::atomic<int> blocks_per_sm{0};  // a property of the compiled kernel, equal on every sm_100a device
    if (blocks_per_sm == 0) {
        int n = 0;
        SBW_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, sample_kernel<DTYPE, SCHEME, VECTOR, STATS>,
                                                                   kSampleThreads, 0));
        blocks_per_sm = n > 0 ? n : 1;
    }
    const int64_t ctas = static_cast<int64_t>(di.sm_count) * blocks_per_sm;
    const int64_t warps = ctas * kSampleWarps;
    // small batches: no more chunks per row than fill sixteen warps per SM, even when more fit --
    // beyond that the extra partials cost more in the final merge than the extra warps bring
    int64_t max_parts = static_cast<int64_t>(partial_bytes / sizeof(Partial));
    const int64_t two_per_sm = static_cast<int64_t>(di.sm_count) * 16;
    if (two_per_sm / a.B >= 32 && max_parts > two_per_sm) max_parts = two_per_sm;
    a.split = choose_split(a.B, nslot, warps, max_parts);
    a.n_items = a.B * a.split;
    a.slots_per_chunk = static_cast<uint32_t>((nslot + a.split - 1) / a.split);
    // as many blocks as the items fill, but at least one per SM while items last (the kernel hands
    // consecutive items to different blocks)
    int64_t want_ctas = (a.n_items + kSampleWarps - 1) / kSampleWarps;
    const int64_t one_per_sm = a.n_items < di.sm_count ? a.n_items : di.sm_count;
    if (want_ctas < one_per_sm) want_ctas = one_per_sm;
    const unsigned grid = static_cast<unsigned>(want_ctas < ctas ? want_ctas : ctas);
    // Tickets and bounds start at zero.  Inside a stream capture (where the device-side gap between
    // the two nodes is what counts) they are cleared by a small kernel that releases its dependents
    // at once, and the sampler is launched with programmatic stream serialisation: its launch
    // overlaps the clearing, and it waits (griddepcontrol.wait) before it touches the workspace.
    // Outside a capture the plain memset + launch is cheaper for the host.
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    SBW_CUDA_TRY(cudaStreamIsCapturing(s, &capturing));
    if (capturing == cudaStreamCaptureStatusActive) {
        const unsigned words = static_cast<unsigned>(2 * a.B);
        clear_kernel<<<(words + 1023) / 1024, 1024, 0, s>>>(a.tickets, words);
        SBW_CUDA_TRY(cudaGetLastError());
        SBW_CUDA_TRY(launch_pdl(sample_kernel<DTYPE, SCHEME, VECTOR, STATS>, dim3(grid), dim3(kSampleThreads), s, a));
    } else {
        SBW_CUDA_TRY(cudaMemsetAsync(a.tickets, 0, 2 * static_cast<size_t>(a.B) * sizeof(unsigned), s));
        sample_kernel<DTYPE, SCHEME, VECTOR, STATS><<<grid, kSampleThreads, 0, s>>>(a);
        SBW_CUDA_TRY(cudaGetLastError());
    }
    return SBW_OK;
}

template <int DTYPE, int SCHEME>
int launch(SampleArgs &a, bool vector, int64_t nslot, size_t partial_bytes, float *out_probs, cudaStream_t s) {
    const bool stats = a.out_max || a.out_sumexp || a.out_prob || (a.out_shard && !a.shard_ids_only) || out_probs;
    const int rc = stats ? (vector ? launch_one<DTYPE, SCHEME, true, true>(a, nslot, partial_bytes, s)
                                   : launch_one<DTYPE, SCHEME, false, true>(a, nslot, partial_bytes, s))
                         : (vector ? launch_one<DTYPE, SCHEME, true, false>(a, nslot, partial_bytes, s)
                                   : launch_one<DTYPE, SCHEME, false, false>(a, nslot, partial_bytes, s));
    if (rc != SBW_OK) return rc;
    if (out_probs) {
        const unsigned gx = static_cast<unsigned>((a.V + 255) / 256 < 1024 ? (a.V + 255) / 256 : 1024);
        const unsigned gy = static_cast<unsigned>(a.B < 4096 ? a.B : 4096);
        probs_kernel<DTYPE, SCHEME><<<dim3(gx, gy), 256, 0, s>>>(a, out_probs);
        SBW_CUDA_TRY(cudaGetLastError());
    }
    return SBW_OK;
}

// Shared by the two entry points: `workspace_bytes` must cover workspace_min_bytes(B); more
// lets rows be split into more chunks.
// The argument checks of every sampling entry, workspace excepted; host only.
int check_sample_args(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld, int64_t vocab_offset,
                      const int32_t *ctx_tokens, int ctx_width, double gamma, float delta, int scheme,
                      float temperature, const int32_t *out_tokens, const float *out_shard, int64_t row_offset) {
    if (!valid_common(dtype, ctx_width, gamma, scheme)) return SBW_ERR_INVALID_ARG;
    if (B < 0 || V <= 0 || ld < V || vocab_offset < 0) return SBW_ERR_INVALID_ARG;
    if (!(temperature > 0.0f) || temperature - temperature != 0.0f) return SBW_ERR_INVALID_ARG;
    if (!(delta == delta) || delta - delta != 0.0f) return SBW_ERR_INVALID_ARG;
    if (V > 0x7fffffffLL || vocab_offset + V > (int64_t(1) << 32)) return SBW_ERR_UNSUPPORTED;
    // a shard summary carries the global id as a signed 32-bit value
    if (out_shard && vocab_offset + V > (int64_t(1) << 31)) return SBW_ERR_UNSUPPORTED;
    if (B > 0x7fffffffLL / kMaxSplit) return SBW_ERR_UNSUPPORTED;
    if (B == 0) return SBW_OK;
    if (!logits || !ctx_tokens || !out_tokens) return SBW_ERR_INVALID_ARG;
    if (row_offset < 0 || row_offset + B > (int64_t(1) << 32)) return SBW_ERR_INVALID_ARG;
    if (out_shard && reinterpret_cast<uintptr_t>(out_shard) % 16 != 0) return SBW_ERR_INVALID_ARG;
    const float c2_hi = static_cast<float>(1.4426950408889634 / static_cast<double>(temperature));
    if (!(c2_hi * 1e15f < FLT_MAX)) return SBW_ERR_INVALID_ARG;   // temperature too small
    return SBW_OK;
}

int bias_sample_impl(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld, int64_t vocab_offset,
                     const int32_t *ctx_tokens, int ctx_width, uint64_t key, double gamma, float delta,
                     int scheme, float temperature, uint64_t rng_seed, uint64_t rng_step, int32_t *out_tokens,
                     float *out_max, float *out_sumexp, float *out_prob, float *out_probs, void *workspace,
                     size_t workspace_bytes, bool need_full_workspace, cudaStream_t s,
                     float *out_shard = nullptr, int64_t row_offset = 0, bool shard_ids_only = false) {
    if (int rc = check_sample_args(logits, dtype, B, V, ld, vocab_offset, ctx_tokens, ctx_width, gamma, delta, scheme,
                                   temperature, out_tokens, out_shard, row_offset))
        return rc;
    if (B == 0) return SBW_OK;
    const double c2 = 1.4426950408889634 / static_cast<double>(temperature);
    const float c2_hi = static_cast<float>(c2);
    const size_t need = need_full_workspace ? workspace_full_bytes(B) : workspace_min_bytes(B);
    if (!workspace || workspace_bytes < need || reinterpret_cast<uintptr_t>(workspace) % 256 != 0)
        return SBW_ERR_WORKSPACE;
    const Workspace ws = carve(workspace, B);

    const int esize = dtype == SBW_DTYPE_F32 ? 4 : 2;
    const bool vector = (reinterpret_cast<uintptr_t>(logits) % 16 == 0) && ((ld * esize) % 16 == 0);
    const int vec = vector ? 16 / esize : 1;
    const int64_t nslot = (V + vec - 1) / vec;

    SampleArgs a;
    a.logits = logits;
    a.B = B; a.V = V; a.ld = ld;
    a.nslot = static_cast<uint32_t>(nslot);
    a.ctx = ctx_tokens;
    a.W = ctx_width;
    a.vocab_offset = static_cast<uint32_t>(vocab_offset);
    a.key = key;
    a.thr_m1 = threshold_minus_one(gamma);
    a.delta = delta;
    a.delta_bf16 = 0;
    if (dtype == SBW_DTYPE_BF16) {
        const __nv_bfloat16 d = __float2bfloat16_rn(delta);
        a.delta_bf16 = static_cast<uint32_t>(__bfloat16_as_ushort(d));
        a.delta = __bfloat162float(d);
    }
    a.slack = a.delta > 0.0f ? a.delta : 0.0f;
    a.inv_tau = 1.0f / temperature;
    a.c2_hi = c2_hi;
    a.c2_lo = static_cast<float>(c2 - static_cast<double>(c2_hi));
    a.tau = static_cast<double>(temperature);
    a.step_lo = static_cast<uint32_t>(rng_step);
    a.step_hi = static_cast<uint32_t>(rng_step >> 32);
    a.gkeys = make_block_keys(static_cast<uint32_t>(rng_seed), static_cast<uint32_t>(rng_seed >> 32));
    a.weyl = make_weyl();
    a.out_tokens = out_tokens;
    a.out_max = out_max;
    a.out_sumexp = out_sumexp;
    a.out_prob = out_prob;
    a.out_shard = out_shard;
    a.shard_ids_only = shard_ids_only;
    a.row_offset = static_cast<uint32_t>(row_offset);
    a.partials = ws.partials;
    a.tickets = ws.tickets;
    a.bounds = ws.bounds;
    a.rowstats = ws.rowstats;
    const size_t partial_bytes = workspace_bytes - ws.fixed_bytes;

    if (dtype == SBW_DTYPE_F32) {
        return scheme == SBW_SCHEME_CONTEXT
                   ? launch<SBW_DTYPE_F32, SBW_SCHEME_CONTEXT>(a, vector, nslot, partial_bytes, out_probs, s)
                   : launch<SBW_DTYPE_F32, SBW_SCHEME_SELFSALT>(a, vector, nslot, partial_bytes, out_probs, s);
    }
    return scheme == SBW_SCHEME_CONTEXT
               ? launch<SBW_DTYPE_BF16, SBW_SCHEME_CONTEXT>(a, vector, nslot, partial_bytes, out_probs, s)
               : launch<SBW_DTYPE_BF16, SBW_SCHEME_SELFSALT>(a, vector, nslot, partial_bytes, out_probs, s);
}

}  // namespace
}  // namespace sbw

extern "C" size_t sbw_sample_workspace_bytes(int64_t B, int64_t V) {
    if (B <= 0 || V <= 0) return 0;
    return sbw::workspace_full_bytes(B);
}

extern "C" int sbw_bias_sample(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                               int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width,
                               uint64_t key, double gamma, float delta, int scheme, float temperature,
                               uint64_t rng_seed, uint64_t rng_step, int32_t *out_tokens, float *out_max,
                               float *out_sumexp, float *out_prob, float *out_probs, void *workspace,
                               size_t workspace_bytes, void *stream) {
    return sbw::bias_sample_impl(logits, dtype, B, V, ld, vocab_offset, ctx_tokens, ctx_width, key, gamma,
                                 delta, scheme, temperature, rng_seed, rng_step, out_tokens, out_max,
                                 out_sumexp, out_prob, out_probs, workspace, workspace_bytes, true,
                                 static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------------------
// sbw_bias_sample_noalloc: the same call for users that cannot allocate device memory (a plugin
// inside a serving engine whose KV-cache pool owns the whole GPU, a component under a fixed
// memory budget).  The scratch is a fixed array that is part of the library image.
// ---------------------------------------------------------------------------------------------
namespace sbw {
namespace {

constexpr size_t kNoallocScratchBytes = 256 * 1024;   // covers SBW_NOALLOC_MAX_ROWS rows
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoallocScratchBytes];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not a device address: the
// address the kernels need comes from cudaGetSymbolAddress, asked once per device with that
// device current, and is cached here.
int noalloc_scratch_address(void **out) {
    constexpr int kMaxDevices = 64;
    static void *cached[kMaxDevices] = {nullptr};
    static std::mutex mu;
    int dev = 0;
    SBW_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SBW_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mu);
    if (!cached[dev]) {
        void *p = nullptr;
        SBW_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        cached[dev] = p;
    }
    *out = cached[dev];
    return SBW_OK;
}

}  // namespace
}  // namespace sbw

extern "C" int sbw_bias_sample_noalloc(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                                       int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width,
                                       uint64_t key, double gamma, float delta, int scheme,
                                       float temperature, uint64_t rng_seed, uint64_t rng_step,
                                       int32_t *out_tokens, float *out_max, float *out_sumexp,
                                       float *out_prob, float *out_probs, void *stream) {
    using namespace sbw;
    // host-side argument checks first, as in every other entry; the capacity next; the device is
    // asked for the array's address only by a call that will launch
    if (int rc = check_sample_args(logits, dtype, B, V, ld, vocab_offset, ctx_tokens, ctx_width, gamma, delta, scheme,
                                   temperature, out_tokens, nullptr, 0))
        return rc;
    if (B == 0) return SBW_OK;
    if (B > SBW_NOALLOC_MAX_ROWS) return SBW_ERR_TOO_LARGE;
    static_assert(sizeof(double2) * SBW_NOALLOC_MAX_ROWS + 2 * sizeof(unsigned) * SBW_NOALLOC_MAX_ROWS +
                          sizeof(Partial) * SBW_NOALLOC_MAX_ROWS + 3 * 256 <=
                      kNoallocScratchBytes,
                  "the built-in scratch must hold the workspace of SBW_NOALLOC_MAX_ROWS rows");
    if (workspace_min_bytes(B) > kNoallocScratchBytes) return SBW_ERR_TOO_LARGE;
    void *scratch = nullptr;
    if (int rc = noalloc_scratch_address(&scratch)) return rc;
    // The shared array keeps whatever the previous call left in it.  The only part that must
    // start at zero is the per-row ticket counters, and the launch code clears those on the
    // stream before every launch that uses them; everything else is written before it is read.
    // Rows are split into as many chunks as the fixed array has room for.
    return bias_sample_impl(logits, dtype, B, V, ld, vocab_offset, ctx_tokens, ctx_width, key, gamma, delta,
                            scheme, temperature, rng_seed, rng_step, out_tokens, out_max, out_sumexp,
                            out_prob, out_probs, scratch, kNoallocScratchBytes, false,
                            static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------------------
// Vocabulary-sharded sampling.  The paper notes that each device can derive identical green
// lists from the shared key (Limitations) without validating it; here a row whose vocabulary is
// split over S shards is sampled by S independent sbw_bias_sample_shard calls -- no shard reads
// another's logits -- and one tiny combine over the S per-row summaries, which is the only data
// that has to cross devices (32 bytes per row and shard).
// ---------------------------------------------------------------------------------------------
namespace sbw {
namespace {

__global__ void combine_kernel(const float *shards, int64_t S, int64_t B, double tau, int32_t *out_tokens,
                               float *out_max, float *out_sumexp, float *out_prob) {
    const int64_t row = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (row >= B) return;
    // pass 1: row maximum and winner (ties -> lowest global id); pass 2: rescaled sum
    float m = -INFINITY, s = -INFINITY, l = -INFINITY;
    int id = INT_MAX;
    for (int64_t r = 0; r < S; ++r) {
        const float4 q = *reinterpret_cast<const float4 *>(shards + (r * B + row) * 8);
        m = fmaxf(m, q.x);
        const int qid = __float_as_int(q.w);
        if (better(q.z, qid, s, id)) { s = q.z; id = qid; l = shards[(r * B + row) * 8 + 4]; }
    }
    double Z = 0.0;
    for (int64_t r = 0; r < S; ++r) {
        const float4 q = *reinterpret_cast<const float4 *>(shards + (r * B + row) * 8);
        if (q.x > -INFINITY) Z += static_cast<double>(q.y) * exp((static_cast<double>(q.x) - m) / tau);
    }
    out_tokens[row] = id;
    if (out_max) out_max[row] = m;
    if (out_sumexp) out_sumexp[row] = static_cast<float>(Z);
    if (out_prob) out_prob[row] = static_cast<float>(exp((static_cast<double>(l) - m) / tau) / Z);
}

}  // namespace
}  // namespace sbw

extern "C" int sbw_bias_sample_shard(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                                     int64_t vocab_offset, int64_t row_offset, const int32_t *ctx_tokens,
                                     int ctx_width, uint64_t key, double gamma, float delta, int scheme,
                                     float temperature, uint64_t rng_seed, uint64_t rng_step,
                                     float *out_shard, int32_t *out_tokens, void *workspace,
                                     size_t workspace_bytes, void *stream) {
    if (B > 0 && !out_shard) return SBW_ERR_INVALID_ARG;
    return sbw::bias_sample_impl(logits, dtype, B, V, ld, vocab_offset, ctx_tokens, ctx_width, key, gamma,
                                 delta, scheme, temperature, rng_seed, rng_step, out_tokens, nullptr, nullptr,
                                 nullptr, nullptr, workspace, workspace_bytes, true,
                                 static_cast<cudaStream_t>(stream), out_shard, row_offset);
}

extern "C" int sbw_bias_sample_shard_ids(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                                         int64_t vocab_offset, int64_t row_offset, const int32_t *ctx_tokens,
                                         int ctx_width, uint64_t key, double gamma, float delta, int scheme,
                                         float temperature, uint64_t rng_seed, uint64_t rng_step,
                                         float *out_shard, int32_t *out_tokens, void *workspace,
                                         size_t workspace_bytes, void *stream) {
    if (B > 0 && !out_shard) return SBW_ERR_INVALID_ARG;
    return sbw::bias_sample_impl(logits, dtype, B, V, ld, vocab_offset, ctx_tokens, ctx_width, key, gamma,
                                 delta, scheme, temperature, rng_seed, rng_step, out_tokens, nullptr, nullptr,
                                 nullptr, nullptr, workspace, workspace_bytes, true,
                                 static_cast<cudaStream_t>(stream), out_shard, row_offset, true);
}

extern "C" int sbw_sample_combine(const float *shards, int64_t S, int64_t B, float temperature,
                                  int32_t *out_tokens, float *out_max, float *out_sumexp, float *out_prob,
                                  void *stream) {
    if (S < 1 || B < 0 || !(temperature > 0.0f) || temperature - temperature != 0.0f) return SBW_ERR_INVALID_ARG;
    if (B == 0) return SBW_OK;
    if (!shards || !out_tokens || reinterpret_cast<uintptr_t>(shards) % 16 != 0) return SBW_ERR_INVALID_ARG;
    const unsigned grid = static_cast<unsigned>((B + 127) / 128);
    sbw::combine_kernel<<<grid, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        shards, S, B, static_cast<double>(temperature), out_tokens, out_max, out_sumexp, out_prob);
    SBW_CUDA_TRY(cudaGetLastError());
    return SBW_OK;
}
