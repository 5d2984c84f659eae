// sbw_bias_logits: Eq. 1 + Eq. 2 of the paper in one in-place pass over the [B, V] logits.
//
// Layout of the work.  A row is cut into 16-byte "slots" (4 fp32 or 8 bf16 logits); the B*nslot
// slots form one flat index space that is divided evenly over a persistent grid (a multiple of
// the SM count), so every SM receives the same number of slots whatever B and V are.  A block
// walks its share row by row: per row it derives the seed material once (context scheme: the ten
// Philox round keys; self-salt scheme: the smallest context hash), then its threads stride over
// the row's slots.  Per trip a thread issues 128-bit loads for 8 logits, evaluates the 8 hash
// chains round by round in registers (the interleaving is what keeps the multiply pipe busy: the
// kernel is bound by the 32x32->64 multiplier, not by HBM), applies the bias, and stores 128 bits
// back.  No shared memory, no mask tensor, no other global traffic.  Rows that do not start on
// 16-byte boundaries, and the ragged last slot of a row, go through a scalar routine.
//
// The kernel is launched with programmatic stream serialisation: it lets the next kernel of the
// stream begin its launch while this one drains, and itself waits for everything before it in the
// stream before it touches memory, so stream order is preserved.
#include <cuda_bf16.h>

#include <atomic>

#include "sbw_common.cuh"
#include "sbw_hash.cuh"

namespace sbw {
namespace {

constexpr int kBiasThreads = 512;   // one block of 16 warps per SM: measured 2-3 % ahead of two blocks of 8

struct BiasArgs {
    void *logits;
    int64_t B, V, ld;
    int64_t nslot;          // slots per row
    const int32_t *ctx;
    int W;
    uint32_t vocab_offset;  // global id of column 0 (mod 2^32)
    uint64_t key;
    uint32_t thr_m1;        // green <=> x <= thr_m1
    float delta;            // fp32 path: delta; bf16 path: delta rounded to bf16, widened
    uint32_t delta_bf16;    // bf16 bits of delta
    Weyl weyl;              // Philox key-schedule increments (see sbw_hash.cuh)
    const void *src;        // out-of-place variant only: rows are read here and written to `logits`
    int64_t ld_src;
};

__device__ __forceinline__ uint32_t add_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// Per-row seed material.
template <int SCHEME>
struct RowSeed;
template <>
struct RowSeed<SBW_SCHEME_CONTEXT> {
    RowKeys rk;
    __device__ __forceinline__ void init(uint64_t key, const int32_t *ctx, int W) {
        rk = make_row_keys(seed_context(key, ctx, W));
    }
    __device__ __forceinline__ uint32_t word0(uint32_t v, uint64_t, const Weyl) const {
        return philox_word0(v, rk);
    }
};
template <>
struct RowSeed<SBW_SCHEME_SELFSALT> {
    uint32_t jmin;
    __device__ __forceinline__ void init(uint64_t, const int32_t *ctx, int W) { jmin = jenkins_min(ctx, W); }
    __device__ __forceinline__ uint32_t word0(uint32_t v, uint64_t key, const Weyl w) const {
        return philox_word0(v, seed_selfsalt(key, jmin, v), w);
    }
};

// Columns [c_begin, c_end) of one row, one logit at a time, any alignment: ragged tails and rows
// that are not 16-byte aligned.  Kept out of line so that it does not weigh on the fast path.
template <int DTYPE, int SCHEME>
__device__ __noinline__ void bias_scalar(const BiasArgs &a, const RowSeed<SCHEME> &rs, void *row_ptr,
                                         uint32_t c_begin, uint32_t c_end, uint32_t c_step) {
    for (uint32_t col = c_begin; col < c_end; col += c_step) {
        if (!SBW_CHECKED(col < static_cast<uint32_t>(a.V), SBW_SITE_BIAS_SCALAR)) continue;
        const uint32_t v = a.vocab_offset + col;
        if (rs.word0(v, a.key, a.weyl) > a.thr_m1) continue;
        if constexpr (DTYPE == SBW_DTYPE_F32) {
            float *p = static_cast<float *>(row_ptr) + col;
            *p = __fadd_rn(*p, a.delta);
        } else {
            __nv_bfloat16 *p = static_cast<__nv_bfloat16 *>(row_ptr) + col;
            // both operands are bf16 values, so rounding their fp32 sum once more gives the
            // correctly rounded bf16 sum
            *p = __float2bfloat16_rn(__fadd_rn(__bfloat162float(*p), a.delta));
        }
    }
}

// Green flags of the 8 consecutive ids vg .. vg+7.
template <int SCHEME>
__device__ __forceinline__ void green8(const BiasArgs &a, const RowSeed<SCHEME> &rs, uint32_t vg,
                                       bool (&g)[8]) {
    uint32_t x[8];
    if constexpr (SCHEME == SBW_SCHEME_CONTEXT) {
        philox_word0_n<8>(vg, rs.rk, x);
    } else {
        uint32_t v[8];
        uint64_t r[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            v[i] = vg + i;
            r[i] = seed_selfsalt(a.key, rs.jmin, v[i]);
        }
        philox_word0_n<8>(v, r, x, a.weyl);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) g[i] = x[i] <= a.thr_m1;
}
template <int SCHEME>
__device__ __forceinline__ void green4x2(const BiasArgs &a, const RowSeed<SCHEME> &rs, uint32_t vg0,
                                         uint32_t vg1, bool (&g)[8]) {
    uint32_t x[8];
    if constexpr (SCHEME == SBW_SCHEME_CONTEXT) {
        uint32_t xa[4], xb[4];
        philox_word0_n<4>(vg0, rs.rk, xa);
        philox_word0_n<4>(vg1, rs.rk, xb);
#pragma unroll
        for (int i = 0; i < 4; ++i) { x[i] = xa[i]; x[4 + i] = xb[i]; }
    } else {
        uint32_t v[8];
        uint64_t r[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            v[i] = (i < 4 ? vg0 : vg1) + (i & 3);
            r[i] = seed_selfsalt(a.key, rs.jmin, v[i]);
        }
        philox_word0_n<8>(v, r, x, a.weyl);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) g[i] = x[i] <= a.thr_m1;
}

// COPY = true is the out-of-place variant used by the truncated sampler: the same pass, reading the
// rows from a.src (16-byte aligned rows) and writing the biased rows to a.logits.
template <int DTYPE, int SCHEME, bool VECTOR, bool COPY = false>
__global__ void __launch_bounds__(kBiasThreads, 1)
bias_kernel(const BiasArgs a) {
    constexpr int VEC = VECTOR ? (DTYPE == SBW_DTYPE_F32 ? 4 : 8) : 1;
    constexpr int ESIZE = DTYPE == SBW_DTYPE_F32 ? 4 : 2;
    // let the next kernel in the stream start launching; wait for the previous ones to finish
    asm volatile("griddepcontrol.launch_dependents;");
    // The rows are cut into units of one trip of the whole block (kBiasThreads slots, twice that
    // for fp32); a row's last unit may be partly empty.  Every block takes the same number of
    // units (to within one) of the B * units_per_row there are, so a range that crosses a row
    // boundary costs no extra trip.
    constexpr uint32_t kUnitSlots = VECTOR ? kBiasThreads * (DTYPE == SBW_DTYPE_F32 ? 2 : 1) : kBiasThreads;
    const uint32_t nslot = static_cast<uint32_t>(a.nslot);
    const uint32_t units_per_row = (nslot + kUnitSlots - 1) / kUnitSlots;
    const int64_t units = a.B * units_per_row;
    const int64_t u_begin = units / gridDim.x * blockIdx.x + (units % gridDim.x) * blockIdx.x / gridDim.x;
    const int64_t u_end = units / gridDim.x * (blockIdx.x + 1) + (units % gridDim.x) * (blockIdx.x + 1) / gridDim.x;
    int64_t row = u_begin / units_per_row;
    uint32_t unit = static_cast<uint32_t>(u_begin - row * units_per_row);
    int64_t left = u_end - u_begin;
    const uint32_t V = static_cast<uint32_t>(a.V);
    const uint32_t nfull = V / VEC;       // slots of the row that are complete vectors
    asm volatile("griddepcontrol.wait;" ::: "memory");

    while (left > 0) {
        const uint32_t seg_units = static_cast<uint32_t>(min(static_cast<int64_t>(units_per_row - unit), left));
        RowSeed<SCHEME> rs;
        rs.init(a.key, a.ctx + row * a.W, a.W);
        char *row_ptr = static_cast<char *>(a.logits) + row * a.ld * ESIZE;
        const uint32_t col = unit * kUnitSlots;
        const uint32_t j_end = min(nslot, col + seg_units * kUnitSlots);
        if constexpr (!VECTOR) {
            bias_scalar<DTYPE, SCHEME>(a, rs, row_ptr, col + threadIdx.x, j_end, kBiasThreads);
        } else {
            const uint32_t jf_end = min(j_end, nfull);
            uint4 *slots = reinterpret_cast<uint4 *>(row_ptr);
            const uint4 *in = slots;
            if constexpr (COPY)
                in = reinterpret_cast<const uint4 *>(static_cast<const char *>(a.src) + row * a.ld_src * ESIZE);
            if constexpr (DTYPE == SBW_DTYPE_BF16) {
                const uint32_t dlo = a.delta_bf16, dhi = a.delta_bf16 << 16;
                for (uint32_t j = col + threadIdx.x; j < jf_end; j += kBiasThreads) {
                    if (!SBW_CHECKED(row < a.B && (static_cast<uint64_t>(j) + 1) * 8 <= static_cast<uint64_t>(a.V),
                                     SBW_SITE_BIAS_VECTOR))
                        continue;
                    uint4 w = in[j];
                    bool g[8];
                    green8<SCHEME>(a, rs, a.vocab_offset + j * 8, g);
                    // adding -0.0 returns the other operand unchanged, so a packed add with
                    // {delta or -0.0} per half biases exactly the green halves
                    uint32_t *e = reinterpret_cast<uint32_t *>(&w);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t d = (g[2 * i] ? dlo : 0x8000u) | (g[2 * i + 1] ? dhi : 0x80000000u);
                        e[i] = add_bf16x2(e[i], d);
                    }
                    slots[j] = w;
                }
            } else {
                // two slots (8 logits) per trip; the second one may fall off the end of the segment
                for (uint32_t j = col + threadIdx.x; j < jf_end; j += 2 * kBiasThreads) {
                    const uint32_t j2 = j + kBiasThreads;
                    const bool two = j2 < jf_end;
                    if (!SBW_CHECKED(row < a.B && (static_cast<uint64_t>(two ? j2 : j) + 1) * 4 <= static_cast<uint64_t>(a.V),
                                     SBW_SITE_BIAS_VECTOR))
                        continue;
                    uint4 w0 = in[j];
                    uint4 w1 = two ? in[j2] : make_uint4(0, 0, 0, 0);
                    bool g[8];
                    green4x2<SCHEME>(a, rs, a.vocab_offset + j * 4, a.vocab_offset + j2 * 4, g);
                    uint32_t *e0 = reinterpret_cast<uint32_t *>(&w0);
                    uint32_t *e1 = reinterpret_cast<uint32_t *>(&w1);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float s0 = __fadd_rn(__uint_as_float(e0[i]), a.delta);
                        const float s1 = __fadd_rn(__uint_as_float(e1[i]), a.delta);
                        e0[i] = g[i] ? __float_as_uint(s0) : e0[i];
                        e1[i] = g[4 + i] ? __float_as_uint(s1) : e1[i];
                    }
                    slots[j] = w0;
                    if (two) slots[j2] = w1;
                }
            }
            // ragged last slot of the row, if this block owns it
            if (nfull < nslot && j_end == nslot && threadIdx.x == 0) {
                if constexpr (COPY) {
                    const char *tail = reinterpret_cast<const char *>(in);
                    for (uint32_t b = nfull * VEC * ESIZE; b < V * ESIZE; ++b) row_ptr[b] = tail[b];
                }
                bias_scalar<DTYPE, SCHEME>(a, rs, row_ptr, nfull * VEC, V, 1);
            }
        }
        left -= seg_units;
        ++row;
        unit = 0;
    }
}

template <int DTYPE, int SCHEME, bool VECTOR, bool COPY = false>
int launch(const BiasArgs &a, cudaStream_t stream) {
    DeviceInfo di;
    int rc = current_device_info(&di);
    if (rc != SBW_OK) return rc;
    static std::atomic<int> blocks_per_sm{0};  // a property of the compiled kernel, equal on every sm_100a device
    if (blocks_per_sm == 0) {
        int n = 0;
        SBW_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, bias_kernel<DTYPE, SCHEME, VECTOR, COPY>,
                                                                   kBiasThreads, 0));
        blocks_per_sm = n > 0 ? n : 1;
    }
    constexpr int64_t kUnitSlots = VECTOR ? kBiasThreads * (DTYPE == SBW_DTYPE_F32 ? 2 : 1) : kBiasThreads;
    const int64_t want = a.B * ((a.nslot + kUnitSlots - 1) / kUnitSlots);
    const int64_t cap = static_cast<int64_t>(di.sm_count) * blocks_per_sm;
    const unsigned grid = static_cast<unsigned>(want < cap ? want : cap);
    SBW_CUDA_TRY(launch_pdl(bias_kernel<DTYPE, SCHEME, VECTOR, COPY>, dim3(grid), dim3(kBiasThreads), stream, a));
    return SBW_OK;
}

template <int DTYPE, int SCHEME>
int launch_v(const BiasArgs &a, bool vector, cudaStream_t stream) {
    return vector ? launch<DTYPE, SCHEME, true>(a, stream) : launch<DTYPE, SCHEME, false>(a, stream);
}

}  // namespace

// Checks and argument set-up shared by the in-place and the out-of-place entry.  Returns SBW_OK
// with *run = false when there is nothing to do (empty batch, or a bias that is zero in the
// logits' precision: the paper's delta = 0 control, which leaves every bit alone -- an IEEE add of
// +0 would turn -0 into +0).
static int prepare(BiasArgs &a, void *logits, int dtype, int64_t B, int64_t V, int64_t ld, int64_t vocab_offset,
                   const int32_t *ctx_tokens, int ctx_width, uint64_t key, double gamma, float delta, int scheme,
                   bool *run) {
    *run = false;
    if (!valid_common(dtype, ctx_width, gamma, scheme)) return SBW_ERR_INVALID_ARG;
    if (B < 0 || V <= 0 || ld < V || vocab_offset < 0) return SBW_ERR_INVALID_ARG;
    if (V > 0x7fffffffLL || B > (int64_t(1) << 40)) return SBW_ERR_UNSUPPORTED;
    if (vocab_offset + V > (int64_t(1) << 32)) return SBW_ERR_UNSUPPORTED;   // ids are 32-bit
    if (!(delta == delta) || delta - delta != 0.0f) return SBW_ERR_INVALID_ARG;  // NaN or inf
    if (B == 0) return SBW_OK;
    if (!logits || !ctx_tokens) return SBW_ERR_INVALID_ARG;
    a.logits = logits;
    a.B = B; a.V = V; a.ld = ld;
    a.ctx = ctx_tokens;
    a.W = ctx_width;
    a.vocab_offset = static_cast<uint32_t>(vocab_offset);
    a.key = key;
    a.thr_m1 = threshold_minus_one(gamma);
    a.delta = delta;
    a.delta_bf16 = 0;
    a.weyl = make_weyl();
    a.src = nullptr;
    a.ld_src = 0;
    if (dtype == SBW_DTYPE_BF16) {
        const __nv_bfloat16 d = __float2bfloat16_rn(delta);
        a.delta_bf16 = static_cast<uint32_t>(__bfloat16_as_ushort(d));
        a.delta = __bfloat162float(d);
    }
    *run = a.delta != 0.0f;
    return SBW_OK;
}

int bias_logits_impl(void *logits, int dtype, int64_t B, int64_t V, int64_t ld, int64_t vocab_offset,
                     const int32_t *ctx_tokens, int ctx_width, uint64_t key, double gamma, float delta,
                     int scheme, cudaStream_t stream) {
    BiasArgs a;
    bool run;
    if (int rc = prepare(a, logits, dtype, B, V, ld, vocab_offset, ctx_tokens, ctx_width, key, gamma, delta, scheme,
                         &run))
        return rc;
    if (!run) return SBW_OK;
    const int esize = dtype == SBW_DTYPE_F32 ? 4 : 2;
    const bool vector = (reinterpret_cast<uintptr_t>(logits) % 16 == 0) && ((ld * esize) % 16 == 0);
    const int vec = vector ? 16 / esize : 1;
    a.nslot = (V + vec - 1) / vec;

    if (dtype == SBW_DTYPE_F32) {
        return scheme == SBW_SCHEME_CONTEXT
                   ? launch_v<SBW_DTYPE_F32, SBW_SCHEME_CONTEXT>(a, vector, stream)
                   : launch_v<SBW_DTYPE_F32, SBW_SCHEME_SELFSALT>(a, vector, stream);
    }
    return scheme == SBW_SCHEME_CONTEXT
               ? launch_v<SBW_DTYPE_BF16, SBW_SCHEME_CONTEXT>(a, vector, stream)
               : launch_v<SBW_DTYPE_BF16, SBW_SCHEME_SELFSALT>(a, vector, stream);
}

// Out-of-place bias: dst[b, j] = bias(src[b, j]) for j < V in one pass.  *done = false (and nothing
// launched) when the rows of src or dst are not 16-byte aligned or the bias is zero in the logits'
// precision; the caller then copies the rows itself and biases them in place.
int bias_copy_impl(const void *src, int64_t ld_src, void *dst, int dtype, int64_t B, int64_t V, int64_t ld,
                   int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width, uint64_t key, double gamma,
                   float delta, int scheme, cudaStream_t stream, bool *done) {
    *done = false;
    BiasArgs a;
    bool run;
    if (int rc = prepare(a, dst, dtype, B, V, ld, vocab_offset, ctx_tokens, ctx_width, key, gamma, delta, scheme,
                         &run))
        return rc;
    if (!src || ld_src < V) return SBW_ERR_INVALID_ARG;
    const int esize = dtype == SBW_DTYPE_F32 ? 4 : 2;
    const bool aligned = reinterpret_cast<uintptr_t>(dst) % 16 == 0 && (ld * esize) % 16 == 0 &&
                         reinterpret_cast<uintptr_t>(src) % 16 == 0 && (ld_src * esize) % 16 == 0;
    if (!run || !aligned) return SBW_OK;
    a.src = src;
    a.ld_src = ld_src;
    const int vec = 16 / esize;
    a.nslot = (V + vec - 1) / vec;
    *done = true;
    if (dtype == SBW_DTYPE_F32) {
        return scheme == SBW_SCHEME_CONTEXT ? launch<SBW_DTYPE_F32, SBW_SCHEME_CONTEXT, true, true>(a, stream)
                                            : launch<SBW_DTYPE_F32, SBW_SCHEME_SELFSALT, true, true>(a, stream);
    }
    return scheme == SBW_SCHEME_CONTEXT ? launch<SBW_DTYPE_BF16, SBW_SCHEME_CONTEXT, true, true>(a, stream)
                                        : launch<SBW_DTYPE_BF16, SBW_SCHEME_SELFSALT, true, true>(a, stream);
}

}  // namespace sbw

extern "C" int sbw_bias_logits(void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                               int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width,
                               uint64_t key, double gamma, float delta, int scheme, void *stream) {
    return sbw::bias_logits_impl(logits, dtype, B, V, ld, vocab_offset, ctx_tokens, ctx_width, key,
                                 gamma, delta, scheme, static_cast<cudaStream_t>(stream));
}

extern "C" size_t sbw_bias_logits_host_staging_bytes(int dtype, int64_t B, int64_t ld, int ctx_width) {
    if ((dtype != SBW_DTYPE_F32 && dtype != SBW_DTYPE_BF16) || B < 0 || ld < 0 || ctx_width < 0) return 0;
    const size_t esize = dtype == SBW_DTYPE_F32 ? 4 : 2;
    return sbw::align_up(static_cast<size_t>(B) * ld * esize, 256) +
           sbw::align_up(static_cast<size_t>(B) * ctx_width * sizeof(int32_t), 256);
}

extern "C" int sbw_bias_logits_host(void *logits_host, int dtype, int64_t B, int64_t V, int64_t ld,
                                    int64_t vocab_offset, const int32_t *ctx_tokens_host,
                                    int ctx_width, uint64_t key, double gamma, float delta,
                                    int scheme, void *staging, size_t staging_bytes, void *stream) {
    if (!sbw::valid_common(dtype, ctx_width, gamma, scheme)) return SBW_ERR_INVALID_ARG;
    if (B < 0 || V <= 0 || ld < V || vocab_offset < 0) return SBW_ERR_INVALID_ARG;
    if (B == 0) return SBW_OK;
    if (!logits_host || !ctx_tokens_host) return SBW_ERR_INVALID_ARG;
    const size_t need = sbw_bias_logits_host_staging_bytes(dtype, B, ld, ctx_width);
    if (!staging || staging_bytes < need || reinterpret_cast<uintptr_t>(staging) % 256 != 0)
        return SBW_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t esize = dtype == SBW_DTYPE_F32 ? 4 : 2;
    const size_t lbytes = static_cast<size_t>(B) * ld * esize;
    const size_t cbytes = static_cast<size_t>(B) * ctx_width * sizeof(int32_t);
    char *d_logits = static_cast<char *>(staging);
    int32_t *d_ctx = reinterpret_cast<int32_t *>(d_logits + sbw::align_up(lbytes, 256));
    // every check the device entry makes, before anything is enqueued
    sbw::BiasArgs probe;
    bool run = false;
    if (int rc = sbw::prepare(probe, d_logits, dtype, B, V, ld, vocab_offset, d_ctx, ctx_width, key, gamma, delta,
                              scheme, &run))
        return rc;
    if (!run) return SBW_OK;      // a bias that is zero in the logits' precision changes no bit: no copy needed
    SBW_CUDA_TRY(cudaMemcpyAsync(d_ctx, ctx_tokens_host, cbytes, cudaMemcpyHostToDevice, s));
    SBW_CUDA_TRY(cudaMemcpyAsync(d_logits, logits_host, lbytes, cudaMemcpyHostToDevice, s));
    const int rc = sbw::bias_logits_impl(d_logits, dtype, B, V, ld, vocab_offset, d_ctx, ctx_width, key,
                                         gamma, delta, scheme, s);
    if (rc != SBW_OK) return rc;
    SBW_CUDA_TRY(cudaMemcpyAsync(logits_host, d_logits, lbytes, cudaMemcpyDeviceToHost, s));
    return SBW_OK;
}
