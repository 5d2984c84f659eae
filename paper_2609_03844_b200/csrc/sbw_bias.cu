// sbw_bias_logits: Eq. 1 + Eq. 2 of the paper in one in-place pass over the [B, V] logits.
//
// Layout of the work.  A row is cut into 16-byte "slots" (4 fp32 or 8 bf16 logits); the B*nslot
// slots form one flat index space that is divided evenly over a persistent grid (a multiple of
// the SM count), so every SM receives the same number of slots whatever B and V are.  A block
// walks its share row by row: per row it derives the seed material once (context scheme: the ten
// Philox round keys; self-salt scheme: the smallest context hash), then its threads stride over
// the row's slots.  Per slot a thread issues one 128-bit load, evaluates the 4 or 8 independent
// hash chains in registers (that independence is the instruction-level parallelism that keeps
// the integer pipes busy), applies the bias, and issues one 128-bit store.  No shared memory, no
// mask tensor, no other global traffic.  Rows that do not start on 16-byte boundaries, and the
// ragged last slot of a row, go through the same code one element at a time.
#include <cuda_bf16.h>

#include "sbw_common.cuh"
#include "sbw_hash.cuh"

namespace sbw {
namespace {

constexpr int kBiasThreads = 256;

struct BiasArgs {
    void *logits;
    int64_t B, V, ld;
    int64_t nslot;          // slots per row
    int64_t total;          // B * nslot
    const int32_t *ctx;
    int W;
    uint32_t vocab_offset;  // global id of column 0 (mod 2^32)
    uint64_t key;
    uint32_t thr_m1;        // green <=> x <= thr_m1
    float delta;            // fp32 path: delta; bf16 path: delta rounded to bf16, widened
    uint32_t delta_bf16;    // bf16 bits of delta
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
    __device__ __forceinline__ uint32_t word0(uint32_t v, uint64_t) const { return philox_word0(v, rk); }
};
template <>
struct RowSeed<SBW_SCHEME_SELFSALT> {
    uint32_t jmin;
    __device__ __forceinline__ void init(uint64_t, const int32_t *ctx, int W) { jmin = jenkins_min(ctx, W); }
    __device__ __forceinline__ uint32_t word0(uint32_t v, uint64_t key) const {
        return philox_word0(v, seed_selfsalt(key, jmin, v));
    }
};

// One logit, any alignment: used for ragged tails and for rows that are not 16-byte aligned.
template <int DTYPE, int SCHEME>
__device__ __forceinline__ void bias_one(const BiasArgs &a, const RowSeed<SCHEME> &rs, void *row_ptr,
                                         uint32_t col) {
    const uint32_t v = a.vocab_offset + col;
    const bool green = rs.word0(v, a.key) <= a.thr_m1;
    if (!green) return;
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

template <int DTYPE, int SCHEME, bool VECTOR>
__global__ void __launch_bounds__(kBiasThreads)
bias_kernel(const BiasArgs a) {
    constexpr int VEC = VECTOR ? (DTYPE == SBW_DTYPE_F32 ? 4 : 8) : 1;
    constexpr int ESIZE = DTYPE == SBW_DTYPE_F32 ? 4 : 2;
    const int64_t s_begin = a.total / gridDim.x * blockIdx.x +
                            (a.total % gridDim.x) * blockIdx.x / gridDim.x;
    const int64_t s_end = a.total / gridDim.x * (blockIdx.x + 1) +
                          (a.total % gridDim.x) * (blockIdx.x + 1) / gridDim.x;
    if (s_begin >= s_end) return;
    int64_t row = s_begin / a.nslot;
    uint32_t col = static_cast<uint32_t>(s_begin - row * a.nslot);
    int64_t left = s_end - s_begin;
    const uint32_t nslot = static_cast<uint32_t>(a.nslot);
    const uint32_t V = static_cast<uint32_t>(a.V);

    while (left > 0) {
        const uint32_t seg = static_cast<uint32_t>(min(static_cast<int64_t>(nslot - col), left));
        RowSeed<SCHEME> rs;
        rs.init(a.key, a.ctx + row * a.W, a.W);
        char *row_ptr = static_cast<char *>(a.logits) + row * a.ld * ESIZE;
        const uint32_t j_end = col + seg;
        for (uint32_t j = col + threadIdx.x; j < j_end; j += kBiasThreads) {
            const uint32_t cb = j * VEC;
            if constexpr (!VECTOR) {
                bias_one<DTYPE, SCHEME>(a, rs, row_ptr, cb);
            } else {
                if (cb + VEC > V) {  // ragged last slot of the row
                    for (uint32_t c = cb; c < V; ++c) bias_one<DTYPE, SCHEME>(a, rs, row_ptr, c);
                    continue;
                }
                uint4 *p = reinterpret_cast<uint4 *>(row_ptr) + j;
                uint4 w = *p;
                const uint32_t vg = a.vocab_offset + cb;
                bool g[VEC];
#pragma unroll
                for (int i = 0; i < VEC; ++i) g[i] = rs.word0(vg + i, a.key) <= a.thr_m1;
                if constexpr (DTYPE == SBW_DTYPE_F32) {
                    uint32_t *e = reinterpret_cast<uint32_t *>(&w);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float s = __fadd_rn(__uint_as_float(e[i]), a.delta);
                        e[i] = g[i] ? __float_as_uint(s) : e[i];
                    }
                } else {
                    // adding -0.0 returns the other operand unchanged, so a packed add with
                    // {delta or -0.0} per half biases exactly the green halves
                    uint32_t *e = reinterpret_cast<uint32_t *>(&w);
                    const uint32_t dlo = a.delta_bf16, dhi = a.delta_bf16 << 16;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t d = (g[2 * i] ? dlo : 0x8000u) | (g[2 * i + 1] ? dhi : 0x80000000u);
                        e[i] = add_bf16x2(e[i], d);
                    }
                }
                *p = w;
            }
        }
        left -= seg;
        ++row;
        col = 0;
    }
}

template <int DTYPE, int SCHEME, bool VECTOR>
int launch(const BiasArgs &a, cudaStream_t stream) {
    DeviceInfo di;
    int rc = current_device_info(&di);
    if (rc != SBW_OK) return rc;
    static int blocks_per_sm = 0;  // same kernel on every device of a process: B200 only
    if (blocks_per_sm == 0) {
        int n = 0;
        SBW_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, bias_kernel<DTYPE, SCHEME, VECTOR>,
                                                                   kBiasThreads, 0));
        blocks_per_sm = n > 0 ? n : 1;
    }
    const int64_t want = (a.total + kBiasThreads - 1) / kBiasThreads;
    const int64_t cap = static_cast<int64_t>(di.sm_count) * blocks_per_sm;
    const unsigned grid = static_cast<unsigned>(want < cap ? want : cap);
    bias_kernel<DTYPE, SCHEME, VECTOR><<<grid, kBiasThreads, 0, stream>>>(a);
    SBW_CUDA_TRY(cudaGetLastError());
    return SBW_OK;
}

template <int DTYPE, int SCHEME>
int launch_v(const BiasArgs &a, bool vector, cudaStream_t stream) {
    return vector ? launch<DTYPE, SCHEME, true>(a, stream) : launch<DTYPE, SCHEME, false>(a, stream);
}

}  // namespace

int bias_logits_impl(void *logits, int dtype, int64_t B, int64_t V, int64_t ld, int64_t vocab_offset,
                     const int32_t *ctx_tokens, int ctx_width, uint64_t key, double gamma, float delta,
                     int scheme, cudaStream_t stream) {
    if (!valid_common(dtype, ctx_width, gamma, scheme)) return SBW_ERR_INVALID_ARG;
    if (B < 0 || V <= 0 || ld < V || vocab_offset < 0) return SBW_ERR_INVALID_ARG;
    if (V > 0x7fffffffLL || B > (int64_t(1) << 40)) return SBW_ERR_UNSUPPORTED;
    if (!(delta == delta) || delta - delta != 0.0f) return SBW_ERR_INVALID_ARG;  // NaN or inf
    if (B == 0) return SBW_OK;
    if (!logits || !ctx_tokens) return SBW_ERR_INVALID_ARG;

    BiasArgs a;
    a.logits = logits;
    a.B = B; a.V = V; a.ld = ld;
    a.ctx = ctx_tokens;
    a.W = ctx_width;
    a.vocab_offset = static_cast<uint32_t>(vocab_offset);
    a.key = key;
    a.thr_m1 = threshold_minus_one(gamma);
    a.delta = delta;
    a.delta_bf16 = 0;
    const int esize = dtype == SBW_DTYPE_F32 ? 4 : 2;
    if (dtype == SBW_DTYPE_BF16) {
        const __nv_bfloat16 d = __float2bfloat16_rn(delta);
        a.delta_bf16 = static_cast<uint32_t>(__bfloat16_as_ushort(d));
        a.delta = __bfloat162float(d);
    }
    // A bias that is zero in the logits' precision is the paper's delta = 0 control: the logits
    // are left alone bit for bit (an IEEE add of +0 would turn -0 into +0).
    if (a.delta == 0.0f) return SBW_OK;

    const bool vector = (reinterpret_cast<uintptr_t>(logits) % 16 == 0) && ((ld * esize) % 16 == 0);
    const int vec = vector ? 16 / esize : 1;
    a.nslot = (V + vec - 1) / vec;
    a.total = B * a.nslot;

    if (dtype == SBW_DTYPE_F32) {
        return scheme == SBW_SCHEME_CONTEXT
                   ? launch_v<SBW_DTYPE_F32, SBW_SCHEME_CONTEXT>(a, vector, stream)
                   : launch_v<SBW_DTYPE_F32, SBW_SCHEME_SELFSALT>(a, vector, stream);
    }
    return scheme == SBW_SCHEME_CONTEXT
               ? launch_v<SBW_DTYPE_BF16, SBW_SCHEME_CONTEXT>(a, vector, stream)
               : launch_v<SBW_DTYPE_BF16, SBW_SCHEME_SELFSALT>(a, vector, stream);
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
    SBW_CUDA_TRY(cudaMemcpyAsync(d_ctx, ctx_tokens_host, cbytes, cudaMemcpyHostToDevice, s));
    SBW_CUDA_TRY(cudaMemcpyAsync(d_logits, logits_host, lbytes, cudaMemcpyHostToDevice, s));
    const int rc = sbw::bias_logits_impl(d_logits, dtype, B, V, ld, vocab_offset, d_ctx, ctx_width, key,
                                         gamma, delta, scheme, s);
    if (rc != SBW_OK) return rc;
    SBW_CUDA_TRY(cudaMemcpyAsync(logits_host, d_logits, lbytes, cudaMemcpyDeviceToHost, s));
    return SBW_OK;
}
