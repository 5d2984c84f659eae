/*
 * sbw.h -- C ABI of the B200 (sm_100a) library for Stateless Bernoulli Watermarking (SBW).
 *
 * The library is the data-parallel hot path of the method: the per-decode-step logits bias
 * (Section 2.2, Eq. 1 and Eq. 2 of the paper), the same bias fused with temperature softmax and
 * Gumbel-max sampling, and batch detection (Section 2.2 "Detection", Eq. 5).  Every step runs
 * in hand-written CUDA kernels; there is no CPU fallback and no other backend.
 *
 * Conventions for every call
 *   - Pointers are DEVICE pointers owned by the caller unless a parameter says "host".
 *   - The library allocates nothing, frees nothing and never synchronises: work is enqueued on
 *     `stream` (a cudaStream_t passed as void*, NULL = the legacy default stream) and the call
 *     returns at once.  Scratch memory, where a call needs it, is passed in as `workspace`.
 *   - Return value: SBW_OK or a negative SBW_ERR_* code.  Nothing is enqueued when an argument
 *     is rejected.  After SBW_ERR_CUDA, sbw_last_cuda_error() returns the cudaError_t seen by
 *     the calling thread.  No exceptions, no exit(), no device-side traps.
 *   - Token ids are reinterpreted as unsigned 32-bit values; any bit pattern gives a
 *     deterministic result and is never used as an address.
 *   - B == 0 or N == 0 is SBW_OK and launches nothing.
 *
 * Readings taken where the paper names an operation without printing it ("SBW-spec v1"):
 *   Jenkins hash J      (Section 2.3)  a=(a+0x7ed55d16)+(a<<12); a=(a^0xc761c23c)^(a>>19);
 *                                      a=(a+0x165667b1)+(a<<5);  a=(a+0xd3a2646c)^(a<<9);
 *                                      a=(a+0xfd7046c5)+(a<<3);  a=(a^0xb55a4f09)^(a>>16)
 *   CBRNG               (Section 2.2)  x = word 0 of Philox4x32-10(counter (v,0,0,0),
 *                                      key (lo32 r, hi32 r)), v = vocab_offset + column
 *   green               (Eq. 1)        x < ceil(gamma * 2^32)   (strict, integer compare)
 *   seed r, CONTEXT     (Table 12, "additive")          r = key * (sum of the ctx ids)  mod 2^64
 *   seed r, SELFSALT    (Table 12, "anchored minhash";  r = key * J(v) * min(J(v), min_i J(ctx_i))
 *                        Section 5.2, every candidate)      mod 2^64, J(.)J(.) taken in 64 bits
 *   bias                (Eq. 2)        green: one round-to-nearest-even add of delta in the
 *                                      logits' precision (bf16: delta rounded to bf16 first);
 *                                      not green: value unchanged
 */
#ifndef SBW_H
#define SBW_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SBW_OK 0
#define SBW_ERR_INVALID_ARG (-1) /* null required pointer, size < 0, ld < V, gamma outside (0,1), ... */
#define SBW_ERR_UNSUPPORTED (-2) /* a value the ABI reserves but this build does not implement */
#define SBW_ERR_WORKSPACE (-3)   /* workspace missing, misaligned or too small */
#define SBW_ERR_CUDA (-4)        /* a CUDA runtime call failed; see sbw_last_cuda_error() */
#define SBW_ERR_TOO_LARGE (-5)   /* the problem exceeds a fixed built-in capacity (see the call) */

#define SBW_SCHEME_CONTEXT 0  /* seed from the preceding tokens only (SBW-1, SBW-4) */
#define SBW_SCHEME_SELFSALT 1 /* seed from the preceding tokens and the candidate (SBW-ss-V) */

#define SBW_DTYPE_F32 0  /* IEEE binary32 logits */
#define SBW_DTYPE_BF16 1 /* bfloat16 logits */

#define SBW_MAX_CTX_WIDTH 8

/* Library version string (static storage, host). */
const char *sbw_version(void);

/* cudaError_t recorded by the calling thread's last call that returned SBW_ERR_CUDA, else 0. */
int sbw_last_cuda_error(void);

/*
 * sbw_bias_logits -- Eq. 1 + Eq. 2, one decode step, in place, one pass, no mask tensor
 * (Section 5.1: in-place mutation, a single CBRNG evaluation per token, no CPU synchronisation).
 *
 *   logits       in/out, device, [B, ld] row-major, element type `dtype`; columns 0..V-1 of each
 *                row are biased, columns V..ld-1 are neither read nor written.  Any alignment is
 *                accepted; rows that start on 16-byte boundaries take the vectorised path.
 *   B, V, ld     rows, vocabulary columns, row stride in elements (ld >= V > 0, B >= 0).
 *   vocab_offset global id of column 0 (>= 0; non-zero when the vocabulary is sharded);
 *                vocab_offset + V may not exceed 2^32 (ids are 32-bit), else SBW_ERR_UNSUPPORTED.
 *   ctx_tokens   device, [B, ctx_width] int32: the ctx_width tokens preceding the one being
 *                generated, per row.  1 <= ctx_width <= SBW_MAX_CTX_WIDTH.
 *   key          64-bit secret key.      gamma  green fraction, 0 < gamma < 1.
 *   delta        bias added to green logits (any finite float; 0 leaves every bit unchanged).
 *   scheme       SBW_SCHEME_*.           stream cudaStream_t.
 * NaN logits stay NaN (payload unspecified); +-inf follow IEEE addition.
 */
int sbw_bias_logits(void *logits, int dtype, int64_t B, int64_t V, int64_t ld, int64_t vocab_offset,
                    const int32_t *ctx_tokens, int ctx_width, uint64_t key, double gamma,
                    float delta, int scheme, void *stream);

/*
 * sbw_bias_logits_topk -- the paper's SBW-ss scheme (Table 1: Bernoulli list, self-salt, candidates
 * "top-40"; Section 5.2 describes the top-k restriction it inherits from KGW): per row only the
 * top_k largest logits are tested (Eq. 1) and biased (Eq. 2); every other element of the row
 * keeps its bits.  "Largest" is the total order on order-encoded bit patterns -- +NaN > +inf >
 * ... > +0 > -0 > ... > -inf > -NaN -- with ties to the lowest column (the paper states no tie
 * rule).  Arguments as for sbw_bias_logits; top_k >= 1; top_k >= V is the full-vocabulary call.
 * Needs no workspace.  Fast for ordinary rows and top_k <= 256; rows of mostly equal values or
 * larger top_k take a slow, exact fallback (top_k block reductions per row).
 */
int sbw_bias_logits_topk(void *logits, int dtype, int64_t B, int64_t V, int64_t ld, int64_t vocab_offset,
                         const int32_t *ctx_tokens, int ctx_width, uint64_t key, double gamma,
                         float delta, int scheme, int64_t top_k, void *stream);

/*
 * sbw_bias_logits_host -- the same step for callers whose logits live in HOST memory: copies
 * B*ld elements and the context tokens to the device staging buffer, runs sbw_bias_logits on
 * it, and copies the logits back, all enqueued on `stream` (the copies are asynchronous only if
 * the host buffers are page-locked).  The paper has the logits on the GPU already; this entry
 * exists so that end-to-end cost including the PCIe transfers can be measured.
 *
 *   logits_host  in/out, HOST, [B, ld].        ctx_tokens_host  HOST, [B, ctx_width] int32.
 *   staging      device scratch of at least sbw_bias_logits_host_staging_bytes(...) bytes,
 *                256-byte aligned; owned by the caller, contents undefined afterwards.
 * The results are in logits_host once `stream` has been synchronised by the caller.
 */
size_t sbw_bias_logits_host_staging_bytes(int dtype, int64_t B, int64_t ld, int ctx_width);
int sbw_bias_logits_host(void *logits_host, int dtype, int64_t B, int64_t V, int64_t ld,
                         int64_t vocab_offset, const int32_t *ctx_tokens_host, int ctx_width,
                         uint64_t key, double gamma, float delta, int scheme, void *staging,
                         size_t staging_bytes, void *stream);

/*
 * sbw_bias_sample -- the bias of Eq. 1 + Eq. 2 fused with temperature softmax statistics and
 * Gumbel-max sampling, one pass over read-only logits.  The paper leaves sampling to the
 * serving engine (Section 5.1 speaks of absorbing the watermark into existing logit
 * post-processing); this call is that absorption.  Per row b, with l'_v the biased logit in the
 * logits' own precision and tau = temperature:
 *     m  = max_v l'_v                      Z = sum_v exp((l'_v - m) / tau)
 *     id = argmax_v fmaf(l'_v, 1/tau, g_v)  (fp32, 1/tau rounded once; ties -> lowest v)
 *     p  = exp((l'_id - m) / tau) / Z
 * g_v = -L(-L(u_v)) is a standard Gumbel variate from a counter-based stream of its own:
 *     y   = word (vg & 3) of Philox4x32-10(counter (vg >> 2, b, lo32 rng_step, hi32 rng_step),
 *           key (lo32 rng_seed, hi32 rng_seed)),  vg = vocab_offset + v
 *     u_v = ((y >> 9) + 0.5) * 2^-23
 * and L is a fixed fp32 logarithm made of exactly rounded operations (see sbw_sample.cu), so
 * that `out_tokens` is reproducible bit for bit on any IEEE machine.
 *
 *   logits        device, read only, [B, ld] of `dtype`.
 *   temperature   tau > 0.                 rng_seed, rng_step  select the Gumbel stream; use a
 *                 new rng_step for every decode step.
 *   out_tokens    device [B] int32: sampled column index (0-based within this shard).
 *   out_max, out_sumexp, out_prob   device [B] float, each may be NULL: m, Z, p.
 *   out_probs     device [B, V] float or NULL: the full softmax of the biased logits
 *                 (costs a second pass; meant for tests and small batches).
 *                 With all four NULL only the ids are produced, and the green test is evaluated
 *                 only for candidates whose Gumbel variate could make them win (same ids, about
 *                 twice the throughput).
 *   workspace     device scratch, 256-byte aligned, at least
 *                 sbw_sample_workspace_bytes(B, V) bytes; contents undefined afterwards.
 *                 Calls that share a workspace must not overlap on the GPU.
 * Rows whose logits are all -inf return id 0; m, Z, p of such rows, and every output of rows
 * that contain NaN or +inf, are unspecified.
 */
size_t sbw_sample_workspace_bytes(int64_t B, int64_t V);
int sbw_bias_sample(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                    int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width, uint64_t key,
                    double gamma, float delta, int scheme, float temperature, uint64_t rng_seed,
                    uint64_t rng_step, int32_t *out_tokens, float *out_max, float *out_sumexp,
                    float *out_prob, float *out_probs, void *workspace, size_t workspace_bytes,
                    void *stream);

/*
 * sbw_bias_sample_shard / sbw_sample_combine -- fused sampling of rows whose vocabulary is split
 * over S shards (tensor-parallel language-model heads).  The paper states that every device can
 * derive identical green lists from the shared key (Limitations) and leaves it unvalidated; with
 * these two calls no shard reads another shard's logits and 32 bytes per row and shard are all
 * that has to be exchanged.
 *
 * sbw_bias_sample_shard is sbw_bias_sample on one shard: `logits` holds columns vocab_offset ..
 * vocab_offset+V-1 of rows row_offset .. row_offset+B-1 (row_offset enters the Gumbel counter, so
 * a shard of the rows draws the same variates as the whole batch would; sbw_bias_sample uses 0).
 *   out_shard   device, 16-byte aligned, [B, 8] float: per row (m, Z, best score s, GLOBAL id of
 *               the best candidate as int bits, its biased logit, 0, 0, 0) of this shard.
 *   out_tokens  device [B] int32: the shard-local column of that candidate (required).
 *   vocab_offset + V may not exceed 2^31 here (the summary holds the global id as a signed
 *   32-bit value), else SBW_ERR_UNSUPPORTED.
 * sbw_sample_combine merges S such summaries laid out [S, B, 8] (shard-major, e.g. the result of
 * an all-gather): m = max m_r, Z = sum Z_r exp((m_r - m)/tau) in fp64, id = the global id with
 * the largest s (ties -> lowest global id), p = exp((l_id - m)/tau)/Z.  out_max / out_sumexp /
 * out_prob may be NULL.  The combined id, m, and (to 1e-6 relative) Z and p equal what
 * sbw_bias_sample returns on the unsplit rows.
 */
int sbw_bias_sample_shard(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                          int64_t vocab_offset, int64_t row_offset, const int32_t *ctx_tokens,
                          int ctx_width, uint64_t key, double gamma, float delta, int scheme,
                          float temperature, uint64_t rng_seed, uint64_t rng_step, float *out_shard,
                          int32_t *out_tokens, void *workspace, size_t workspace_bytes, void *stream);
int sbw_sample_combine(const float *shards, int64_t S, int64_t B, float temperature,
                       int32_t *out_tokens, float *out_max, float *out_sumexp, float *out_prob,
                       void *stream);

/*
 * sbw_bias_sample_shard_ids -- sbw_bias_sample_shard for callers that want the global ids only:
 * same arguments and summary layout, but the summary carries no statistics (m = -inf, Z = 0), so
 * the shard takes the ids-only path of sbw_bias_sample (the green test runs only for candidates
 * that could win).  sbw_sample_combine on such summaries gives the same out_tokens; its m, Z and
 * p outputs must then be NULL.
 */
int sbw_bias_sample_shard_ids(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                              int64_t vocab_offset, int64_t row_offset, const int32_t *ctx_tokens,
                              int ctx_width, uint64_t key, double gamma, float delta, int scheme,
                              float temperature, uint64_t rng_seed, uint64_t rng_step, float *out_shard,
                              int32_t *out_tokens, void *workspace, size_t workspace_bytes, void *stream);

/*
 * sbw_bias_sample_noalloc -- sbw_bias_sample for callers that cannot hand over a workspace.
 * The paper has no counterpart for this call; it exists for deployment.  Some users of this
 * library cannot allocate device memory at all: a logits processor plugged into a serving
 * engine that gave every free byte of the GPU to its KV-cache pool at start-up, or a component
 * that runs inside another process under a fixed memory budget.  For them cudaMalloc either
 * fails or stalls the whole device, so this variant needs none: the scratch that
 * sbw_bias_sample takes as `workspace` lives in a fixed array inside the library instead
 * (256 KiB of device memory, held by every GPU that loads the library until the process exits).
 *
 * Arguments and results are exactly those of sbw_bias_sample without `workspace` and
 * `workspace_bytes`; inputs and outputs are still the caller's.  Differences:
 *   - B may be at most SBW_NOALLOC_MAX_ROWS; a larger batch returns SBW_ERR_TOO_LARGE and
 *     enqueues nothing (split it, or use sbw_bias_sample).  The other arguments are checked
 *     first, so a call that is wrong in another way as well reports that.
 *   - The first call on each device looks up the array's device address (with that device
 *     current) before launching; make that first call outside any stream capture.
 *   - All calls on a device share the one array.  The library clears what has to start at zero
 *     on every call, but two calls that overlap on the GPU (different streams, no ordering
 *     between them) race on it and give undefined results: order them.
 * The call itself allocates nothing: no cudaMalloc, no cudaFree, no allocating library routine.
 */
#define SBW_NOALLOC_MAX_ROWS 4096
int sbw_bias_sample_noalloc(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                            int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width,
                            uint64_t key, double gamma, float delta, int scheme, float temperature,
                            uint64_t rng_seed, uint64_t rng_step, int32_t *out_tokens,
                            float *out_max, float *out_sumexp, float *out_prob, float *out_probs,
                            void *stream);

/*
 * sbw_detect -- batch detection (Section 2.2 "Detection": one membership test per token, no
 * green list is built; Eq. 5 for the score).  For sequence s with tokens t_0..t_{L-1}:
 *     scored positions  i = W .. L-1  (the first W = ctx_width tokens only seed), T = max(L-W, 0)
 *     Y_i = green(seed(t_{i-W..i-1}[, t_i]), v = t_i),   G = sum Y_i
 *     z   = (G - gamma T) / sqrt(T gamma (1 - gamma))     in fp64;  T = 0 gives G = 0, z = 0.
 *
 *   tokens        device, int32, the N sequences back to back (total_tokens ids).
 *   lengths       device [N] int32 (negative values count as 0).
 *   offsets       device [N+1] int64 start of each sequence in `tokens`, or NULL: the library
 *                 then scans `lengths` into the workspace first.
 *   total_tokens  number of ids in `tokens`; positions at or beyond it are never read, and a
 *                 sequence that would run past it is scored only up to it.
 *   out_counts    device [N] int32: G.    out_T  device [N] int32 or NULL: T.
 *   out_z         device [N] double: z.
 *   workspace     device scratch, 256-byte aligned, at least sbw_detect_workspace_bytes(N) bytes
 *                 (may be NULL with size 0 when `offsets` is given).
 */
size_t sbw_detect_workspace_bytes(int64_t N);
int sbw_detect(const int32_t *tokens, const int32_t *lengths, const int64_t *offsets, int64_t N,
               int64_t total_tokens, int ctx_width, uint64_t key, double gamma, int scheme,
               int32_t *out_counts, int32_t *out_T, double *out_z, void *workspace,
               size_t workspace_bytes, void *stream);

/*
 * sbw_detect_bits -- sbw_detect that also keeps the per-token indicators Y_i of Section 3 (the
 * paper's robustness study, Appendix G, scores cut and edited text; partly watermarked text needs
 * more than one count per sequence).  Arguments and results as for sbw_detect, plus
 *   out_bits   device, uint32[sbw_detect_bits_words(N, total_tokens)].  The bits of sequence s
 *              start at word (offset_s >> 5) + 2 s; scored position i (token W + i) is bit i & 31
 *              of word i >> 5 of that region; ceil(T / 32) words per sequence are written, unused
 *              high bits of the last one are 0, other words are left as they were.
 * When `offsets` is NULL the scanned int64[N + 1] offsets are left at the start of `workspace`,
 * where sbw_window_z can read them.
 *
 * sbw_window_z -- windowed detection on those bits: per sequence, the window of `window`
 * consecutive scored positions (all T of them if T < window) with the most green tokens, ties to
 * the earliest start, and Eq. 5 on that window.  T = 0 gives count 0, start 0, z 0.
 *   bits, lengths, offsets (required, device), total_tokens, ctx_width  as used by sbw_detect_bits.
 *   prefix_scratch  device, uint32[sbw_detect_bits_words(N, total_tokens)], contents undefined after.
 *   out_count, out_start  device [N] int32;  out_z  device [N] double.
 */
size_t sbw_detect_bits_words(int64_t N, int64_t total_tokens);
int sbw_detect_bits(const int32_t *tokens, const int32_t *lengths, const int64_t *offsets, int64_t N,
                    int64_t total_tokens, int ctx_width, uint64_t key, double gamma, int scheme,
                    int32_t *out_counts, int32_t *out_T, double *out_z, uint32_t *out_bits,
                    void *workspace, size_t workspace_bytes, void *stream);
int sbw_window_z(const uint32_t *bits, const int32_t *lengths, const int64_t *offsets, int64_t N,
                 int64_t total_tokens, int ctx_width, int64_t window, double gamma,
                 uint32_t *prefix_scratch, int32_t *out_count, int32_t *out_start, double *out_z,
                 void *stream);

/*
 * sbw_prefix_z -- detection on truncated text (the paper's robustness study, Appendix G, cuts
 * text to a prefix): Eq. 5 over the first keep[s] tokens of sequence s only, from the bits
 * sbw_detect_bits stored.  keep is clamped to [0, length]; T = max(keep - W, 0); T = 0 gives z 0.
 *   bits, lengths, offsets (required, device), total_tokens, ctx_width  as used by sbw_detect_bits.
 *   keep        device [N] int32.
 *   out_counts  device [N] int32;  out_T  device [N] int32 or NULL;  out_z  device [N] double.
 */
int sbw_prefix_z(const uint32_t *bits, const int32_t *lengths, const int64_t *offsets, const int32_t *keep,
                 int64_t N, int64_t total_tokens, int ctx_width, double gamma, int32_t *out_counts,
                 int32_t *out_T, double *out_z, void *stream);

/*
 * sbw_detect_unique -- sbw_detect that scores every distinct (context, token) tuple of a sequence
 * once (what KGW-family detectors call "ignore repeated n-grams"; Section 3 of the paper treats the
 * indicators Y_i as independent trials, which repeated text is not).  A scored position t counts
 * iff no earlier scored position of the same sequence has the same W + 1 tokens tok[t-W .. t];
 * out_T is the number of such positions, out_counts the green ones among them, out_z Eq. 5 on
 * the two.  Arguments as for sbw_detect, plus
 *   max_length  an upper bound on every length.  Sequences with more than 1536 scored tokens keep
 *               their hash set in the workspace; the workspace holds room for that only if
 *               max_length says such sequences exist.  A sequence longer than max_length that
 *               needs that room is not scored: count -1, T -1, z NaN.
 *   workspace   device, 256-byte aligned, at least
 *               sbw_detect_unique_workspace_bytes(N, total_tokens, max_length) bytes (always
 *               required; 16 bytes per token more when max_length > 1537).
 */
size_t sbw_detect_unique_workspace_bytes(int64_t N, int64_t total_tokens, int64_t max_length);
int sbw_detect_unique(const int32_t *tokens, const int32_t *lengths, const int64_t *offsets, int64_t N,
                      int64_t total_tokens, int64_t max_length, int ctx_width, uint64_t key, double gamma,
                      int scheme, int32_t *out_counts, int32_t *out_T, double *out_z, void *workspace,
                      size_t workspace_bytes, void *stream);

/*
 * sbw_roc_auc -- Section 4.3: area under the ROC curve of z-scores as a detector of label 1
 * (watermarked) against label 0, computed exactly as the pair statistic
 *   AUC = (2 #{z_pos > z_neg} + #{z_pos == z_neg}) / (2 n_pos n_neg),
 * which equals the trapezoid area under the (FPR, TPR) curve swept over every threshold.  NaN
 * scores are left out of both classes; -0 and +0 tie.
 *   z          device [n] double;  labels  device [n] uint8 (0 or non-zero);  n <= 2^31.
 *   out_auc    device double[1]; NaN when a class is empty.
 *   out_stats  device uint64[4] or NULL: {pairs greater, pairs equal, n_pos, n_neg}.
 *   workspace  device, 256-byte aligned, at least sbw_roc_auc_workspace_bytes(n) bytes.
 */
size_t sbw_roc_auc_workspace_bytes(int64_t n);
int sbw_roc_auc(const double *z, const uint8_t *labels, int64_t n, double *out_auc, uint64_t *out_stats,
                void *workspace, size_t workspace_bytes, void *stream);

/*
 * sbw_roc_auc_batched -- M independent ROC-AUCs in one launch (the paper's Table 4 holds one AUC per
 * configuration, each over 500 watermarked and 500 unmarked texts).  Problem i is the scores and
 * labels [offsets[i], offsets[i + 1]) of the flat arrays; each result is what sbw_roc_auc gives on
 * that slice.  One CTA per problem: meant for many problems of up to a few ten thousand scores.
 *   z, labels   device, flat;  offsets  device int64[M + 1], non-decreasing.
 *   out_auc     device double[M];  out_stats  device uint64[4 M] or NULL.
 * Needs no workspace.
 */
int sbw_roc_auc_batched(const double *z, const uint8_t *labels, const int64_t *offsets, int64_t M,
                        double *out_auc, uint64_t *out_stats, void *stream);

/*
 * sbw_bias_sample_filtered -- sbw_bias_sample on the top-k / top-p truncated distribution (the
 * paper's Appendix F samples with temperature 0.7 and top_p = 0.8; the paper gives no arithmetic
 * for the truncation, the one below is this library's).  Per row, with l' the biased logits of Eq. 2:
 *   order    candidates are ranked by order-encoded bit pattern, descending, ties to the lowest
 *            column (the order of sbw_bias_logits_topk); m is the first one's value.
 *   top_k    > 0 keeps the first min(top_k, V) of the order; 0 switches the filter off.
 *   top_p    < 1 keeps candidate i of what top_k left iff the integer weights of the candidates
 *            before it sum to S with S 2^32 < floor(top_p 2^32) Z, Z being the sum over all of
 *            them; >= 1 switches the filter off; must be > 0.  The weight of a candidate is 2^40
 *            for the bits of m, else with c = (float)(log2(e) / (double)temperature), y = (l' - m) c
 *            in fp32: 0 if not y >= -41, else trunc(2^(40 + n) P(y - n)), n = rintf(y), P the
 *            degree-7 Taylor polynomial of 2^f with coefficients rounded to fp32, evaluated by
 *            Horner's rule with fused multiply-adds.  The sums are exact, so the kept set does
 *            not depend on the order of addition.
 *   sample   arg max over the kept candidates of fmaf(l', 1 / temperature, g), g the Gumbel
 *            variate sbw_bias_sample draws for (rng_seed, rng_step, row, vocab_offset + column),
 *            ties to the lowest column.  With both filters off the ids equal sbw_bias_sample's.
 * Arguments as for sbw_bias_sample (logits are not modified), plus
 *   out_tokens  device [B] int32: the sampled column per row.
 *   out_kept    device [B] int32 or NULL: the number of candidates left per row.
 *   workspace   device, 256-byte aligned, at least sbw_sample_filtered_workspace_bytes(dtype, B, V)
 *               bytes (a biased copy of the logits); contents undefined afterwards.
 * With top_k set and 16-byte aligned rows the full-vocabulary hash is not evaluated: the columns that
 * can reach the biased top-k are found on the unbiased logits (l >= k-th largest l - |delta|) and only
 * they are hashed; the result is the same.
 * Rows that contain NaN are not supported (the result is some kept column).  V <= 2^21
 * (SBW_ERR_UNSUPPORTED beyond: the weight histogram's counters hold that many candidates).
 */
size_t sbw_sample_filtered_workspace_bytes(int dtype, int64_t B, int64_t V);
int sbw_bias_sample_filtered(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                             int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width, uint64_t key,
                             double gamma, float delta, int scheme, float temperature, int64_t top_k,
                             double top_p, uint64_t rng_seed, uint64_t rng_step, int32_t *out_tokens,
                             int32_t *out_kept, void *workspace, size_t workspace_bytes, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SBW_H */
