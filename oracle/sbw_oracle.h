/*
 * sbw_oracle.h -- plain CPU oracle for Stateless Bernoulli Watermarking (SBW).
 *
 * TEST INFRASTRUCTURE, NOT PRODUCT.  This is the slow, step-by-step restatement of the
 * method that the CUDA kernels are compared against.  Only the test-suite, the smoke
 * check and the benchmark's CPU-baseline leg may load it.  It shares no code, header,
 * table or constant generator with the CUDA library and imports nothing from it.
 *
 * Everything is plain C11, one thread per call unless the `_mt` wrapper is used, integer
 * arithmetic unsigned and wrapping (mod 2^32 / 2^64 as typed), floating point compiled
 * with -ffp-contract=off so that every operation written here is one IEEE operation.
 *
 * Parity status of each part (what pins it, see the tests named in parentheses):
 *   jenkins            pinned: frozen known answers, bijection, avalanche   (test_oracle_hash)
 *   philox4x32_10      pinned: cuRAND host generator (library special case) (test_oracle_hash)
 *   seeds, green       pinned: big-integer restatement, Binomial(V,gamma)   (test_oracle_hash,
 *                      green-list statistics of Appendix H                   test_oracle_stats)
 *   bias add           pinned: numpy float32 / torch bfloat16 adds           (test_oracle_bias)
 *   top-k restriction  pinned: torch.topk, brute force on ties, k >= V case  (test_oracle_topk)
 *   detect             pinned: brute force, closed forms, null law of Eq. 5  (test_oracle_detect)
 *   detect_unique,     pinned: Python set of tuples, closed forms; slices of  (test_oracle_eval)
 *   prefix_z, roc_auc  the plain detector; scikit-learn's roc_auc_score,
 *                      exact threshold sweep in rationals, binormal closed form
 *   log / gumbel /     pinned: fp64 log, chi-square of sampled ids against    (test_oracle_sample)
 *   sample             softmax, scipy softmax / logsumexp, closed form
 *   top-k / top-p      pinned: fp64 softmax + cumulative sums (numpy), torch.topk,  (test_oracle_filter)
 *   sampling           2^f in fp64, closed forms, chi-square of sampled ids
 *   bit compatibility with the paper authors' own package: PARITY UNPINNED (the paper
 *   prints no hash input/output pair; the constants below are this library's frozen
 *   reading, "SBW-spec v1").
 */
#ifndef SBW_ORACLE_H
#define SBW_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { SBW_O_SCHEME_CONTEXT = 0, SBW_O_SCHEME_SELFSALT = 1 };
enum { SBW_O_DTYPE_F32 = 0, SBW_O_DTYPE_BF16 = 1 };

/* Section 2.3: integer hash of a token id (reading: six-step 32-bit mix). */
uint32_t sbw_oracle_jenkins(uint32_t a);

/* Section 2.2: the counter-based RNG, Philox 4x32 with 10 rounds. */
void sbw_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);

/* Section 2.2 "seed r_t from the preceding context via a PRF"; Table 12 names the PRFs.
 * ctx points at W token ids (reinterpreted as uint32). */
uint64_t sbw_oracle_seed_context(uint64_t key, const int32_t *ctx, int W);
uint64_t sbw_oracle_seed_selfsalt(uint64_t key, const int32_t *ctx, int W, uint32_t v);

/* Eq. 1: integer form of the threshold gamma, ceil(gamma * 2^32). */
uint64_t sbw_oracle_threshold(double gamma);

/* Eq. 1: 1 if candidate v is green under seed r. */
int sbw_oracle_green(uint64_t r, uint32_t v, uint64_t thr);

/* Eq. 1 for a whole [B,V] step: mask[b*V + j] = green(seed(row b[, candidate]), vocab_offset + j). */
void sbw_oracle_green_mask(uint8_t *mask, int64_t B, int64_t V, int64_t vocab_offset,
                           const int32_t *ctx_tokens, int ctx_width, uint64_t key,
                           double gamma, int scheme);

/* bf16 helpers (round-to-nearest-even narrowing, exact widening). */
uint16_t sbw_oracle_f32_to_bf16(float x);
float sbw_oracle_bf16_to_f32(uint16_t h);

/* Eq. 2 on one element. */
float sbw_oracle_bias_elem_f32(float l, float delta, int green);
uint16_t sbw_oracle_bias_elem_bf16(uint16_t l, float delta, int green);

/* Eq. 2 for a whole step, in place.  logits is [B, ld] of float or of uint16 (bf16 bits).
 * threads <= 1 runs on the calling thread; otherwise rows are split over that many threads. */
void sbw_oracle_bias_logits(void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                            int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width,
                            uint64_t key, double gamma, float delta, int scheme, int threads);

/* Top-k candidate restriction (the paper's SBW-ss scheme, Table 1: self-salt on the top-40
 * candidates only, as KGW's selfhash does).  Per row the k candidates are the k largest logits in
 * the total order "bit pattern order-encoded descending, then column ascending" (so ties go to the
 * lowest ids and every bit pattern, NaN included, has a place); only they are tested and biased.
 * k >= V biases like sbw_oracle_bias_logits.  sel (nullable) receives the chosen columns, [B, min(k,V)],
 * in rank order. */
void sbw_oracle_bias_logits_topk(void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                                 int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width,
                                 uint64_t key, double gamma, float delta, int scheme, int64_t top_k,
                                 int32_t *sel);

/* Eq. 5 and the O(1)-per-token membership test of Section 2.2.
 * tokens: concatenation of N sequences; lengths[N].  Writes counts[N], T[N] (nullable), z[N]. */
void sbw_oracle_detect(const int32_t *tokens, const int32_t *lengths, int64_t N, int ctx_width,
                       uint64_t key, double gamma, int scheme, int32_t *counts, int32_t *T,
                       double *z, int threads);
/* The per-token indicators Y_t of Section 3 themselves: green[offset_s + t] for every token of the
 * flat array (0 for the first W tokens of a sequence, which are not scored). */
void sbw_oracle_detect_bits(const int32_t *tokens, const int32_t *lengths, int64_t N, int ctx_width,
                            uint64_t key, double gamma, int scheme, uint8_t *green);
/* Windowed detection for partly watermarked or truncated text (the paper's robustness study cuts
 * and edits text, Appendix G): over the T scored positions of a sequence, the window of `window`
 * consecutive positions (the whole sequence if T < window) with the most green tokens, ties to
 * the earliest start; Eq. 5 on that window.  T = 0 gives count 0, start 0, z 0. */
void sbw_oracle_window_z(const uint8_t *green, const int32_t *lengths, int64_t N, int ctx_width,
                         int64_t window, double gamma, int32_t *best_count, int32_t *best_start,
                         double *best_z);
/* "Ignore repeated n-grams" detection: every distinct (context, token) tuple of a sequence is
 * scored once; T counts the distinct tuples, counts the green ones among them. */
void sbw_oracle_detect_unique(const int32_t *tokens, const int32_t *lengths, int64_t N, int ctx_width,
                              uint64_t key, double gamma, int scheme, int32_t *counts, int32_t *T,
                              double *z, int threads);
/* Detection on the first keep[s] tokens of each sequence (truncated text, Appendix G), from the
 * per-token array of sbw_oracle_detect_bits. */
void sbw_oracle_prefix_z(const uint8_t *green, const int32_t *lengths, const int32_t *keep, int64_t N,
                         int ctx_width, double gamma, int32_t *counts, int32_t *T, double *z);
/* Section 4.3: ROC-AUC of z against binary labels = P(z_pos > z_neg) + P(z_pos == z_neg) / 2 over
 * all (positive, negative) pairs.  stats (nullable): {greater, equal, n_pos, n_neg}. */
double sbw_oracle_roc_auc(const double *z, const uint8_t *labels, int64_t n, uint64_t stats[4], int threads);
/* Eq. 5 alone. */
double sbw_oracle_zscore(int64_t G, int64_t T, double gamma);

/* Fused sampling (not in the paper; specified by this library, see sbw_oracle.c). */
float sbw_oracle_log(float x);
float sbw_oracle_gumbel_uniform(uint64_t rng_seed, uint64_t rng_step, uint32_t row, uint32_t v_global);
float sbw_oracle_gumbel(uint64_t rng_seed, uint64_t rng_step, uint32_t row, uint32_t v_global);
/* out_probs may be NULL; otherwise [B,V] doubles.  out_max/out_sumexp/out_prob are doubles [B].
 * out_score (nullable) receives the winning s value per row as float. */
void sbw_oracle_bias_sample(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                            int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width,
                            uint64_t key, double gamma, float delta, int scheme,
                            float temperature, uint64_t rng_seed, uint64_t rng_step,
                            int32_t *out_tokens, double *out_max, double *out_sumexp,
                            double *out_prob, double *out_probs, float *out_score, int threads);

/* Fused sampling from the top-k / top-p truncated distribution (Appendix F samples with top_p = 0.8;
 * the integer-weight arithmetic is this library's, see sbw_oracle.c).  top_k = 0 and top_p >= 1 switch
 * the filters off.  out_kept (nullable) [B]: candidates left per row; out_mask (nullable) [B, V]: 1
 * for kept candidates. */
uint64_t sbw_oracle_nucleus_weight(float l, float m, int is_max, float c);
void sbw_oracle_bias_sample_filtered(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                                     int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width,
                                     uint64_t key, double gamma, float delta, int scheme,
                                     float temperature, int64_t top_k, double top_p, uint64_t rng_seed,
                                     uint64_t rng_step, int32_t *out_tokens, int32_t *out_kept,
                                     uint8_t *out_mask, int threads);

/* Exhaustive checks that are too slow from Python; each returns a summary. */
/* Number of 32-bit values hit more than once by jenkins over all 2^32 inputs (0 = bijection).
 * Needs a 512 MiB bitmap, allocated and freed inside. Returns -1 if allocation fails. */
int64_t sbw_oracle_jenkins_collisions(void);
/* Largest error of sbw_oracle_log against fp64 log, in units in the last place of the result,
 * over all 2^23 uniforms u_k = (k + 0.5) 2^-23 (which = 0) or over w_k = -log(u_k) (which = 1). */
double sbw_oracle_log_max_ulp(int which);

#ifdef __cplusplus
}
#endif
#endif
