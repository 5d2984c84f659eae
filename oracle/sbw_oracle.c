/*
 * sbw_oracle.c -- plain CPU oracle for Stateless Bernoulli Watermarking (SBW).
 *
 * TEST INFRASTRUCTURE, NOT PRODUCT (see sbw_oracle.h for who may load it and for the
 * parity status of each function).  Build: gcc -std=c11 -O2 -ffp-contract=off -fopenmp.
 *
 * The paper fixes the structure of the method -- Eq. 1 (Bernoulli green list by a threshold
 * test on a counter-based RNG), Eq. 2 (additive bias), Eq. 5 (z-score), "Philox 4x32-10"
 * (Section 2.2), "Bob Jenkins integer hash" (Section 2.3), the "additive" and "anchored
 * minhash" PRFs (Table 12) -- but prints no formula, constant or worked example for the
 * hashes.  Where it is silent this file takes one reading, frozen as "SBW-spec v1":
 *
 *  R1  Jenkins hash: the 32-bit six-step full-avalanche integer mix (constants below).
 *  R2  Philox: key words (k0,k1) = (lo32 r, hi32 r) of the 64-bit seed r ("seed"), counter
 *      (v,0,0,0) with v the global candidate id ("position"), output word 0.  One Philox
 *      evaluation per candidate, as Section 5.1 promises.
 *  R3  Threshold: u = x 2^-32 < gamma  <=>  x < ceil(gamma 2^32), strict as in Eq. 1; the
 *      threshold is computed once in fp64 and everything after is integer.
 *  R4  "additive" PRF (context scheme):  r = key * (sum of the W context ids) mod 2^64.
 *  R5  "anchored minhash" PRF (self-salt scheme): window = the W context ids followed by the
 *      candidate v; anchor = the candidate; r = key * min_{x in window} J(x) J(v) mod 2^64,
 *      products of two 32-bit hashes taken in 64 bits.
 *  R6  Bias: green -> one IEEE round-to-nearest-even add in the logits' own precision;
 *      not green -> the element's bits are untouched.  bf16: delta is first rounded to bf16.
 *      A delta that is zero in that precision is the paper's delta = 0 control (Section 4.5:
 *      "non-watermarked completions"): nothing is added and every bit stays (an IEEE add of
 *      +0 would turn -0 into +0).
 *  R7  Detection scores positions t = W .. L-1 (the first W tokens only seed), T = max(L-W,0),
 *      every position counted (no repeated-n-gram filter); T = 0 gives G = 0, z = 0.
 *  R9  SBW-ss (Table 1: self-salt, candidates "top-40"): per row only the k largest logits are
 *      tested and biased; "largest" is the total order on order-encoded bit patterns with ties
 *      to the lowest column (the paper inherits KGW's top-k and states no tie rule).
 *  R8  The fused sampler is this library's own (the paper leaves sampling to the engine):
 *      bias first, then temperature; Gumbel-max with a Philox stream of its own and a
 *      fully specified fp32 logarithm so that sampled ids are reproducible bit for bit.
 */
#include "sbw_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ Section 2.3 ---- */
/* R1.  Each step is invertible, so the whole map is a bijection on 32-bit words. */
uint32_t sbw_oracle_jenkins(uint32_t a)
{
    a = (a + 0x7ed55d16u) + (a << 12);
    a = (a ^ 0xc761c23cu) ^ (a >> 19);
    a = (a + 0x165667b1u) + (a << 5);
    a = (a + 0xd3a2646cu) ^ (a << 9);
    a = (a + 0xfd7046c5u) + (a << 3);
    a = (a ^ 0xb55a4f09u) ^ (a >> 16);
    return a;
}

/* ------------------------------------------------------------------ Section 2.2 ---- */
/* Philox 4x32-10: ten rounds; round i uses the key bumped i times by the Weyl constants. */
void sbw_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)M0 * (uint64_t)c0;
        uint64_t p1 = (uint64_t)M1 * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0;
        k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* R4: additive PRF over the context window (Table 12, schemes SBW-1 / SBW-4). */
uint64_t sbw_oracle_seed_context(uint64_t key, const int32_t *ctx, int W)
{
    uint64_t sigma = 0;
    for (int i = 0; i < W; ++i)
        sigma += (uint64_t)(uint32_t)ctx[i];
    return key * sigma;
}

/* R5: anchored minhash PRF (Table 12, scheme SBW-ss-V; Section 5.2: the candidate itself
 * enters the seed, for every candidate of the vocabulary). */
uint64_t sbw_oracle_seed_selfsalt(uint64_t key, const int32_t *ctx, int W, uint32_t v)
{
    uint64_t anchor = (uint64_t)sbw_oracle_jenkins(v);
    uint64_t best = anchor * anchor;            /* the candidate is a member of the window */
    for (int i = 0; i < W; ++i) {
        uint64_t prod = (uint64_t)sbw_oracle_jenkins((uint32_t)ctx[i]) * anchor;
        if (prod < best)
            best = prod;
    }
    return key * best;
}

/* R3. */
uint64_t sbw_oracle_threshold(double gamma)
{
    return (uint64_t)ceil(gamma * 4294967296.0);
}

/* Eq. 1 with R2 and R3. */
int sbw_oracle_green(uint64_t r, uint32_t v, uint64_t thr)
{
    uint32_t ctr[4] = { v, 0u, 0u, 0u };
    uint32_t key[2] = { (uint32_t)r, (uint32_t)(r >> 32) };
    uint32_t out[4];
    sbw_oracle_philox4x32_10(ctr, key, out);
    return (uint64_t)out[0] < thr;
}

static uint64_t seed_for(int scheme, uint64_t key, const int32_t *ctx, int W, uint32_t v)
{
    if (scheme == SBW_O_SCHEME_SELFSALT)
        return sbw_oracle_seed_selfsalt(key, ctx, W, v);
    return sbw_oracle_seed_context(key, ctx, W);
}

void sbw_oracle_green_mask(uint8_t *mask, int64_t B, int64_t V, int64_t vocab_offset,
                           const int32_t *ctx_tokens, int ctx_width, uint64_t key,
                           double gamma, int scheme)
{
    uint64_t thr = sbw_oracle_threshold(gamma);
    for (int64_t b = 0; b < B; ++b) {
        const int32_t *ctx = ctx_tokens + b * ctx_width;
        for (int64_t j = 0; j < V; ++j) {
            uint32_t v = (uint32_t)(vocab_offset + j);
            uint64_t r = seed_for(scheme, key, ctx, ctx_width, v);
            mask[b * V + j] = (uint8_t)sbw_oracle_green(r, v, thr);
        }
    }
}

/* ------------------------------------------------------------------ Eq. 2 ---------- */
float sbw_oracle_bf16_to_f32(uint16_t h)
{
    uint32_t bits = (uint32_t)h << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return f;
}

/* Round-to-nearest-even narrowing of an fp32 value to bf16 (NaN stays NaN). */
uint16_t sbw_oracle_f32_to_bf16(float x)
{
    uint32_t bits;
    memcpy(&bits, &x, sizeof bits);
    if ((bits & 0x7fffffffu) > 0x7f800000u)
        return (uint16_t)((bits >> 16) | 0x0040u);
    uint32_t keep = bits >> 16;
    uint32_t drop = bits & 0xffffu;
    if (drop > 0x8000u || (drop == 0x8000u && (keep & 1u)))
        keep += 1u;
    return (uint16_t)keep;
}

/* R6, fp32 logits. */
float sbw_oracle_bias_elem_f32(float l, float delta, int green)
{
    if (!green || delta == 0.0f)
        return l;
    return l + delta;
}

/* R6, bf16 logits: both operands are bf16 values, the exact sum is rounded once to bf16.
 * The fp32 sum of two bf16 values is exact unless their exponents are more than 16 apart, and
 * then it lies strictly within half a bf16 ulp of the larger operand, so rounding the fp32 sum
 * to bf16 equals rounding the exact sum. */
uint16_t sbw_oracle_bias_elem_bf16(uint16_t l, float delta, int green)
{
    if (!green)
        return l;
    float d = sbw_oracle_bf16_to_f32(sbw_oracle_f32_to_bf16(delta));
    if (d == 0.0f)
        return l;
    float s = sbw_oracle_bf16_to_f32(l) + d;
    return sbw_oracle_f32_to_bf16(s);
}

static void bias_row(void *logits, int dtype, int64_t b, int64_t V, int64_t ld, int64_t vocab_offset,
                     const int32_t *ctx, int W, uint64_t key, uint64_t thr, float delta, int scheme)
{
    for (int64_t j = 0; j < V; ++j) {
        uint32_t v = (uint32_t)(vocab_offset + j);
        uint64_t r = seed_for(scheme, key, ctx, W, v);
        int g = sbw_oracle_green(r, v, thr);
        if (dtype == SBW_O_DTYPE_BF16) {
            uint16_t *p = (uint16_t *)logits + b * ld + j;
            *p = sbw_oracle_bias_elem_bf16(*p, delta, g);
        } else {
            float *p = (float *)logits + b * ld + j;
            *p = sbw_oracle_bias_elem_f32(*p, delta, g);
        }
    }
}

void sbw_oracle_bias_logits(void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                            int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width,
                            uint64_t key, double gamma, float delta, int scheme, int threads)
{
    uint64_t thr = sbw_oracle_threshold(gamma);
    if (threads < 1)
        threads = 1;
#pragma omp parallel for num_threads(threads) schedule(static)
    for (int64_t b = 0; b < B; ++b)
        bias_row(logits, dtype, b, V, ld, vocab_offset, ctx_tokens + b * ctx_width, ctx_width,
                 key, thr, delta, scheme);
}

/* ------------------------------------------------------------------ top-k (SBW-ss) - */
/* Order-preserving code of a logit's bit pattern: larger float, larger code; every pattern
 * (both zeros, infinities, NaNs) gets its own code, so the order is total. */
static uint32_t order_code(uint32_t bits32)
{
    return (bits32 & 0x80000000u) ? ~bits32 : (bits32 | 0x80000000u);
}

typedef struct {
    uint32_t code;
    int64_t col;
} ranked_t;

static int ranked_cmp(const void *pa, const void *pb)
{
    const ranked_t *a = (const ranked_t *)pa, *b = (const ranked_t *)pb;
    if (a->code != b->code)
        return a->code > b->code ? -1 : 1;        /* larger logit first */
    return a->col < b->col ? -1 : (a->col > b->col ? 1 : 0);   /* ties: lowest column first */
}

void sbw_oracle_bias_logits_topk(void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                                 int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width,
                                 uint64_t key, double gamma, float delta, int scheme, int64_t top_k,
                                 int32_t *sel)
{
    uint64_t thr = sbw_oracle_threshold(gamma);
    int64_t k = top_k < V ? top_k : V;
    ranked_t *order = (ranked_t *)malloc((size_t)V * sizeof(ranked_t));
    if (!order)
        return;
    for (int64_t b = 0; b < B; ++b) {
        const int32_t *ctx = ctx_tokens + b * ctx_width;
        for (int64_t j = 0; j < V; ++j) {
            uint32_t bits;
            if (dtype == SBW_O_DTYPE_BF16) {
                bits = (uint32_t)((const uint16_t *)logits)[b * ld + j] << 16;
            } else {
                float f = ((const float *)logits)[b * ld + j];
                memcpy(&bits, &f, sizeof bits);
            }
            order[j].code = order_code(bits);
            order[j].col = j;
        }
        qsort(order, (size_t)V, sizeof(ranked_t), ranked_cmp);
        for (int64_t i = 0; i < k; ++i) {
            int64_t j = order[i].col;
            if (sel)
                sel[b * k + i] = (int32_t)j;
            uint32_t v = (uint32_t)(vocab_offset + j);
            uint64_t r = seed_for(scheme, key, ctx, ctx_width, v);
            int g = sbw_oracle_green(r, v, thr);
            if (dtype == SBW_O_DTYPE_BF16) {
                uint16_t *p = (uint16_t *)logits + b * ld + j;
                *p = sbw_oracle_bias_elem_bf16(*p, delta, g);
            } else {
                float *p = (float *)logits + b * ld + j;
                *p = sbw_oracle_bias_elem_f32(*p, delta, g);
            }
        }
    }
    free(order);
}

/* ------------------------------------------------------------------ Eq. 5 ---------- */
double sbw_oracle_zscore(int64_t G, int64_t T, double gamma)
{
    if (T <= 0)
        return 0.0;                                  /* R7: Eq. 5 is 0/0 there */
    double num = (double)G - gamma * (double)T;
    double den = sqrt((double)T * gamma * (1.0 - gamma));
    return num / den;
}

void sbw_oracle_detect(const int32_t *tokens, const int32_t *lengths, int64_t N, int ctx_width,
                       uint64_t key, double gamma, int scheme, int32_t *counts, int32_t *T,
                       double *z, int threads)
{
    uint64_t thr = sbw_oracle_threshold(gamma);
    int64_t *offsets = (int64_t *)malloc((size_t)(N + 1) * sizeof(int64_t));
    if (!offsets)
        return;
    offsets[0] = 0;
    for (int64_t s = 0; s < N; ++s)
        offsets[s + 1] = offsets[s] + (lengths[s] > 0 ? lengths[s] : 0);
    if (threads < 1)
        threads = 1;
#pragma omp parallel for num_threads(threads) schedule(dynamic, 64)
    for (int64_t s = 0; s < N; ++s) {
        const int32_t *tok = tokens + offsets[s];
        int64_t L = lengths[s] > 0 ? lengths[s] : 0;
        int64_t G = 0;
        for (int64_t t = ctx_width; t < L; ++t) {
            uint32_t v = (uint32_t)tok[t];
            uint64_t r = seed_for(scheme, key, tok + (t - ctx_width), ctx_width, v);
            G += sbw_oracle_green(r, v, thr);        /* Y_t of Section 3 */
        }
        int64_t Ts = L > ctx_width ? L - ctx_width : 0;
        counts[s] = (int32_t)G;
        if (T)
            T[s] = (int32_t)Ts;
        z[s] = sbw_oracle_zscore(G, Ts, gamma);
    }
    free(offsets);
}

void sbw_oracle_detect_bits(const int32_t *tokens, const int32_t *lengths, int64_t N, int ctx_width,
                            uint64_t key, double gamma, int scheme, uint8_t *green)
{
    uint64_t thr = sbw_oracle_threshold(gamma);
    int64_t off = 0;
    for (int64_t s = 0; s < N; ++s) {
        int64_t L = lengths[s] > 0 ? lengths[s] : 0;
        const int32_t *tok = tokens + off;
        for (int64_t t = 0; t < L; ++t) {
            int g = 0;
            if (t >= ctx_width) {
                uint32_t v = (uint32_t)tok[t];
                g = sbw_oracle_green(seed_for(scheme, key, tok + (t - ctx_width), ctx_width, v), v, thr);
            }
            green[off + t] = (uint8_t)g;
        }
        off += L;
    }
}

void sbw_oracle_window_z(const uint8_t *green, const int32_t *lengths, int64_t N, int ctx_width,
                         int64_t window, double gamma, int32_t *best_count, int32_t *best_start,
                         double *best_z)
{
    int64_t off = 0;
    for (int64_t s = 0; s < N; ++s) {
        int64_t L = lengths[s] > 0 ? lengths[s] : 0;
        int64_t T = L > ctx_width ? L - ctx_width : 0;
        const uint8_t *y = green + off + (L > ctx_width ? ctx_width : L);   /* scored positions */
        int64_t w = window < T ? window : T;
        int64_t bc = 0, bs = 0;
        for (int64_t start = 0; start + w <= T && w > 0; ++start) {
            int64_t c = 0;
            for (int64_t i = 0; i < w; ++i)
                c += y[start + i];
            if (c > bc) {               /* strict: ties keep the earliest start */
                bc = c;
                bs = start;
            }
        }
        best_count[s] = (int32_t)bc;
        best_start[s] = (int32_t)bs;
        best_z[s] = sbw_oracle_zscore(bc, w, gamma);
        off += L;
    }
}

/* Detection that scores every distinct (context, token) tuple of a sequence once -- the option
 * KGW-family detectors call "ignore repeated n-grams" (Section 3 takes the Y_t as independent;
 * repeated text repeats the same trial).  Position t >= W counts iff no earlier scored position
 * t' in [W, t) has tok[t'-W .. t'] equal to tok[t-W .. t] element by element; T is the number of
 * such positions, G the green ones among them; Eq. 5 on (G, T). */
void sbw_oracle_detect_unique(const int32_t *tokens, const int32_t *lengths, int64_t N, int ctx_width,
                              uint64_t key, double gamma, int scheme, int32_t *counts, int32_t *T,
                              double *z, int threads)
{
    uint64_t thr = sbw_oracle_threshold(gamma);
    int64_t *offsets = (int64_t *)malloc((size_t)(N + 1) * sizeof(int64_t));
    if (!offsets)
        return;
    offsets[0] = 0;
    for (int64_t s = 0; s < N; ++s)
        offsets[s + 1] = offsets[s] + (lengths[s] > 0 ? lengths[s] : 0);
    if (threads < 1)
        threads = 1;
#pragma omp parallel for num_threads(threads) schedule(dynamic, 16)
    for (int64_t s = 0; s < N; ++s) {
        const int32_t *tok = tokens + offsets[s];
        int64_t L = lengths[s] > 0 ? lengths[s] : 0;
        int64_t G = 0, Tu = 0;
        for (int64_t t = ctx_width; t < L; ++t) {
            int seen = 0;
            for (int64_t e = ctx_width; e < t && !seen; ++e) {
                int same = 1;
                for (int i = 0; i <= ctx_width; ++i)
                    if (tok[e - i] != tok[t - i])
                        same = 0;
                seen = same;
            }
            if (seen)
                continue;
            uint32_t v = (uint32_t)tok[t];
            uint64_t r = seed_for(scheme, key, tok + (t - ctx_width), ctx_width, v);
            G += sbw_oracle_green(r, v, thr);
            Tu += 1;
        }
        counts[s] = (int32_t)G;
        if (T)
            T[s] = (int32_t)Tu;
        z[s] = sbw_oracle_zscore(G, Tu, gamma);
    }
    free(offsets);
}

/* Detection on a truncated copy of each sequence (the truncation attacks of Appendix G keep a
 * prefix of the text): only the first keep[s] tokens of sequence s count, keep clamped to
 * [0, length].  green is the per-token array sbw_oracle_detect_bits wrote for the whole text. */
void sbw_oracle_prefix_z(const uint8_t *green, const int32_t *lengths, const int32_t *keep, int64_t N,
                         int ctx_width, double gamma, int32_t *counts, int32_t *T, double *z)
{
    int64_t off = 0;
    for (int64_t s = 0; s < N; ++s) {
        int64_t L = lengths[s] > 0 ? lengths[s] : 0;
        int64_t K = keep[s] < 0 ? 0 : (keep[s] > L ? L : keep[s]);
        int64_t G = 0;
        for (int64_t t = ctx_width; t < K; ++t)
            G += green[off + t];
        int64_t Tk = K > ctx_width ? K - ctx_width : 0;
        counts[s] = (int32_t)G;
        if (T)
            T[s] = (int32_t)Tk;
        z[s] = sbw_oracle_zscore(G, Tk, gamma);
        off += L;
    }
}

/* Section 4.3: area under the ROC curve of the z-score as a detector of label 1 against label 0,
 * written as the probability that a watermarked text outscores an unmarked one, ties counting a
 * half (equal to the trapezoid area under the curve swept over all thresholds).  NaN scores are
 * left out of both classes.  stats (nullable) receives {pairs with z_pos > z_neg, pairs with
 * z_pos == z_neg, n_pos, n_neg}.  Returns NaN when a class is empty. */
double sbw_oracle_roc_auc(const double *z, const uint8_t *labels, int64_t n, uint64_t stats[4], int threads)
{
    uint64_t greater = 0, equal = 0, npos = 0, nneg = 0;
    for (int64_t i = 0; i < n; ++i) {
        if (z[i] != z[i])
            continue;
        if (labels[i])
            npos += 1;
        else
            nneg += 1;
    }
    if (threads < 1)
        threads = 1;
#pragma omp parallel for num_threads(threads) reduction(+ : greater, equal) schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        if (!labels[i] || z[i] != z[i])
            continue;
        for (int64_t j = 0; j < n; ++j) {
            if (labels[j] || z[j] != z[j])
                continue;
            if (z[i] > z[j])
                greater += 1;
            else if (z[i] == z[j])
                equal += 1;
        }
    }
    if (stats) {
        stats[0] = greater;
        stats[1] = equal;
        stats[2] = npos;
        stats[3] = nneg;
    }
    if (npos == 0 || nneg == 0)
        return NAN;
    /* (2 greater + equal) / (2 npos nneg): numerator and denominator are exact integers */
    return (double)(2 * greater + equal) / (double)(2 * npos * nneg);
}

/* ------------------------------------------------------------------ R8: sampler ---- */
/*
 * Specified fp32 natural logarithm for positive normal x (every step one IEEE operation):
 *   ix = bits(x); e = (int32)(ix - 0x3f3504f3) >> 23 (arithmetic shift);
 *   m = float with bits ix - (e << 23), so m lies in [sqrt(1/2), sqrt(2)); f = m - 1 (exact);
 *   r = Horner in f of C6..C0 with fmaf; q = fmaf(r, f, -0.5); t = fmaf(f*f, q, f);
 *   result = fmaf(e, LN2_HI, fmaf(e, LN2_LO, t)).
 * Coefficients (own least-maximum fit of (log1p(f) - f + f^2/2)/f^3 on the interval, rounded
 * to fp32): C0..C6 = 0x1.5556d8p-2, -0x1.000382p-2, 0x1.98d7fp-3, -0x1.53824cp-3,
 * 0x1.31747p-3, -0x1.2432aap-3, 0x1.645de2p-4; LN2_HI = 0x1.62e43p-1, LN2_LO = -0x1.05c61p-29.
 */
float sbw_oracle_log(float x)
{
    static const float C[7] = { 0x1.5556d8p-2f, -0x1.000382p-2f, 0x1.98d7fp-3f, -0x1.53824cp-3f,
                                0x1.31747p-3f, -0x1.2432aap-3f, 0x1.645de2p-4f };
    const float LN2_HI = 0x1.62e43p-1f, LN2_LO = -0x1.05c61p-29f;
    uint32_t ix;
    memcpy(&ix, &x, sizeof ix);
    uint32_t shifted = ix - 0x3f3504f3u;
    int32_t e = (int32_t)shifted >> 23;              /* gcc: arithmetic shift of a signed value */
    uint32_t im = ix - ((uint32_t)e << 23);
    float m;
    memcpy(&m, &im, sizeof m);
    float f = m - 1.0f;
    float r = C[6];
    for (int i = 5; i >= 0; --i)
        r = fmaf(r, f, C[i]);
    float q = fmaf(r, f, -0.5f);
    float f2 = f * f;
    float t = fmaf(f2, q, f);
    float fe = (float)e;
    return fmaf(fe, LN2_HI, fmaf(fe, LN2_LO, t));
}

/* Uniform in (0,1) for (row, candidate): Philox block (v>>2, row, lo step, hi step) under the
 * key (lo rng_seed, hi rng_seed), word v&3; top 23 bits, centred: u = (y>>9 + 1/2) 2^-23. */
float sbw_oracle_gumbel_uniform(uint64_t rng_seed, uint64_t rng_step, uint32_t row, uint32_t v_global)
{
    uint32_t ctr[4] = { v_global >> 2, row, (uint32_t)rng_step, (uint32_t)(rng_step >> 32) };
    uint32_t key[2] = { (uint32_t)rng_seed, (uint32_t)(rng_seed >> 32) };
    uint32_t out[4];
    sbw_oracle_philox4x32_10(ctr, key, out);
    uint32_t y = out[v_global & 3u];
    return ((float)(y >> 9) + 0.5f) * 0x1p-23f;
}

/* Standard Gumbel variate g = -log(-log(u)) with the specified logarithm. */
float sbw_oracle_gumbel(uint64_t rng_seed, uint64_t rng_step, uint32_t row, uint32_t v_global)
{
    float u = sbw_oracle_gumbel_uniform(rng_seed, rng_step, row, v_global);
    float w = -sbw_oracle_log(u);
    return -sbw_oracle_log(w);
}

static void sample_row(const void *logits, int dtype, int64_t b, int64_t V, int64_t ld,
                       int64_t vocab_offset, const int32_t *ctx, int W, uint64_t key, uint64_t thr,
                       float delta, int scheme, float temperature, uint64_t rng_seed,
                       uint64_t rng_step, int32_t *out_tokens, double *out_max, double *out_sumexp,
                       double *out_prob, double *out_probs, float *out_score)
{
    float inv_tau = 1.0f / temperature;
    double tau = (double)temperature;
    float *biased = (float *)malloc((size_t)V * sizeof(float));
    if (!biased)
        return;
    /* l' of Eq. 2, in the logits' own precision, widened exactly to fp32 */
    for (int64_t j = 0; j < V; ++j) {
        uint32_t v = (uint32_t)(vocab_offset + j);
        uint64_t r = seed_for(scheme, key, ctx, W, v);
        int g = sbw_oracle_green(r, v, thr);
        if (dtype == SBW_O_DTYPE_BF16) {
            uint16_t h = ((const uint16_t *)logits)[b * ld + j];
            biased[j] = sbw_oracle_bf16_to_f32(sbw_oracle_bias_elem_bf16(h, delta, g));
        } else {
            biased[j] = sbw_oracle_bias_elem_f32(((const float *)logits)[b * ld + j], delta, g);
        }
    }
    /* m = max l' */
    double m = -INFINITY;
    for (int64_t j = 0; j < V; ++j)
        if ((double)biased[j] > m)
            m = (double)biased[j];
    /* Z = sum exp((l' - m)/tau) in fp64 */
    double Z = 0.0;
    for (int64_t j = 0; j < V; ++j)
        Z += exp(((double)biased[j] - m) / tau);
    /* Gumbel-max: id = argmax_v fmaf(l'_v, 1/tau, g_v), ties to the lowest v */
    int64_t best = 0;
    float best_s = -INFINITY;
    for (int64_t j = 0; j < V; ++j) {
        uint32_t v = (uint32_t)(vocab_offset + j);
        float g = sbw_oracle_gumbel(rng_seed, rng_step, (uint32_t)b, v);
        float s = fmaf(biased[j], inv_tau, g);
        if (s > best_s) {
            best_s = s;
            best = j;
        }
    }
    out_tokens[b] = (int32_t)best;
    if (out_max)
        out_max[b] = m;
    if (out_sumexp)
        out_sumexp[b] = Z;
    if (out_prob)
        out_prob[b] = exp(((double)biased[best] - m) / tau) / Z;
    if (out_score)
        out_score[b] = best_s;
    if (out_probs)
        for (int64_t j = 0; j < V; ++j)
            out_probs[b * V + j] = exp(((double)biased[j] - m) / tau) / Z;
    free(biased);
}

void sbw_oracle_bias_sample(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                            int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width,
                            uint64_t key, double gamma, float delta, int scheme,
                            float temperature, uint64_t rng_seed, uint64_t rng_step,
                            int32_t *out_tokens, double *out_max, double *out_sumexp,
                            double *out_prob, double *out_probs, float *out_score, int threads)
{
    uint64_t thr = sbw_oracle_threshold(gamma);
    if (threads < 1)
        threads = 1;
#pragma omp parallel for num_threads(threads) schedule(static)
    for (int64_t b = 0; b < B; ++b)
        sample_row(logits, dtype, b, V, ld, vocab_offset, ctx_tokens + b * ctx_width, ctx_width,
                   key, thr, delta, scheme, temperature, rng_seed, rng_step, out_tokens, out_max,
                   out_sumexp, out_prob, out_probs, out_score);
}

/* ------------------------------------------------------------------ R10: top-k / top-p ---- */
/*
 * Sampling from the truncated distribution (Appendix F of the paper samples with top_p = 0.8;
 * the paper gives no arithmetic for it, this library fixes one so that the kept set is a pure
 * function of the biased logits).  Per row, with l' the biased logits of Eq. 2:
 *   order    candidates sorted by order-encoded bits descending, ties by column ascending (the
 *            order of the top-k restriction above); m = the first one's value.
 *   top-k    top_k > 0 keeps the first min(top_k, V) of that order; top_k = 0 keeps all.
 *   weights  integers, so that sums do not depend on the order of addition:
 *            c = (float)(log2(e) / (double)temperature);
 *            a candidate with the bits of m has W = 2^40; otherwise d = l' - m, y = d * c (fp32);
 *            W = 0 unless y >= -41; n = rintf(y), f = y - n (exact), p = degree-7 Horner in f
 *            with fmaf over the coefficients (ln 2)^k / k! rounded to fp32, W = trunc(p 2^(n+40)).
 *   top-p    top_p < 1: with Z the sum of W over the candidates top-k kept, p32 = floor(top_p
 *            2^32) clamped to [1, 2^32], candidate number i of the order stays iff the weights of
 *            the candidates before it sum to S with S 2^32 < p32 Z (the candidate that crosses
 *            top_p stays, as in the usual nucleus rule; the first always stays).
 *   sample   Gumbel-max over the kept candidates with the stream of sbw_oracle_gumbel:
 *            argmax fmaf(l', 1/temperature, g), ties to the lowest column.
 */
uint64_t sbw_oracle_nucleus_weight(float l, float m, int is_max, float c)
{
    static const float K[8] = { 0x1p+0f, 0x1.62e43p-1f, 0x1.ebfbep-3f, 0x1.c6b08ep-5f,
                                0x1.3b2ab6p-7f, 0x1.5d87fep-10f, 0x1.430912p-13f, 0x1.ffcbfcp-17f };
    if (is_max)
        return (uint64_t)1 << 40;
    float d = l - m;
    float y = d * c;
    if (!(y >= -41.0f))
        return 0;                                    /* also NaN and -inf */
    if (y > 0.0f)
        y = 0.0f;                                    /* cannot happen for ordered finite values */
    float n = rintf(y);
    float f = y - n;
    float p = K[7];
    for (int i = 6; i >= 0; --i)
        p = fmaf(p, f, K[i]);
    float scaled = ldexpf(p, (int)n + 40);
    return (uint64_t)scaled;
}

void sbw_oracle_bias_sample_filtered(const void *logits, int dtype, int64_t B, int64_t V, int64_t ld,
                                     int64_t vocab_offset, const int32_t *ctx_tokens, int ctx_width,
                                     uint64_t key, double gamma, float delta, int scheme,
                                     float temperature, int64_t top_k, double top_p, uint64_t rng_seed,
                                     uint64_t rng_step, int32_t *out_tokens, int32_t *out_kept,
                                     uint8_t *out_mask, int threads)
{
    uint64_t thr = sbw_oracle_threshold(gamma);
    float inv_tau = 1.0f / temperature;
    float c = (float)(1.4426950408889634 / (double)temperature);
    double p_scaled = floor(top_p * 4294967296.0);
    uint64_t p32 = p_scaled < 1.0 ? 1u : (p_scaled > 4294967296.0 ? (uint64_t)1 << 32 : (uint64_t)p_scaled);
    if (threads < 1)
        threads = 1;
#pragma omp parallel for num_threads(threads) schedule(dynamic, 1)
    for (int64_t b = 0; b < B; ++b) {
        const int32_t *ctx = ctx_tokens + b * ctx_width;
        float *biased = (float *)malloc((size_t)V * sizeof(float));
        ranked_t *order = (ranked_t *)malloc((size_t)V * sizeof(ranked_t));
        if (!biased || !order) {
            free(biased);
            free(order);
            continue;
        }
        for (int64_t j = 0; j < V; ++j) {
            uint32_t v = (uint32_t)(vocab_offset + j);
            int g = sbw_oracle_green(seed_for(scheme, key, ctx, ctx_width, v), v, thr);
            uint32_t bits;
            if (dtype == SBW_O_DTYPE_BF16) {
                uint16_t h = sbw_oracle_bias_elem_bf16(((const uint16_t *)logits)[b * ld + j], delta, g);
                biased[j] = sbw_oracle_bf16_to_f32(h);
            } else {
                biased[j] = sbw_oracle_bias_elem_f32(((const float *)logits)[b * ld + j], delta, g);
            }
            memcpy(&bits, &biased[j], sizeof bits);
            order[j].code = order_code(bits);
            order[j].col = j;
        }
        qsort(order, (size_t)V, sizeof(ranked_t), ranked_cmp);
        int64_t n1 = (top_k > 0 && top_k < V) ? top_k : V;          /* after top-k */
        int64_t n2 = n1;                                            /* after top-p */
        if (top_p < 1.0) {
            float m = biased[order[0].col];
            unsigned __int128 Z = 0;
            for (int64_t i = 0; i < n1; ++i)
                Z += sbw_oracle_nucleus_weight(biased[order[i].col], m, order[i].code == order[0].code, c);
            unsigned __int128 S = 0;
            n2 = 0;
            for (int64_t i = 0; i < n1; ++i) {
                if (!((S << 32) < (unsigned __int128)p32 * Z))
                    break;
                n2 = i + 1;
                S += sbw_oracle_nucleus_weight(biased[order[i].col], m, order[i].code == order[0].code, c);
            }
        }
        if (out_mask)
            memset(out_mask + b * V, 0, (size_t)V);
        int64_t best = -1;
        float best_s = -INFINITY;
        for (int64_t i = 0; i < n2; ++i) {
            int64_t j = order[i].col;
            if (out_mask)
                out_mask[b * V + j] = 1;
            float g = sbw_oracle_gumbel(rng_seed, rng_step, (uint32_t)b, (uint32_t)(vocab_offset + j));
            float sc = fmaf(biased[j], inv_tau, g);
            if (best < 0 || sc > best_s || (sc == best_s && j < best)) {
                best_s = sc;
                best = j;
            }
        }
        out_tokens[b] = (int32_t)best;
        if (out_kept)
            out_kept[b] = (int32_t)n2;
        free(biased);
        free(order);
    }
}

/* ------------------------------------------------------------------ exhaustive checks */
int64_t sbw_oracle_jenkins_collisions(void)
{
    const size_t words = (size_t)1 << 26;            /* 2^32 bits */
    uint64_t *bitmap = (uint64_t *)calloc(words, sizeof(uint64_t));
    if (!bitmap)
        return -1;
    int64_t collisions = 0;
    /* inputs are split over the available cores; the bitmap is shared through atomic ORs */
#pragma omp parallel for reduction(+ : collisions) schedule(static)
    for (int64_t i = 0; i < ((int64_t)1 << 32); ++i) {
        uint32_t h = sbw_oracle_jenkins((uint32_t)i);
        uint64_t bit = (uint64_t)1 << (h & 63u);
        uint64_t before = __atomic_fetch_or(&bitmap[h >> 6], bit, __ATOMIC_RELAXED);
        if (before & bit)
            ++collisions;
    }
    free(bitmap);
    return collisions;
}

static double ulps_off(float got, double ref)
{
    int ex;
    frexp(ref, &ex);
    double ulp = ldexp(1.0, ex - 24);
    return fabs((double)got - ref) / ulp;
}

double sbw_oracle_log_max_ulp(int which)
{
    double worst = 0.0;
    for (uint32_t k = 0; k < (1u << 23); ++k) {
        float u = ((float)k + 0.5f) * 0x1p-23f;
        float lu = sbw_oracle_log(u);
        double err;
        if (which == 0) {
            err = ulps_off(lu, log((double)u));
        } else {
            float w = -lu;
            if (!(w > 0.0f))
                return INFINITY;
            err = ulps_off(sbw_oracle_log(w), log((double)w));
        }
        if (err > worst)
            worst = err;
    }
    return worst;
}
