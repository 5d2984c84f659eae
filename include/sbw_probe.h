/*
 * sbw_probe.h -- integer-throughput probe used to place the SBW kernels on a roofline.
 *
 * The paper has no counterpart for this call: it is measurement infrastructure.  The hot path of
 * Stateless Bernoulli Watermarking is a chain of 32x32->64 multiplies and three-input xors
 * (Philox4x32-10, Section 2.2), so its ceiling on a given GPU is the rate at which the SMs can
 * issue that mix.  The probe runs register-only loops of one instruction kind and reports how
 * many SM cycles they took.
 */
#ifndef SBW_PROBE_H
#define SBW_PROBE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SBW_PROBE_MULWIDE 0 /* mad.wide.u32 chains (32x32+64 -> 64)          1 op / step */
#define SBW_PROBE_LOP3 1    /* three-input xor chains                         1 op / step */
#define SBW_PROBE_IADD3 2   /* three-input add chains                         1 op / step */
#define SBW_PROBE_IMAD 3    /* 32-bit multiply-add chains                     1 op / step */
#define SBW_PROBE_PHILOX 4  /* Philox rounds: 2 wide multiplies + 2 xor3      4 ops / step */
#define SBW_PROBE_FFMA 5    /* fp32 fused multiply-add chains (for contrast)  1 op / step */
#define SBW_PROBE_MULHI 6       /* mul.hi.u32 chains (high half of a 32x32 product)        1 op / step */
#define SBW_PROBE_MULWIDE_XOR 7 /* mul.wide.u32, then lo ^ hi: 1 wide multiply + 1 xor     2 ops / step */
#define SBW_PROBE_DUAL_FP 8     /* one xor3 and one fp32 FMA: two pipes, issue-slot bound  2 ops / step */
#define SBW_PROBE_DUAL_INT 9    /* one xor3 and one 32-bit multiply-add: ALU + multiplier  2 ops / step */
#define SBW_PROBE_ADD64 10      /* 64-bit integer add chains                               1 op / step */
#define SBW_PROBE_KINDS 11

/*
 * Launches sm_count * blocks_per_sm blocks of `threads` threads; every thread runs `steps` steps
 * of 8 independent chains of the chosen kind.  out_cycles (device, int64[sm_count *
 * blocks_per_sm]) receives each block's elapsed SM clock cycles; out_sink (device, uint32[1])
 * receives a value that keeps the loops alive.  Work per thread = steps * 8 * (ops per step).
 * Returns SBW_OK or a negative SBW_ERR_* code (see sbw.h); enqueues on `stream`, no sync.
 */
int sbw_int_probe(int kind, int steps, int blocks_per_sm, int threads, int64_t *out_cycles,
                  uint32_t *out_sink, void *stream);

#ifdef __cplusplus
}
#endif
#endif
