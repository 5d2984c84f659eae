"""B200-native Stateless Bernoulli Watermarking: logits bias, fused sampling, batch detection.

The work is done by ``libsbw.so`` (hand-written sm_100a kernels behind a C ABI declared in
``include/sbw.h``); this package is its thin ctypes binding plus the seeded input generators.
"""
from .binding import (DTYPE_BF16, DTYPE_F32, SCHEME_CONTEXT, SCHEME_SELFSALT, SbwError, lib,
                      library_path, sbw_bias_logits, sbw_bias_logits_host, sbw_bias_logits_topk,
                      sbw_bias_logits_host_staging_bytes, sbw_bias_sample, sbw_bias_sample_noalloc, sbw_bias_sample_shard, sbw_sample_combine,
                      sbw_detect, sbw_detect_bits, sbw_detect_bits_words, sbw_window_z,
                      sbw_prefix_z, sbw_detect_unique, sbw_detect_unique_workspace_bytes,
                      sbw_roc_auc, sbw_roc_auc_batched, sbw_roc_auc_workspace_bytes, sbw_bias_sample_filtered,
                      sbw_sample_filtered_workspace_bytes,
                      sbw_detect_workspace_bytes, sbw_int_probe, sbw_sample_workspace_bytes,
                      sbw_version)

__all__ = ["DTYPE_BF16", "DTYPE_F32", "SCHEME_CONTEXT", "SCHEME_SELFSALT", "SbwError", "lib",
           "library_path", "sbw_bias_logits", "sbw_bias_logits_host", "sbw_bias_logits_topk",
           "sbw_bias_logits_host_staging_bytes", "sbw_bias_sample", "sbw_bias_sample_noalloc", "sbw_bias_sample_shard", "sbw_sample_combine",
           "sbw_detect", "sbw_detect_bits", "sbw_detect_bits_words", "sbw_window_z",
           "sbw_prefix_z", "sbw_detect_unique", "sbw_detect_unique_workspace_bytes",
           "sbw_roc_auc", "sbw_roc_auc_batched", "sbw_roc_auc_workspace_bytes", "sbw_bias_sample_filtered",
           "sbw_sample_filtered_workspace_bytes",
           "sbw_detect_workspace_bytes", "sbw_int_probe", "sbw_sample_workspace_bytes", "sbw_version"]
