"""CPU oracle for Stateless Bernoulli Watermarking: loader and numpy-facing wrappers.

TEST INFRASTRUCTURE, NOT PRODUCT.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg import this package; it imports nothing from the CUDA library and the CUDA
library imports nothing from here.  The arithmetic lives in ``sbw_oracle.c`` (plain C, one
IEEE operation per written operation); this module only compiles it with gcc, loads it with
ctypes and marshals numpy arrays.  ``py_ref`` is a second, big-integer restatement of the
integer hashes used to pin the C code.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "sbw_oracle.c"
_HDR = _HERE / "sbw_oracle.h"
_LIB = _HERE / "libsbw_oracle.so"

SCHEME_CONTEXT = 0
SCHEME_SELFSALT = 1
DTYPE_F32 = 0
DTYPE_BF16 = 1

_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle next to its source if missing or older than the source."""
    newest = max(_SRC.stat().st_mtime, _HDR.stat().st_mtime)
    if force or not _LIB.exists() or _LIB.stat().st_mtime < newest:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-fPIC", "-shared", "-Wall", "-Wextra", "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(str(_LIB))
        c = ctypes
        i64, u64, u32, i32 = c.c_int64, c.c_uint64, c.c_uint32, c.c_int
        vp = c.c_void_p
        L.sbw_oracle_jenkins.restype = u32
        L.sbw_oracle_jenkins.argtypes = [u32]
        L.sbw_oracle_philox4x32_10.restype = None
        L.sbw_oracle_philox4x32_10.argtypes = [vp, vp, vp]
        L.sbw_oracle_seed_context.restype = u64
        L.sbw_oracle_seed_context.argtypes = [u64, vp, i32]
        L.sbw_oracle_seed_selfsalt.restype = u64
        L.sbw_oracle_seed_selfsalt.argtypes = [u64, vp, i32, u32]
        L.sbw_oracle_threshold.restype = u64
        L.sbw_oracle_threshold.argtypes = [c.c_double]
        L.sbw_oracle_green.restype = i32
        L.sbw_oracle_green.argtypes = [u64, u32, u64]
        L.sbw_oracle_green_mask.restype = None
        L.sbw_oracle_green_mask.argtypes = [vp, i64, i64, i64, vp, i32, u64, c.c_double, i32]
        L.sbw_oracle_f32_to_bf16.restype = c.c_uint16
        L.sbw_oracle_f32_to_bf16.argtypes = [c.c_float]
        L.sbw_oracle_bf16_to_f32.restype = c.c_float
        L.sbw_oracle_bf16_to_f32.argtypes = [c.c_uint16]
        L.sbw_oracle_bias_elem_f32.restype = c.c_float
        L.sbw_oracle_bias_elem_f32.argtypes = [c.c_float, c.c_float, i32]
        L.sbw_oracle_bias_elem_bf16.restype = c.c_uint16
        L.sbw_oracle_bias_elem_bf16.argtypes = [c.c_uint16, c.c_float, i32]
        L.sbw_oracle_bias_logits.restype = None
        L.sbw_oracle_bias_logits.argtypes = [vp, i32, i64, i64, i64, i64, vp, i32, u64, c.c_double,
                                             c.c_float, i32, i32]
        L.sbw_oracle_bias_logits_topk.restype = None
        L.sbw_oracle_bias_logits_topk.argtypes = [vp, i32, i64, i64, i64, i64, vp, i32, u64, c.c_double,
                                                  c.c_float, i32, i64, vp]
        L.sbw_oracle_detect.restype = None
        L.sbw_oracle_detect.argtypes = [vp, vp, i64, i32, u64, c.c_double, i32, vp, vp, vp, i32]
        L.sbw_oracle_detect_bits.restype = None
        L.sbw_oracle_detect_bits.argtypes = [vp, vp, i64, i32, u64, c.c_double, i32, vp]
        L.sbw_oracle_window_z.restype = None
        L.sbw_oracle_window_z.argtypes = [vp, vp, i64, i32, i64, c.c_double, vp, vp, vp]
        L.sbw_oracle_detect_unique.restype = None
        L.sbw_oracle_detect_unique.argtypes = [vp, vp, i64, i32, u64, c.c_double, i32, vp, vp, vp, i32]
        L.sbw_oracle_prefix_z.restype = None
        L.sbw_oracle_prefix_z.argtypes = [vp, vp, vp, i64, i32, c.c_double, vp, vp, vp]
        L.sbw_oracle_roc_auc.restype = c.c_double
        L.sbw_oracle_roc_auc.argtypes = [vp, vp, i64, vp, i32]
        L.sbw_oracle_zscore.restype = c.c_double
        L.sbw_oracle_zscore.argtypes = [i64, i64, c.c_double]
        L.sbw_oracle_log.restype = c.c_float
        L.sbw_oracle_log.argtypes = [c.c_float]
        L.sbw_oracle_gumbel_uniform.restype = c.c_float
        L.sbw_oracle_gumbel_uniform.argtypes = [u64, u64, u32, u32]
        L.sbw_oracle_gumbel.restype = c.c_float
        L.sbw_oracle_gumbel.argtypes = [u64, u64, u32, u32]
        L.sbw_oracle_bias_sample.restype = None
        L.sbw_oracle_bias_sample.argtypes = [vp, i32, i64, i64, i64, i64, vp, i32, u64, c.c_double,
                                             c.c_float, i32, c.c_float, u64, u64, vp, vp, vp, vp,
                                             vp, vp, i32]
        L.sbw_oracle_nucleus_weight.restype = u64
        L.sbw_oracle_nucleus_weight.argtypes = [c.c_float, c.c_float, i32, c.c_float]
        L.sbw_oracle_bias_sample_filtered.restype = None
        L.sbw_oracle_bias_sample_filtered.argtypes = [vp, i32, i64, i64, i64, i64, vp, i32, u64, c.c_double,
                                                      c.c_float, i32, c.c_float, i64, c.c_double, u64, u64,
                                                      vp, vp, vp, i32]
        L.sbw_oracle_jenkins_collisions.restype = i64
        L.sbw_oracle_jenkins_collisions.argtypes = []
        L.sbw_oracle_log_max_ulp.restype = c.c_double
        L.sbw_oracle_log_max_ulp.argtypes = [i32]
        _lib = L
    return _lib


def _ptr(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _ctx(ctx_tokens, B: int) -> tuple[np.ndarray, int]:
    ctx = np.ascontiguousarray(np.asarray(ctx_tokens, dtype=np.int32))
    if ctx.ndim == 1:
        ctx = ctx.reshape(B, -1)
    assert ctx.shape[0] == B
    return ctx, int(ctx.shape[1])


def jenkins(a: int) -> int:
    return int(lib().sbw_oracle_jenkins(a & 0xFFFFFFFF))


def philox(ctr, key) -> tuple[int, int, int, int]:
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().sbw_oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return tuple(int(x) for x in out)


def seed_context(key: int, ctx) -> int:
    c = np.asarray(ctx, dtype=np.int64).astype(np.uint32).view(np.int32).copy()
    return int(lib().sbw_oracle_seed_context(key, _ptr(c), len(c)))


def seed_selfsalt(key: int, ctx, v: int) -> int:
    c = np.asarray(ctx, dtype=np.int64).astype(np.uint32).view(np.int32).copy()
    return int(lib().sbw_oracle_seed_selfsalt(key, _ptr(c), len(c), v & 0xFFFFFFFF))


def threshold(gamma: float) -> int:
    return int(lib().sbw_oracle_threshold(gamma))


def green(r: int, v: int, thr: int) -> int:
    return int(lib().sbw_oracle_green(r, v & 0xFFFFFFFF, thr))


def green_mask(B, V, ctx_tokens, key, gamma, scheme, vocab_offset=0) -> np.ndarray:
    ctx, W = _ctx(ctx_tokens, B)
    mask = np.zeros((B, V), dtype=np.uint8)
    lib().sbw_oracle_green_mask(_ptr(mask), B, V, vocab_offset, _ptr(ctx), W, key, gamma, scheme)
    return mask


def bias_logits(logits: np.ndarray, V, ctx_tokens, key, gamma, delta, scheme,
                vocab_offset=0, threads=1) -> np.ndarray:
    """Eq. 2 on a copy of ``logits`` ([B, ld] float32, or uint16 holding bf16 bits)."""
    assert logits.ndim == 2 and logits.dtype in (np.float32, np.uint16)
    out = np.ascontiguousarray(logits).copy()
    B, ld = out.shape
    ctx, W = _ctx(ctx_tokens, B)
    dtype = DTYPE_F32 if out.dtype == np.float32 else DTYPE_BF16
    lib().sbw_oracle_bias_logits(_ptr(out), dtype, B, V, ld, vocab_offset, _ptr(ctx), W, key,
                                 gamma, delta, scheme, threads)
    return out


def bias_logits_topk(logits: np.ndarray, V, ctx_tokens, key, gamma, delta, scheme, top_k,
                     vocab_offset=0):
    """Top-k restricted bias (SBW-ss) on a copy of ``logits``; returns (biased, chosen columns)."""
    assert logits.ndim == 2 and logits.dtype in (np.float32, np.uint16)
    out = np.ascontiguousarray(logits).copy()
    B, ld = out.shape
    ctx, W = _ctx(ctx_tokens, B)
    dtype = DTYPE_F32 if out.dtype == np.float32 else DTYPE_BF16
    sel = np.zeros((B, min(top_k, V)), dtype=np.int32)
    lib().sbw_oracle_bias_logits_topk(_ptr(out), dtype, B, V, ld, vocab_offset, _ptr(ctx), W, key,
                                      gamma, delta, scheme, top_k, _ptr(sel))
    return out, sel


def detect(tokens, lengths, key, gamma, scheme, ctx_width=1, threads=1):
    tok = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
    lens = np.ascontiguousarray(np.asarray(lengths, dtype=np.int32))
    N = lens.shape[0]
    counts = np.zeros(N, dtype=np.int32)
    T = np.zeros(N, dtype=np.int32)
    z = np.zeros(N, dtype=np.float64)
    lib().sbw_oracle_detect(_ptr(tok), _ptr(lens), N, ctx_width, key, gamma, scheme, _ptr(counts),
                            _ptr(T), _ptr(z), threads)
    return counts, T, z


def detect_bits(tokens, lengths, key, gamma, scheme, ctx_width=1) -> np.ndarray:
    """Y_t for every token of the flat array (0 for the unscored first ctx_width tokens)."""
    tok = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
    lens = np.ascontiguousarray(np.asarray(lengths, dtype=np.int32))
    green = np.zeros(tok.shape[0], dtype=np.uint8)
    lib().sbw_oracle_detect_bits(_ptr(tok), _ptr(lens), lens.shape[0], ctx_width, key, gamma, scheme,
                                 _ptr(green))
    return green


def window_z(green, lengths, window, gamma, ctx_width=1):
    """Best window of ``window`` scored positions per sequence: (count, start, z)."""
    g = np.ascontiguousarray(np.asarray(green, dtype=np.uint8))
    lens = np.ascontiguousarray(np.asarray(lengths, dtype=np.int32))
    N = lens.shape[0]
    bc = np.zeros(N, dtype=np.int32)
    bs = np.zeros(N, dtype=np.int32)
    bz = np.zeros(N, dtype=np.float64)
    lib().sbw_oracle_window_z(_ptr(g), _ptr(lens), N, ctx_width, window, gamma, _ptr(bc), _ptr(bs), _ptr(bz))
    return bc, bs, bz


def detect_unique(tokens, lengths, key, gamma, scheme, ctx_width=1, threads=1):
    """Detection that scores each distinct (context, token) tuple once: (counts, T, z)."""
    tok = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
    lens = np.ascontiguousarray(np.asarray(lengths, dtype=np.int32))
    N = lens.shape[0]
    counts = np.zeros(N, dtype=np.int32)
    T = np.zeros(N, dtype=np.int32)
    z = np.zeros(N, dtype=np.float64)
    lib().sbw_oracle_detect_unique(_ptr(tok), _ptr(lens), N, ctx_width, key, gamma, scheme,
                                   _ptr(counts), _ptr(T), _ptr(z), threads)
    return counts, T, z


def prefix_z(green, lengths, keep, gamma, ctx_width=1):
    """Detection on the first ``keep[s]`` tokens of each sequence: (counts, T, z)."""
    g = np.ascontiguousarray(np.asarray(green, dtype=np.uint8))
    lens = np.ascontiguousarray(np.asarray(lengths, dtype=np.int32))
    kp = np.ascontiguousarray(np.asarray(keep, dtype=np.int32))
    N = lens.shape[0]
    counts = np.zeros(N, dtype=np.int32)
    T = np.zeros(N, dtype=np.int32)
    z = np.zeros(N, dtype=np.float64)
    lib().sbw_oracle_prefix_z(_ptr(g), _ptr(lens), _ptr(kp), N, ctx_width, gamma, _ptr(counts),
                              _ptr(T), _ptr(z))
    return counts, T, z


def roc_auc(z, labels, threads=1):
    """ROC-AUC of z against 0/1 labels and the pair statistics {greater, equal, n_pos, n_neg}."""
    zz = np.ascontiguousarray(np.asarray(z, dtype=np.float64))
    lb = np.ascontiguousarray(np.asarray(labels, dtype=np.uint8))
    assert zz.shape == lb.shape and zz.ndim == 1
    stats = np.zeros(4, dtype=np.uint64)
    auc = float(lib().sbw_oracle_roc_auc(_ptr(zz), _ptr(lb), zz.shape[0], _ptr(stats), threads))
    return auc, stats


def zscore(G: int, T: int, gamma: float) -> float:
    return float(lib().sbw_oracle_zscore(G, T, gamma))


def log32(x: float) -> float:
    return float(lib().sbw_oracle_log(x))


def gumbel_uniform(rng_seed, rng_step, row, v) -> float:
    return float(lib().sbw_oracle_gumbel_uniform(rng_seed, rng_step, row, v))


def gumbel(rng_seed, rng_step, row, v) -> float:
    return float(lib().sbw_oracle_gumbel(rng_seed, rng_step, row, v))


def bias_sample(logits: np.ndarray, V, ctx_tokens, key, gamma, delta, scheme, temperature,
                rng_seed, rng_step, vocab_offset=0, want_probs=False, threads=1):
    """Fused bias + softmax statistics + Gumbel-max id.  Returns a dict of numpy arrays."""
    assert logits.ndim == 2 and logits.dtype in (np.float32, np.uint16)
    x = np.ascontiguousarray(logits)
    B, ld = x.shape
    ctx, W = _ctx(ctx_tokens, B)
    dtype = DTYPE_F32 if x.dtype == np.float32 else DTYPE_BF16
    tokens = np.zeros(B, dtype=np.int32)
    m = np.zeros(B, dtype=np.float64)
    Z = np.zeros(B, dtype=np.float64)
    p = np.zeros(B, dtype=np.float64)
    score = np.zeros(B, dtype=np.float32)
    probs = np.zeros((B, V), dtype=np.float64) if want_probs else None
    lib().sbw_oracle_bias_sample(_ptr(x), dtype, B, V, ld, vocab_offset, _ptr(ctx), W, key, gamma,
                                 delta, scheme, temperature, rng_seed, rng_step, _ptr(tokens),
                                 _ptr(m), _ptr(Z), _ptr(p), _ptr(probs), _ptr(score), threads)
    return {"tokens": tokens, "max": m, "sumexp": Z, "prob": p, "probs": probs, "score": score}


def nucleus_weight(l: float, m: float, is_max: bool, c: float) -> int:
    return int(lib().sbw_oracle_nucleus_weight(l, m, int(is_max), c))


def bias_sample_filtered(logits: np.ndarray, V, ctx_tokens, key, gamma, delta, scheme, temperature,
                         top_k, top_p, rng_seed, rng_step, vocab_offset=0, want_mask=False, threads=1):
    """Fused bias + top-k / top-p truncation + Gumbel-max id: dict of tokens, kept counts, mask."""
    assert logits.ndim == 2 and logits.dtype in (np.float32, np.uint16)
    x = np.ascontiguousarray(logits)
    B, ld = x.shape
    ctx, W = _ctx(ctx_tokens, B)
    dtype = DTYPE_F32 if x.dtype == np.float32 else DTYPE_BF16
    tokens = np.zeros(B, dtype=np.int32)
    kept = np.zeros(B, dtype=np.int32)
    mask = np.zeros((B, V), dtype=np.uint8) if want_mask else None
    lib().sbw_oracle_bias_sample_filtered(_ptr(x), dtype, B, V, ld, vocab_offset, _ptr(ctx), W, key, gamma,
                                          delta, scheme, temperature, top_k, top_p, rng_seed, rng_step,
                                          _ptr(tokens), _ptr(kept), _ptr(mask), threads)
    return {"tokens": tokens, "kept": kept, "mask": mask}


def jenkins_collisions() -> int:
    return int(lib().sbw_oracle_jenkins_collisions())


def log_max_ulp(which: int) -> float:
    return float(lib().sbw_oracle_log_max_ulp(which))
