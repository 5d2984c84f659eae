"""ctypes binding of the SBW CUDA library: one Python function per C entry point, same names.

Argument marshalling only -- every step of the path runs in the library's kernels.  PyTorch is
used for device memory and streams.  There is no fallback: if ``libsbw.so`` is missing or fails
to load, importing the symbols raises.
"""
from __future__ import annotations

import atexit
import ctypes
from pathlib import Path

import torch

from . import build as _build

SBW_OK = 0
SBW_ERR_INVALID_ARG = -1
SBW_ERR_UNSUPPORTED = -2
SBW_ERR_WORKSPACE = -3
SBW_ERR_CUDA = -4
SBW_ERR_TOO_LARGE = -5
NOALLOC_MAX_ROWS = 4096
SCHEME_CONTEXT = 0
SCHEME_SELFSALT = 1
DTYPE_F32 = 0
DTYPE_BF16 = 1

EXPORTS = ("sbw_version", "sbw_last_cuda_error", "sbw_bias_logits",
           "sbw_bias_logits_host_staging_bytes", "sbw_bias_logits_host",
           "sbw_sample_workspace_bytes", "sbw_bias_sample", "sbw_detect_workspace_bytes",
           "sbw_detect", "sbw_int_probe", "sbw_bias_sample_noalloc", "sbw_bias_logits_topk",
           "sbw_bias_sample_shard", "sbw_sample_combine", "sbw_detect_bits_words", "sbw_detect_bits",
           "sbw_window_z", "sbw_prefix_z", "sbw_detect_unique_workspace_bytes", "sbw_detect_unique",
           "sbw_roc_auc_workspace_bytes", "sbw_roc_auc", "sbw_sample_filtered_workspace_bytes",
           "sbw_bias_sample_filtered", "sbw_roc_auc_batched", "sbw_bias_sample_shard_ids")

_lib = None


def _drain_at_exit() -> None:
    """Waits for queued GPU work before the interpreter starts tearing libraries down, so that no
    kernel of this library is in flight while the CUDA runtime it shares with torch unloads."""
    try:
        if torch.cuda.is_available() and torch.cuda.is_initialized():
            torch.cuda.synchronize()
    except Exception:
        pass


class SbwError(RuntimeError):
    def __init__(self, call: str, code: int, cuda_error: int = 0):
        names = {-1: "SBW_ERR_INVALID_ARG", -2: "SBW_ERR_UNSUPPORTED", -3: "SBW_ERR_WORKSPACE",
                 -4: "SBW_ERR_CUDA", -5: "SBW_ERR_TOO_LARGE"}
        msg = f"{call} returned {names.get(code, code)}"
        if code == SBW_ERR_CUDA:
            msg += f" (cudaError_t {cuda_error})"
        super().__init__(msg)
        self.code = code
        self.cuda_error = cuda_error


def library_path() -> Path:
    return _build.LIB


def lib() -> ctypes.CDLL:
    """Load libsbw.so (building it first if the sources are newer).  Raises if unavailable."""
    global _lib
    if _lib is None:
        if _build.is_stale():
            _build.build()
        L = ctypes.CDLL(str(_build.LIB))
        c = ctypes
        i64, u64, i32, vp, sz = c.c_int64, c.c_uint64, c.c_int, c.c_void_p, c.c_size_t
        L.sbw_version.restype = c.c_char_p
        L.sbw_version.argtypes = []
        L.sbw_last_cuda_error.restype = i32
        L.sbw_last_cuda_error.argtypes = []
        L.sbw_bias_logits.restype = i32
        L.sbw_bias_logits.argtypes = [vp, i32, i64, i64, i64, i64, vp, i32, u64, c.c_double,
                                      c.c_float, i32, vp]
        L.sbw_bias_logits_topk.restype = i32
        L.sbw_bias_logits_topk.argtypes = [vp, i32, i64, i64, i64, i64, vp, i32, u64, c.c_double,
                                           c.c_float, i32, i64, vp]
        L.sbw_bias_logits_host_staging_bytes.restype = sz
        L.sbw_bias_logits_host_staging_bytes.argtypes = [i32, i64, i64, i32]
        L.sbw_bias_logits_host.restype = i32
        L.sbw_bias_logits_host.argtypes = [vp, i32, i64, i64, i64, i64, vp, i32, u64, c.c_double,
                                           c.c_float, i32, vp, sz, vp]
        L.sbw_sample_workspace_bytes.restype = sz
        L.sbw_sample_workspace_bytes.argtypes = [i64, i64]
        L.sbw_bias_sample.restype = i32
        L.sbw_bias_sample.argtypes = [vp, i32, i64, i64, i64, i64, vp, i32, u64, c.c_double,
                                      c.c_float, i32, c.c_float, u64, u64, vp, vp, vp, vp, vp, vp,
                                      sz, vp]
        L.sbw_bias_sample_noalloc.restype = i32
        L.sbw_bias_sample_noalloc.argtypes = [vp, i32, i64, i64, i64, i64, vp, i32, u64, c.c_double,
                                              c.c_float, i32, c.c_float, u64, u64, vp, vp, vp, vp, vp,
                                              vp]
        L.sbw_bias_sample_shard.restype = i32
        L.sbw_bias_sample_shard.argtypes = [vp, i32, i64, i64, i64, i64, i64, vp, i32, u64, c.c_double,
                                            c.c_float, i32, c.c_float, u64, u64, vp, vp, vp, sz, vp]
        L.sbw_bias_sample_shard_ids.restype = i32
        L.sbw_bias_sample_shard_ids.argtypes = [vp, i32, i64, i64, i64, i64, i64, vp, i32, u64, c.c_double,
                                                c.c_float, i32, c.c_float, u64, u64, vp, vp, vp, sz, vp]
        L.sbw_sample_combine.restype = i32
        L.sbw_sample_combine.argtypes = [vp, i64, i64, c.c_float, vp, vp, vp, vp, vp]
        L.sbw_detect_workspace_bytes.restype = sz
        L.sbw_detect_workspace_bytes.argtypes = [i64]
        L.sbw_detect.restype = i32
        L.sbw_detect.argtypes = [vp, vp, vp, i64, i64, i32, u64, c.c_double, i32, vp, vp, vp, vp,
                                 sz, vp]
        L.sbw_detect_bits_words.restype = sz
        L.sbw_detect_bits_words.argtypes = [i64, i64]
        L.sbw_detect_bits.restype = i32
        L.sbw_detect_bits.argtypes = [vp, vp, vp, i64, i64, i32, u64, c.c_double, i32, vp, vp, vp, vp, vp,
                                      sz, vp]
        L.sbw_window_z.restype = i32
        L.sbw_window_z.argtypes = [vp, vp, vp, i64, i64, i32, i64, c.c_double, vp, vp, vp, vp, vp]
        L.sbw_prefix_z.restype = i32
        L.sbw_prefix_z.argtypes = [vp, vp, vp, vp, i64, i64, i32, c.c_double, vp, vp, vp, vp]
        L.sbw_detect_unique_workspace_bytes.restype = sz
        L.sbw_detect_unique_workspace_bytes.argtypes = [i64, i64, i64]
        L.sbw_detect_unique.restype = i32
        L.sbw_detect_unique.argtypes = [vp, vp, vp, i64, i64, i64, i32, u64, c.c_double, i32, vp, vp, vp,
                                        vp, sz, vp]
        L.sbw_roc_auc_workspace_bytes.restype = sz
        L.sbw_roc_auc_workspace_bytes.argtypes = [i64]
        L.sbw_roc_auc.restype = i32
        L.sbw_roc_auc.argtypes = [vp, vp, i64, vp, vp, vp, sz, vp]
        L.sbw_roc_auc_batched.restype = i32
        L.sbw_roc_auc_batched.argtypes = [vp, vp, vp, i64, vp, vp, vp]
        L.sbw_sample_filtered_workspace_bytes.restype = sz
        L.sbw_sample_filtered_workspace_bytes.argtypes = [i32, i64, i64]
        L.sbw_bias_sample_filtered.restype = i32
        L.sbw_bias_sample_filtered.argtypes = [vp, i32, i64, i64, i64, i64, vp, i32, u64, c.c_double,
                                               c.c_float, i32, c.c_float, i64, c.c_double, u64, u64, vp, vp,
                                               vp, sz, vp]
        L.sbw_int_probe.restype = i32
        L.sbw_int_probe.argtypes = [i32, i32, i32, i32, vp, vp, vp]
        atexit.register(_drain_at_exit)
        _lib = L
    return _lib


def _check(call: str, rc: int) -> None:
    if rc != SBW_OK:
        raise SbwError(call, rc, lib().sbw_last_cuda_error() if rc == SBW_ERR_CUDA else 0)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return DTYPE_F32
    if t.dtype == torch.bfloat16:
        return DTYPE_BF16
    raise TypeError(f"logits must be float32 or bfloat16, got {t.dtype}")


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t: torch.Tensor | None) -> int | None:
    return None if t is None else t.data_ptr()


def _row_layout(logits: torch.Tensor, V: int | None):
    if logits.dim() != 2 or logits.stride(1) != 1:
        raise ValueError("logits must be 2-D with unit column stride")
    B, cols = logits.shape
    ld = logits.stride(0) if B > 1 else max(logits.stride(0), cols)
    return B, (cols if V is None else V), ld


def _ctx(ctx_tokens: torch.Tensor, B: int) -> int:
    if ctx_tokens.dtype != torch.int32 or not ctx_tokens.is_contiguous():
        raise TypeError("ctx_tokens must be a contiguous int32 tensor")
    if B == 0:
        return ctx_tokens.shape[-1] if ctx_tokens.dim() >= 2 and ctx_tokens.shape[-1] > 0 else 1
    if ctx_tokens.numel() % B != 0 or ctx_tokens.numel() == 0:
        raise ValueError("ctx_tokens must hold B * ctx_width ids")
    return ctx_tokens.numel() // B


def sbw_version() -> str:
    return lib().sbw_version().decode()


def sbw_bias_logits(logits: torch.Tensor, ctx_tokens: torch.Tensor, key: int, gamma: float,
                    delta: float, scheme: int, *, V: int | None = None, vocab_offset: int = 0,
                    stream=None) -> torch.Tensor:
    """In-place Eq. 1 + Eq. 2 on a CUDA ``[B, >=V]`` float32/bfloat16 tensor.  Returns ``logits``."""
    if not logits.is_cuda or not ctx_tokens.is_cuda:
        raise ValueError("sbw_bias_logits takes CUDA tensors (see sbw_bias_logits_host)")
    B, V, ld = _row_layout(logits, V)
    W = _ctx(ctx_tokens, B)
    rc = lib().sbw_bias_logits(_ptr(logits), _dtype_code(logits), B, V, ld, vocab_offset,
                               _ptr(ctx_tokens), W, key, gamma, delta, scheme, _stream(stream))
    _check("sbw_bias_logits", rc)
    return logits


def sbw_bias_logits_topk(logits: torch.Tensor, ctx_tokens: torch.Tensor, key: int, gamma: float,
                         delta: float, scheme: int, top_k: int = 40, *, V: int | None = None,
                         vocab_offset: int = 0, stream=None) -> torch.Tensor:
    """In-place bias of the ``top_k`` largest logits of every row only (the paper's SBW-ss)."""
    if not logits.is_cuda or not ctx_tokens.is_cuda:
        raise ValueError("sbw_bias_logits_topk takes CUDA tensors")
    B, V, ld = _row_layout(logits, V)
    W = _ctx(ctx_tokens, B)
    rc = lib().sbw_bias_logits_topk(_ptr(logits), _dtype_code(logits), B, V, ld, vocab_offset,
                                    _ptr(ctx_tokens), W, key, gamma, delta, scheme, top_k,
                                    _stream(stream))
    _check("sbw_bias_logits_topk", rc)
    return logits


def sbw_bias_logits_host_staging_bytes(dtype: torch.dtype, B: int, ld: int, ctx_width: int) -> int:
    code = DTYPE_F32 if dtype == torch.float32 else DTYPE_BF16
    return int(lib().sbw_bias_logits_host_staging_bytes(code, B, ld, ctx_width))


def sbw_bias_logits_host(logits_host: torch.Tensor, ctx_tokens_host: torch.Tensor, key: int,
                         gamma: float, delta: float, scheme: int, staging: torch.Tensor, *,
                         V: int | None = None, vocab_offset: int = 0, stream=None) -> torch.Tensor:
    """Same step for HOST tensors (ideally pinned): H2D, kernel, D2H, all enqueued on the stream.
    The caller synchronises the stream before reading ``logits_host``."""
    if logits_host.is_cuda or ctx_tokens_host.is_cuda or not staging.is_cuda:
        raise ValueError("host logits/ctx and a CUDA staging buffer are required")
    B, V, ld = _row_layout(logits_host, V)
    W = _ctx(ctx_tokens_host, B)
    rc = lib().sbw_bias_logits_host(_ptr(logits_host), _dtype_code(logits_host), B, V, ld,
                                    vocab_offset, _ptr(ctx_tokens_host), W, key, gamma, delta,
                                    scheme, _ptr(staging), staging.numel() * staging.element_size(),
                                    _stream(stream))
    _check("sbw_bias_logits_host", rc)
    return logits_host


def sbw_sample_workspace_bytes(B: int, V: int) -> int:
    return int(lib().sbw_sample_workspace_bytes(B, V))


def sbw_bias_sample(logits: torch.Tensor, ctx_tokens: torch.Tensor, key: int, gamma: float,
                    delta: float, scheme: int, temperature: float, rng_seed: int, rng_step: int,
                    out_tokens: torch.Tensor, workspace: torch.Tensor, *,
                    out_max: torch.Tensor | None = None, out_sumexp: torch.Tensor | None = None,
                    out_prob: torch.Tensor | None = None, out_probs: torch.Tensor | None = None,
                    V: int | None = None, vocab_offset: int = 0, stream=None) -> torch.Tensor:
    """Fused bias + softmax statistics + Gumbel-max id.  Outputs are caller-allocated CUDA
    tensors (int32 ids; float32 statistics).  Returns ``out_tokens``."""
    B, V, ld = _row_layout(logits, V)
    W = _ctx(ctx_tokens, B)
    for name, t, dt in (("out_tokens", out_tokens, torch.int32), ("out_max", out_max, torch.float32),
                        ("out_sumexp", out_sumexp, torch.float32),
                        ("out_prob", out_prob, torch.float32), ("out_probs", out_probs, torch.float32)):
        if t is not None and (t.dtype != dt or not t.is_cuda or not t.is_contiguous()):
            raise TypeError(f"{name} must be a contiguous CUDA {dt} tensor")
    rc = lib().sbw_bias_sample(_ptr(logits), _dtype_code(logits), B, V, ld, vocab_offset,
                               _ptr(ctx_tokens), W, key, gamma, delta, scheme, temperature,
                               rng_seed, rng_step, _ptr(out_tokens), _ptr(out_max),
                               _ptr(out_sumexp), _ptr(out_prob), _ptr(out_probs), _ptr(workspace),
                               workspace.numel() * workspace.element_size(), _stream(stream))
    _check("sbw_bias_sample", rc)
    return out_tokens


def sbw_sample_filtered_workspace_bytes(dtype: torch.dtype, B: int, V: int) -> int:
    code = DTYPE_F32 if dtype == torch.float32 else DTYPE_BF16
    return int(lib().sbw_sample_filtered_workspace_bytes(code, B, V))


def sbw_bias_sample_filtered(logits: torch.Tensor, ctx_tokens: torch.Tensor, key: int, gamma: float,
                             delta: float, scheme: int, temperature: float, top_k: int, top_p: float,
                             rng_seed: int, rng_step: int, out_tokens: torch.Tensor, workspace: torch.Tensor,
                             *, out_kept: torch.Tensor | None = None, V: int | None = None,
                             vocab_offset: int = 0, stream=None) -> torch.Tensor:
    """Fused bias + top-k / top-p truncation + Gumbel-max id (``top_k`` 0 and ``top_p`` >= 1 switch
    the filters off).  Returns ``out_tokens`` (int32 CUDA)."""
    B, V, ld = _row_layout(logits, V)
    W = _ctx(ctx_tokens, B)
    for name, t in (("out_tokens", out_tokens), ("out_kept", out_kept)):
        if t is not None and (t.dtype != torch.int32 or not t.is_cuda or not t.is_contiguous()):
            raise TypeError(f"{name} must be a contiguous CUDA int32 tensor")
    rc = lib().sbw_bias_sample_filtered(_ptr(logits), _dtype_code(logits), B, V, ld, vocab_offset,
                                        _ptr(ctx_tokens), W, key, gamma, delta, scheme, temperature, top_k,
                                        top_p, rng_seed, rng_step, _ptr(out_tokens), _ptr(out_kept),
                                        _ptr(workspace), workspace.numel() * workspace.element_size(),
                                        _stream(stream))
    _check("sbw_bias_sample_filtered", rc)
    return out_tokens


def sbw_bias_sample_noalloc(logits: torch.Tensor, ctx_tokens: torch.Tensor, key: int, gamma: float,
                            delta: float, scheme: int, temperature: float, rng_seed: int,
                            rng_step: int, out_tokens: torch.Tensor, *,
                            out_max: torch.Tensor | None = None,
                            out_sumexp: torch.Tensor | None = None,
                            out_prob: torch.Tensor | None = None,
                            out_probs: torch.Tensor | None = None, V: int | None = None,
                            vocab_offset: int = 0, stream=None) -> torch.Tensor:
    """sbw_bias_sample for callers that cannot allocate device memory (for instance a logits
    processor inside a serving engine whose cache pool already owns the GPU): no workspace
    argument, the scratch is a fixed 256 KiB array inside the library.  At most
    ``NOALLOC_MAX_ROWS`` rows per call; calls on one device share the scratch and must not
    overlap on the GPU; make the first call on a device outside stream capture."""
    B, V, ld = _row_layout(logits, V)
    W = _ctx(ctx_tokens, B)
    rc = lib().sbw_bias_sample_noalloc(_ptr(logits), _dtype_code(logits), B, V, ld, vocab_offset,
                                       _ptr(ctx_tokens), W, key, gamma, delta, scheme, temperature,
                                       rng_seed, rng_step, _ptr(out_tokens), _ptr(out_max),
                                       _ptr(out_sumexp), _ptr(out_prob), _ptr(out_probs),
                                       _stream(stream))
    _check("sbw_bias_sample_noalloc", rc)
    return out_tokens


def sbw_bias_sample_shard(logits: torch.Tensor, ctx_tokens: torch.Tensor, key: int, gamma: float,
                          delta: float, scheme: int, temperature: float, rng_seed: int, rng_step: int,
                          out_shard: torch.Tensor, out_tokens: torch.Tensor, workspace: torch.Tensor, *,
                          vocab_offset: int, row_offset: int = 0, V: int | None = None,
                          ids_only: bool = False, stream=None) -> torch.Tensor:
    """Fused sampling on one vocabulary shard; fills ``out_shard`` ([B, 8] float32) and returns it.
    ``ids_only`` calls sbw_bias_sample_shard_ids: the summary then serves the ids alone."""
    B, V, ld = _row_layout(logits, V)
    W = _ctx(ctx_tokens, B)
    if out_shard.dtype != torch.float32 or out_shard.numel() != B * 8 or not out_shard.is_contiguous():
        raise TypeError("out_shard must be a contiguous float32 tensor of B * 8 values")
    name = "sbw_bias_sample_shard_ids" if ids_only else "sbw_bias_sample_shard"
    rc = getattr(lib(), name)(_ptr(logits), _dtype_code(logits), B, V, ld, vocab_offset, row_offset,
                              _ptr(ctx_tokens), W, key, gamma, delta, scheme, temperature, rng_seed,
                              rng_step, _ptr(out_shard), _ptr(out_tokens), _ptr(workspace),
                              workspace.numel() * workspace.element_size(), _stream(stream))
    _check(name, rc)
    return out_shard


def sbw_sample_combine(shards: torch.Tensor, temperature: float, out_tokens: torch.Tensor, *,
                       out_max: torch.Tensor | None = None, out_sumexp: torch.Tensor | None = None,
                       out_prob: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """Merges per-shard summaries ``[S, B, 8]`` into global token ids (and optional statistics)."""
    if shards.dim() != 3 or shards.shape[2] != 8 or shards.dtype != torch.float32 or not shards.is_contiguous():
        raise TypeError("shards must be a contiguous float32 tensor of shape [S, B, 8]")
    S, B = shards.shape[0], shards.shape[1]
    rc = lib().sbw_sample_combine(_ptr(shards), S, B, temperature, _ptr(out_tokens), _ptr(out_max),
                                  _ptr(out_sumexp), _ptr(out_prob), _stream(stream))
    _check("sbw_sample_combine", rc)
    return out_tokens


def sbw_detect_workspace_bytes(N: int) -> int:
    return int(lib().sbw_detect_workspace_bytes(N))


def sbw_detect(tokens: torch.Tensor, lengths: torch.Tensor, key: int, gamma: float, scheme: int,
               out_counts: torch.Tensor, out_z: torch.Tensor, *, out_T: torch.Tensor | None = None,
               offsets: torch.Tensor | None = None, workspace: torch.Tensor | None = None,
               ctx_width: int = 1, stream=None):
    """Batch detection on a flat int32 token tensor + int32 lengths (CUDA).  Returns
    ``(out_counts, out_z)``."""
    N = lengths.numel()
    if tokens.dtype != torch.int32 or lengths.dtype != torch.int32:
        raise TypeError("tokens and lengths must be int32")
    if out_counts.dtype != torch.int32 or out_z.dtype != torch.float64:
        raise TypeError("out_counts must be int32 and out_z float64")
    if offsets is not None and (offsets.dtype != torch.int64 or offsets.numel() != N + 1):
        raise TypeError("offsets must be int64 with N + 1 entries")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().sbw_detect(_ptr(tokens), _ptr(lengths), _ptr(offsets), N, tokens.numel(), ctx_width,
                          key, gamma, scheme, _ptr(out_counts), _ptr(out_T), _ptr(out_z),
                          _ptr(workspace), ws_bytes, _stream(stream))
    _check("sbw_detect", rc)
    return out_counts, out_z


def sbw_detect_bits_words(N: int, total_tokens: int) -> int:
    return int(lib().sbw_detect_bits_words(N, total_tokens))


def sbw_detect_bits(tokens: torch.Tensor, lengths: torch.Tensor, key: int, gamma: float, scheme: int,
                    out_counts: torch.Tensor, out_z: torch.Tensor, out_bits: torch.Tensor, *,
                    out_T: torch.Tensor | None = None, offsets: torch.Tensor | None = None,
                    workspace: torch.Tensor | None = None, ctx_width: int = 1, stream=None):
    """sbw_detect that also stores the per-token green bits (int32/uint32 words, see sbw.h)."""
    N = lengths.numel()
    if out_bits.element_size() != 4 or out_bits.numel() < sbw_detect_bits_words(N, tokens.numel()):
        raise TypeError("out_bits must hold sbw_detect_bits_words(N, total) 32-bit words")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().sbw_detect_bits(_ptr(tokens), _ptr(lengths), _ptr(offsets), N, tokens.numel(), ctx_width, key,
                               gamma, scheme, _ptr(out_counts), _ptr(out_T), _ptr(out_z), _ptr(out_bits),
                               _ptr(workspace), ws_bytes, _stream(stream))
    _check("sbw_detect_bits", rc)
    return out_bits


def sbw_window_z(bits: torch.Tensor, lengths: torch.Tensor, offsets: torch.Tensor, total_tokens: int,
                 window: int, gamma: float, prefix_scratch: torch.Tensor, out_count: torch.Tensor,
                 out_start: torch.Tensor, out_z: torch.Tensor, *, ctx_width: int = 1, stream=None):
    """Best window of ``window`` scored positions per sequence from stored green bits."""
    N = lengths.numel()
    if offsets.dtype != torch.int64 or offsets.numel() < N + 1:
        raise TypeError("offsets must be int64 with N + 1 entries")
    rc = lib().sbw_window_z(_ptr(bits), _ptr(lengths), _ptr(offsets), N, total_tokens, ctx_width, window, gamma,
                            _ptr(prefix_scratch), _ptr(out_count), _ptr(out_start), _ptr(out_z),
                            _stream(stream))
    _check("sbw_window_z", rc)
    return out_count, out_start, out_z


def sbw_prefix_z(bits: torch.Tensor, lengths: torch.Tensor, offsets: torch.Tensor, keep: torch.Tensor,
                 total_tokens: int, gamma: float, out_counts: torch.Tensor, out_z: torch.Tensor, *,
                 out_T: torch.Tensor | None = None, ctx_width: int = 1, stream=None):
    """Detection on the first ``keep[s]`` tokens of each sequence, from stored green bits."""
    N = lengths.numel()
    if offsets.dtype != torch.int64 or offsets.numel() < N + 1:
        raise TypeError("offsets must be int64 with N + 1 entries")
    if keep.dtype != torch.int32 or keep.numel() != N:
        raise TypeError("keep must be int32 with N entries")
    rc = lib().sbw_prefix_z(_ptr(bits), _ptr(lengths), _ptr(offsets), _ptr(keep), N, total_tokens, ctx_width,
                            gamma, _ptr(out_counts), _ptr(out_T), _ptr(out_z), _stream(stream))
    _check("sbw_prefix_z", rc)
    return out_counts, out_z


def sbw_detect_unique_workspace_bytes(N: int, total_tokens: int, max_length: int) -> int:
    return int(lib().sbw_detect_unique_workspace_bytes(N, total_tokens, max_length))


def sbw_detect_unique(tokens: torch.Tensor, lengths: torch.Tensor, max_length: int, key: int, gamma: float,
                      scheme: int, out_counts: torch.Tensor, out_z: torch.Tensor, workspace: torch.Tensor, *,
                      out_T: torch.Tensor | None = None, offsets: torch.Tensor | None = None,
                      ctx_width: int = 1, stream=None):
    """Batch detection that scores each distinct (context, token) tuple of a sequence once."""
    N = lengths.numel()
    if tokens.dtype != torch.int32 or lengths.dtype != torch.int32:
        raise TypeError("tokens and lengths must be int32")
    if out_counts.dtype != torch.int32 or out_z.dtype != torch.float64:
        raise TypeError("out_counts must be int32 and out_z float64")
    if offsets is not None and (offsets.dtype != torch.int64 or offsets.numel() != N + 1):
        raise TypeError("offsets must be int64 with N + 1 entries")
    rc = lib().sbw_detect_unique(_ptr(tokens), _ptr(lengths), _ptr(offsets), N, tokens.numel(), max_length,
                                 ctx_width, key, gamma, scheme, _ptr(out_counts), _ptr(out_T), _ptr(out_z),
                                 _ptr(workspace), workspace.numel() * workspace.element_size(),
                                 _stream(stream))
    _check("sbw_detect_unique", rc)
    return out_counts, out_z


def sbw_roc_auc_workspace_bytes(n: int) -> int:
    return int(lib().sbw_roc_auc_workspace_bytes(n))


def sbw_roc_auc(z: torch.Tensor, labels: torch.Tensor, out_auc: torch.Tensor, workspace: torch.Tensor, *,
                out_stats: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """ROC-AUC of float64 scores against uint8 labels into ``out_auc`` (float64[1], CUDA)."""
    if z.dtype != torch.float64 or labels.dtype != torch.uint8 or z.numel() != labels.numel():
        raise TypeError("z must be float64 and labels uint8, of equal length")
    if out_auc.dtype != torch.float64 or (out_stats is not None and out_stats.dtype != torch.int64):
        raise TypeError("out_auc must be float64 and out_stats int64 (four 64-bit counters)")
    rc = lib().sbw_roc_auc(_ptr(z), _ptr(labels), z.numel(), _ptr(out_auc), _ptr(out_stats), _ptr(workspace),
                           workspace.numel() * workspace.element_size(), _stream(stream))
    _check("sbw_roc_auc", rc)
    return out_auc


def sbw_roc_auc_batched(z: torch.Tensor, labels: torch.Tensor, offsets: torch.Tensor, out_auc: torch.Tensor, *,
                        out_stats: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """One ROC-AUC per slice ``[offsets[i], offsets[i + 1])`` of the flat scores and labels."""
    M = offsets.numel() - 1
    if z.dtype != torch.float64 or labels.dtype != torch.uint8 or offsets.dtype != torch.int64:
        raise TypeError("z must be float64, labels uint8, offsets int64")
    if out_auc.dtype != torch.float64 or out_auc.numel() < M:
        raise TypeError("out_auc must be float64 with one entry per problem")
    if out_stats is not None and (out_stats.dtype != torch.int64 or out_stats.numel() < 4 * M):
        raise TypeError("out_stats must be int64 with four entries per problem")
    rc = lib().sbw_roc_auc_batched(_ptr(z), _ptr(labels), _ptr(offsets), M, _ptr(out_auc), _ptr(out_stats),
                                   _stream(stream))
    _check("sbw_roc_auc_batched", rc)
    return out_auc


PROBE_KINDS = {"mulwide": (0, 1), "lop3": (1, 1), "iadd3": (2, 1), "imad": (3, 1), "philox": (4, 4),
               "ffma": (5, 1), "mulhi": (6, 1), "mulwide_xor": (7, 2), "dual_fp": (8, 2), "dual_int": (9, 2),
               "add64": (10, 1)}


def sbw_int_probe(kind: str, steps: int = 4096, blocks_per_sm: int = 4, threads: int = 256,
                  stream=None) -> dict:
    """Runs the integer-throughput probe and returns thread-operations per clock per SM (from the
    SM cycle counter) and per second (from CUDA events), with the implied SM clock."""
    code, ops_per_step = PROBE_KINDS[kind]
    dev = torch.device("cuda", torch.cuda.current_device())
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    cycles = torch.zeros(sms * blocks_per_sm, dtype=torch.int64, device=dev)
    sink = torch.zeros(1, dtype=torch.int32, device=dev)
    s = _stream(stream)
    for _ in range(2):   # warm-up
        _check("sbw_int_probe", lib().sbw_int_probe(code, steps, blocks_per_sm, threads,
                                                    _ptr(cycles), _ptr(sink), s))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    _check("sbw_int_probe", lib().sbw_int_probe(code, steps, blocks_per_sm, threads, _ptr(cycles),
                                                _ptr(sink), s))
    e1.record()
    e1.synchronize()
    ms = e0.elapsed_time(e1)
    cyc = float(cycles.max().item())
    ops_sm = float(steps) * 8 * ops_per_step * threads * blocks_per_sm
    return {"kind": kind, "ops_per_clk_per_sm": ops_sm / cyc, "ops_per_s": ops_sm * sms / (ms * 1e-3),
            "sm_mhz_implied": cyc / (ms * 1e-3) / 1e6, "ms": ms, "sms": sms}
