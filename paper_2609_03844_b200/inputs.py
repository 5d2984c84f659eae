"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds input generators only -- no hashing, no thresholds, no bias, no statistics --
so that the CUDA path, the CPU oracle, the tests and the benchmark can all draw the same bytes
without sharing any of the method's arithmetic.  Everything is a pure function of its seed.

Workload shapes (Appendix D of the paper benchmarks fresh random ``(B, 151936)`` logits; its
completions are at most 200 tokens long; its batch sweep runs from 1 to 512):

* logits: i.i.d. normal with a given standard deviation, float32 or bfloat16, optionally with
  a Zipf-shaped spike ``amp * k**-s`` (k = 1..n_ids) added on ``n_ids`` distinct random ids of
  each row, which mimics a confident language-model step;
* context tokens and null token streams: ids uniform in ``[0, V)``;
* sequence lengths: uniform integers in ``[lmin, lmax]``.
"""
from __future__ import annotations

import numpy as np
import torch


def _gen(seed: int, device: str | torch.device = "cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def logits_normal(B: int, V: int, std: float, dtype: torch.dtype, seed: int,
                  device: str | torch.device = "cpu", ld: int | None = None) -> torch.Tensor:
    """``std * randn(B, V)`` narrowed to ``dtype``; with ``ld > V`` the row stride is padded
    and the padding columns hold a recognisable constant (so tests can see they are untouched)."""
    ld = V if ld is None else ld
    x = torch.randn((B, V), generator=_gen(seed, device), device=device, dtype=torch.float32)
    x = (x * std).to(dtype)
    if ld == V:
        return x.contiguous()
    full = torch.full((B, ld), 7.0, dtype=dtype, device=device)
    full[:, :V] = x
    return full


def add_zipf_spike_(logits: torch.Tensor, V: int, seed: int, n_ids: int = 50, s: float = 1.1,
                    amp: float = 20.0) -> torch.Tensor:
    """In place: per row, ``n_ids`` distinct random columns get ``amp * k**-s``, k = 1..n_ids."""
    B = logits.shape[0]
    g = _gen(seed, logits.device)
    scores = torch.rand((B, V), generator=g, device=logits.device)
    ids = scores.topk(n_ids, dim=1).indices                      # distinct per row
    k = torch.arange(1, n_ids + 1, device=logits.device, dtype=torch.float32)
    spike = (amp * k.pow(-s)).to(logits.dtype).expand(B, n_ids)
    rows = torch.arange(B, device=logits.device).unsqueeze(1).expand(B, n_ids)
    logits[rows, ids] = logits[rows, ids] + spike
    return logits


def uniform_tokens(shape, V: int, seed: int, device: str | torch.device = "cpu") -> torch.Tensor:
    """int32 ids uniform in [0, V)."""
    return torch.randint(0, V, tuple(shape), generator=_gen(seed, device), device=device,
                         dtype=torch.int32)


def sequence_lengths(N: int, lmin: int, lmax: int, seed: int,
                     device: str | torch.device = "cpu") -> torch.Tensor:
    """int32 lengths uniform in [lmin, lmax] (both ends included)."""
    return torch.randint(lmin, lmax + 1, (N,), generator=_gen(seed, device), device=device,
                         dtype=torch.int32)


def null_token_streams(N: int, lmin: int, lmax: int, V: int, seed: int,
                       device: str | torch.device = "cpu") -> tuple[torch.Tensor, torch.Tensor]:
    """Flat concatenation of N sequences of uniform ids plus their lengths."""
    lengths = sequence_lengths(N, lmin, lmax, seed, device)
    total = int(lengths.sum().item())
    tokens = uniform_tokens((total,), V, seed + 1, device)
    return tokens, lengths


def bf16_bits(x: torch.Tensor) -> np.ndarray:
    """A bfloat16 tensor's raw bits as a uint16 numpy array (host copy)."""
    assert x.dtype == torch.bfloat16
    return x.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16).copy()


def as_oracle_array(x: torch.Tensor) -> np.ndarray:
    """Host numpy view the oracle accepts: float32 as is, bfloat16 as uint16 bit patterns."""
    if x.dtype == torch.bfloat16:
        return bf16_bits(x)
    return x.detach().cpu().contiguous().numpy().copy()
