"""Vocabulary-sharded fused sampling across ranks: each rank samples on its own columns, the
per-row summaries (32 bytes per row) are all-gathered, and every rank combines them.

The paper observes that each device can derive identical green lists from the shared key and
leaves the multi-device case unvalidated; this module is that case.  The only collective is one
all-gather of a ``[B, 8]`` float32 tensor (NCCL on GPUs; any torch.distributed backend works).
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import binding


def shard_columns(V: int, rank: int, world: int, align: int = 8) -> tuple[int, int]:
    """Columns [lo, hi) of a vocabulary of V ids owned by ``rank``: contiguous, balanced, and cut
    at multiples of ``align`` so that every shard's rows can stay 16-byte aligned."""
    units = (V + align - 1) // align
    base, rem = divmod(units, world)
    lo_u = rank * base + min(rank, rem)
    hi_u = lo_u + base + (1 if rank < rem else 0)
    return min(lo_u * align, V), min(hi_u * align, V)


def gather_summaries(local: torch.Tensor, group=None) -> torch.Tensor:
    """All-gather of the per-rank ``[B, 8]`` summaries into ``[world, B, 8]`` (rank-major)."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    if world == 1:
        return local.reshape(1, *local.shape).contiguous()
    if local.is_cuda and dist.get_backend(group) == "gloo":
        # gloo gathers host tensors only: stage the 32 bytes per row through the host
        host = local.detach().cpu().contiguous()
        parts = [torch.empty_like(host) for _ in range(world)]
        dist.all_gather(parts, host, group=group)
        return torch.stack(parts).to(local.device)
    out = torch.empty((world, *local.shape), dtype=local.dtype, device=local.device)
    dist.all_gather([out[r] for r in range(world)], local.contiguous(), group=group)
    return out


def sharded_bias_sample(logits_shard: torch.Tensor, ctx_tokens: torch.Tensor, key: int, gamma: float,
                        delta: float, scheme: int, temperature: float, rng_seed: int, rng_step: int,
                        vocab_offset: int, workspace: torch.Tensor, group=None, row_offset: int = 0,
                        ids_only: bool = False):
    """Samples one token per row from logits whose columns are spread over the ranks of ``group``.
    ``logits_shard`` holds this rank's columns, ``vocab_offset`` the global id of its column 0.
    Returns (global token ids [B] int32, m [B], Z [B], p [B]) -- identical on every rank; with
    ``ids_only`` the shards take the cheaper ids-only path and m, Z, p are returned as None."""
    B = logits_shard.shape[0]
    dev = logits_shard.device
    summary = torch.empty((B, 8), dtype=torch.float32, device=dev)
    local_ids = torch.empty(B, dtype=torch.int32, device=dev)
    binding.sbw_bias_sample_shard(logits_shard, ctx_tokens, key, gamma, delta, scheme, temperature, rng_seed,
                                  rng_step, summary, local_ids, workspace, vocab_offset=vocab_offset,
                                  row_offset=row_offset, ids_only=ids_only)
    shards = gather_summaries(summary, group)
    tokens = torch.empty(B, dtype=torch.int32, device=dev)
    if ids_only:
        binding.sbw_sample_combine(shards, temperature, tokens)
        return tokens, None, None, None
    m = torch.empty(B, dtype=torch.float32, device=dev)
    Z = torch.empty(B, dtype=torch.float32, device=dev)
    p = torch.empty(B, dtype=torch.float32, device=dev)
    binding.sbw_sample_combine(shards, temperature, tokens, out_max=m, out_sumexp=Z, out_prob=p)
    return tokens, m, Z, p


def same_on_every_rank(t: torch.Tensor, group=None) -> bool:
    """True iff the integer tensor ``t`` holds the same values on every rank of ``group`` (two
    all-reduces: element-wise minimum and maximum over the ranks must coincide)."""
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return True
    lo, hi = t.clone(), t.clone()
    dist.all_reduce(lo, op=dist.ReduceOp.MIN, group=group)
    dist.all_reduce(hi, op=dist.ReduceOp.MAX, group=group)
    return bool(torch.equal(lo, hi))


def shard_sequences(N: int, rank: int, world: int) -> tuple[int, int]:
    """Sequences [lo, hi) of a batch of N owned by ``rank``: contiguous and balanced.  Detection has
    no cross-sequence dependency, so this is all the sharding it needs."""
    base, rem = divmod(N, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def gather_ragged(local: torch.Tensor, group=None) -> torch.Tensor:
    """Concatenation, in rank order, of 1-D tensors whose lengths differ between ranks (two
    collectives: the lengths, then the padded payloads)."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    if world == 1:
        return local.contiguous()
    n = torch.tensor([local.numel()], dtype=torch.int64, device=local.device)
    sizes = [torch.zeros_like(n) for _ in range(world)]
    dist.all_gather(sizes, n, group=group)
    sizes = [int(s.item()) for s in sizes]
    width = max(sizes)
    padded = torch.zeros(width, dtype=local.dtype, device=local.device)
    padded[:local.numel()] = local
    parts = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded, group=group)
    return torch.cat([p[:s] for p, s in zip(parts, sizes)])


def sharded_roc_auc(z_local: torch.Tensor, labels_local: torch.Tensor, group=None) -> torch.Tensor:
    """ROC-AUC over the z-scores of all ranks (each rank detected its own sequences): 9 bytes per
    sequence are all-gathered, then every rank counts the pairs itself.  Returns float64[1]."""
    z = gather_ragged(z_local, group)
    labels = gather_ragged(labels_local, group)
    auc = torch.empty(1, dtype=torch.float64, device=z.device)
    ws = torch.empty(max(binding.sbw_roc_auc_workspace_bytes(z.numel()), 256), dtype=torch.uint8, device=z.device)
    binding.sbw_roc_auc(z, labels, auc, ws)
    return auc
