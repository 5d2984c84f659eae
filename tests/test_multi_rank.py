"""The N > 1 host logic of bench.py on CPU: two gloo ranks shard a batch with no collective on
the data path, each scores its own sequences with the oracle, and the timing reduction takes the
maximum over ranks."""
import os
import socket
import sys
from pathlib import Path

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import oracle
    from paper_2609_03844_b200 import inputs

    assert bench.dist_env() == (rank, rank, world)
    # max over ranks of a per-rank time
    assert bench.max_over_ranks(10.0 + rank, world) == 10.0 + world - 1
    # shard 11 sequences over the ranks: every rank scores its own rows, no exchange needed
    tokens, lengths = inputs.null_token_streams(11, 5, 40, 32000, seed=3)
    lo, hi = bench.shard_rows(11, rank, world)
    off = np.concatenate([[0], np.cumsum(lengths.numpy())])
    c, T, z = oracle.detect(tokens.numpy()[off[lo]:off[hi]], lengths.numpy()[lo:hi], 0x5EED, 0.25, 0)
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), lo=lo, hi=hi, c=c, z=z)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_rows_and_reduce_time(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    import oracle
    from paper_2609_03844_b200 import inputs

    tokens, lengths = inputs.null_token_streams(11, 5, 40, 32000, seed=3)
    c_all, _, z_all = oracle.detect(tokens.numpy(), lengths.numpy(), 0x5EED, 0.25, 0)
    covered = []
    for r in range(world):
        d = np.load(tmp_path / f"rank{r}.npz")
        lo, hi = int(d["lo"]), int(d["hi"])
        covered += list(range(lo, hi))
        assert np.array_equal(d["c"], c_all[lo:hi]) and np.array_equal(d["z"], z_all[lo:hi])
    assert covered == list(range(11))          # a partition: every row exactly once


def test_shard_rows_is_a_balanced_partition():
    import bench

    for total in (0, 1, 7, 64, 100000):
        for world in (1, 2, 3, 8):
            parts = [bench.shard_rows(total, r, world) for r in range(world)]
            assert parts[0][0] == 0 and parts[-1][1] == total
            assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in parts]
            assert max(sizes) - min(sizes) <= 1


def _shard_worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2609_03844_b200 import inputs, sharded

    B, V, tau = 3, 4000, 0.7
    x = inputs.logits_normal(B, V, 4.0, torch.float32, seed=5)
    ctx = inputs.uniform_tokens((B, 1), V, seed=6).numpy()
    lo, hi = sharded.shard_columns(V, rank, world)
    part = np.ascontiguousarray(x.numpy()[:, lo:hi])
    # this rank's summary, from the oracle on its own columns only (global ids via vocab_offset)
    o = oracle.bias_sample(part, hi - lo, ctx, 0x5EED, 0.25, 2.0, 1, tau, 9, 4, vocab_offset=lo)
    biased = oracle.bias_logits(part, hi - lo, ctx, 0x5EED, 0.25, 2.0, 1, vocab_offset=lo)
    summ = np.zeros((B, 8), dtype=np.float32)
    summ[:, 0] = o["max"]
    summ[:, 1] = o["sumexp"]
    summ[:, 2] = o["score"]
    summ[:, 3] = (o["tokens"] + lo).astype(np.int32).view(np.float32)
    summ[:, 4] = biased[np.arange(B), o["tokens"]]
    # the agreement check the multi-GPU benchmark leg uses: equal ids pass, rank-dependent ones do not
    assert sharded.same_on_every_rank(torch.arange(5, dtype=torch.int32))
    assert not sharded.same_on_every_rank(torch.arange(5, dtype=torch.int32) + rank)
    gathered = sharded.gather_summaries(torch.from_numpy(summ))
    assert gathered.shape == (world, B, 8)
    assert torch.equal(gathered[rank], torch.from_numpy(summ))           # rank-major layout
    np.save(os.path.join(out_dir, f"gathered{rank}.npy"), gathered.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_exchange_shard_summaries(tmp_path):
    """Vocabulary-sharded sampling, host side: each rank summarises its own columns, one all-gather,
    and the combination rule (largest score, ties to the lowest global id; rescaled sums) gives
    what the oracle returns on the whole rows."""
    world = 2
    mp.spawn(_shard_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    import oracle
    from paper_2609_03844_b200 import inputs

    g0 = np.load(tmp_path / "gathered0.npy")
    g1 = np.load(tmp_path / "gathered1.npy")
    assert np.array_equal(g0.view(np.uint32), g1.view(np.uint32))         # every rank holds the same table
    B, V, tau = 3, 4000, 0.7
    x = inputs.logits_normal(B, V, 4.0, torch.float32, seed=5).numpy()
    ctx = inputs.uniform_tokens((B, 1), V, seed=6).numpy()
    want = oracle.bias_sample(x, V, ctx, 0x5EED, 0.25, 2.0, 1, tau, 9, 4)
    tau32 = float(np.float32(tau))
    for b in range(B):
        ids = g0[:, b, 3].view(np.int32)
        order = sorted(range(world), key=lambda r: (-g0[r, b, 2], ids[r]))
        assert ids[order[0]] == want["tokens"][b]
        m = g0[:, b, 0].max()
        Z = sum(float(g0[r, b, 1]) * np.exp((float(g0[r, b, 0]) - float(m)) / tau32) for r in range(world))
        assert m == want["max"][b] and abs(Z / want["sumexp"][b] - 1) < 1e-6


def test_shard_columns_partition_is_aligned_and_complete():
    from paper_2609_03844_b200 import sharded

    for V in (1, 7, 8, 128256, 151936, 32001):
        for world in (1, 2, 3, 8):
            parts = [sharded.shard_columns(V, r, world) for r in range(world)]
            assert parts[0][0] == 0 and parts[-1][1] == V
            assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))
            assert all(lo % 8 == 0 or lo == V for lo, _ in parts)


def _roc_worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2609_03844_b200 import inputs, sharded

    N = 13                                                      # odd: the ranks hold different numbers
    tokens, lengths = inputs.null_token_streams(N, 5, 60, 500, seed=11)
    lo, hi = sharded.shard_sequences(N, rank, world)
    off = np.concatenate([[0], np.cumsum(lengths.numpy())])
    _, _, z = oracle.detect(tokens.numpy()[off[lo]:off[hi]], lengths.numpy()[lo:hi], 0x5EED, 0.25, 1)
    labels = (np.arange(lo, hi) % 3 == 0).astype(np.uint8)
    all_z = sharded.gather_ragged(torch.from_numpy(z))
    all_l = sharded.gather_ragged(torch.from_numpy(labels))
    assert all_z.numel() == N and all_l.numel() == N
    np.savez(os.path.join(out_dir, f"roc{rank}.npz"), z=all_z.numpy(), l=all_l.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_gather_scores_for_roc_auc(tmp_path):
    """Sequence-sharded detection, host side: ranks hold different numbers of z-scores, the ragged
    all-gather restores the batch order on every rank, and the AUC of the gathered scores is the
    AUC of the unsharded batch."""
    world = 2
    mp.spawn(_roc_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    import oracle
    from paper_2609_03844_b200 import inputs, sharded

    r0, r1 = np.load(tmp_path / "roc0.npz"), np.load(tmp_path / "roc1.npz")
    assert np.array_equal(r0["z"], r1["z"]) and np.array_equal(r0["l"], r1["l"])
    tokens, lengths = inputs.null_token_streams(13, 5, 60, 500, seed=11)
    _, _, z = oracle.detect(tokens.numpy(), lengths.numpy(), 0x5EED, 0.25, 1)
    labels = (np.arange(13) % 3 == 0).astype(np.uint8)
    assert np.array_equal(r0["z"], z) and np.array_equal(r0["l"], labels)
    assert oracle.roc_auc(r0["z"], r0["l"])[0] == oracle.roc_auc(z, labels)[0]
    for N in (0, 1, 13, 100):
        for w in (1, 2, 3, 8):
            parts = [sharded.shard_sequences(N, r, w) for r in range(w)]
            assert parts[0][0] == 0 and parts[-1][1] == N
            assert all(a[1] == b[0] for a, b in zip(parts, parts[1:]))
            assert max(b - a for a, b in parts) - min(b - a for a, b in parts) <= 1
