"""Vocabulary- and row-sharded fused sampling on one GPU: the shards are sampled one after the
other (nothing waits on anything), their summaries are combined, and the result must equal both
the unsharded call and the oracle on the whole rows."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_03844_b200 as sbw
from paper_2609_03844_b200 import inputs, sharded
from gpu_util import KEY, host_bits, require_gpu

pytestmark = pytest.mark.gpu
REL = 1e-6


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("scheme", [sbw.SCHEME_CONTEXT, sbw.SCHEME_SELFSALT])
@pytest.mark.parametrize("S", [2, 8])
def test_vocabulary_shards_combine_to_the_unsharded_sample(dtype, scheme, S):
    dev = require_gpu()
    B, V, tau = 12, 128256, 0.7
    x = inputs.logits_normal(B, V, 4.0, dtype, seed=1500, device=dev)
    ctx = inputs.uniform_tokens((B, 1), V, seed=1501, device=dev)
    ws = torch.empty(sbw.sbw_sample_workspace_bytes(B, V), dtype=torch.uint8, device=dev)
    summaries = torch.empty((S, B, 8), dtype=torch.float32, device=dev)
    local = torch.empty(B, dtype=torch.int32, device=dev)
    for r in range(S):
        lo, hi = sharded.shard_columns(V, r, S)
        part = x[:, lo:hi]                                   # a view: row stride stays V
        sbw.sbw_bias_sample_shard(part, ctx, KEY, 0.25, 2.0, scheme, tau, 0xC4, 7, summaries[r], local, ws,
                                  vocab_offset=lo)
    tok = torch.empty(B, dtype=torch.int32, device=dev)
    m = torch.empty(B, dtype=torch.float32, device=dev)
    Z = torch.empty(B, dtype=torch.float32, device=dev)
    p = torch.empty(B, dtype=torch.float32, device=dev)
    sbw.sbw_sample_combine(summaries, tau, tok, out_max=m, out_sumexp=Z, out_prob=p)
    ref_tok = torch.empty(B, dtype=torch.int32, device=dev)
    sbw.sbw_bias_sample(x, ctx, KEY, 0.25, 2.0, scheme, tau, 0xC4, 7, ref_tok, ws)
    torch.cuda.synchronize()
    want = oracle.bias_sample(host_bits(x), V, ctx.cpu().numpy(), KEY, 0.25, 2.0, scheme, tau, 0xC4, 7, threads=8)
    assert np.array_equal(tok.cpu().numpy(), want["tokens"])
    assert np.array_equal(ref_tok.cpu().numpy(), want["tokens"])
    assert np.array_equal(m.cpu().numpy().astype(np.float64), want["max"])
    assert np.max(np.abs(Z.cpu().numpy() / want["sumexp"] - 1)) <= REL
    assert np.max(np.abs(p.cpu().numpy() / want["prob"] - 1)) <= REL


def test_row_shards_draw_the_same_gumbels_as_the_whole_batch():
    dev = require_gpu()
    B, V = 10, 32000
    x = inputs.logits_normal(B, V, 4.0, torch.bfloat16, seed=1510, device=dev)
    ctx = inputs.uniform_tokens((B, 1), V, seed=1511, device=dev)
    ws = torch.empty(sbw.sbw_sample_workspace_bytes(B, V), dtype=torch.uint8, device=dev)
    whole = torch.empty(B, dtype=torch.int32, device=dev)
    sbw.sbw_bias_sample(x, ctx, KEY, 0.25, 2.0, 1, 0.7, 5, 6, whole, ws)
    parts = torch.empty(B, dtype=torch.int32, device=dev)
    summ = torch.empty((B, 8), dtype=torch.float32, device=dev)
    for lo, hi in ((0, 3), (3, 4), (4, 10)):
        sbw.sbw_bias_sample_shard(x[lo:hi], ctx[lo:hi], KEY, 0.25, 2.0, 1, 0.7, 5, 6, summ[lo:hi], parts[lo:hi], ws,
                                  vocab_offset=0, row_offset=lo)
    torch.cuda.synchronize()
    assert torch.equal(whole, parts)
    assert torch.equal(summ[:, 3].view(torch.int32), whole)          # global id = local id at offset 0


def test_single_rank_helper_and_all_masked_rows():
    dev = require_gpu()
    B, V = 4, 4096
    x = inputs.logits_normal(B, V, 4.0, torch.float32, seed=1520, device=dev)
    x[1, :] = float("-inf")
    ctx = inputs.uniform_tokens((B, 1), V, seed=1521, device=dev)
    ws = torch.empty(sbw.sbw_sample_workspace_bytes(B, V), dtype=torch.uint8, device=dev)
    tok, m, Z, p = sharded.sharded_bias_sample(x, ctx, KEY, 0.5, 1.0, 0, 0.7, 1, 2, 0, ws)
    torch.cuda.synchronize()
    want = oracle.bias_sample(host_bits(x), V, ctx.cpu().numpy(), KEY, 0.5, 1.0, 0, 0.7, 1, 2)
    assert np.array_equal(tok.cpu().numpy(), want["tokens"]) and tok[1].item() == 0


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("scheme", [sbw.SCHEME_CONTEXT, sbw.SCHEME_SELFSALT])
@pytest.mark.parametrize("S,B", [(2, 12), (8, 3), (4, 600)])
def test_ids_only_shards_give_the_same_ids(dtype, scheme, S, B):
    """Shards that are asked for the ids alone (no statistics in the summary) take the cheaper
    kernel; the combined ids are those of the unsharded call and of the oracle."""
    dev = require_gpu()
    V, tau = 50000, 0.7
    x = inputs.logits_normal(B, V, 4.0, dtype, seed=1600 + B, device=dev)
    ctx = inputs.uniform_tokens((B, 1), V, seed=1601, device=dev)
    ws = torch.empty(sbw.sbw_sample_workspace_bytes(B, V), dtype=torch.uint8, device=dev)
    summaries = torch.empty((S, B, 8), dtype=torch.float32, device=dev)
    local = torch.empty(B, dtype=torch.int32, device=dev)
    for r in range(S):
        lo, hi = sharded.shard_columns(V, r, S)
        sbw.sbw_bias_sample_shard(x[:, lo:hi], ctx, KEY, 0.25, 2.0, scheme, tau, 0xC4, 9, summaries[r], local, ws,
                                  vocab_offset=lo, ids_only=True)
    tok = torch.empty(B, dtype=torch.int32, device=dev)
    sbw.sbw_sample_combine(summaries, tau, tok)
    torch.cuda.synchronize()
    want = oracle.bias_sample(host_bits(x), V, ctx.cpu().numpy(), KEY, 0.25, 2.0, scheme, tau, 0xC4, 9, threads=8)
    assert np.array_equal(tok.cpu().numpy(), want["tokens"])
    s = summaries.cpu().numpy()
    assert np.isneginf(s[:, :, 0]).all() and (s[:, :, 1] == 0).all()       # no statistics in these summaries


def _leg_worker(rank: int, world: int, port: int, out_dir: str):
    import json
    import os
    import sys
    from pathlib import Path

    import torch.distributed as dist

    root = Path(__file__).resolve().parent.parent
    sys.path.insert(0, str(root))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK="0")
    torch.cuda.set_device(0)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import paper_2609_03844_b200 as lib
    from paper_2609_03844_b200 import inputs as inp

    out = bench.run_sharded_leg(lib, inp, torch.device("cuda", 0), rank, world)
    with open(os.path.join(out_dir, f"leg{rank}.json"), "w") as f:
        json.dump(out, f)
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.gpu
def test_benchmark_sharded_leg_with_two_ranks_on_one_gpu(tmp_path):
    """The N > 1 leg of bench.py end to end: two processes share the one GPU (their kernels never wait
    on each other), each samples its half of the vocabulary, the summaries are all-gathered (gloo
    here, NCCL on several GPUs) and combined; both must end with the ids of the unsplit call."""
    import json
    import socket

    import torch.multiprocessing as mp

    require_gpu()
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    world = 2
    mp.spawn(_leg_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        leg = json.loads((tmp_path / f"leg{r}.json").read_text())
        assert leg["shards"] == 2 and leg["ids_equal_on_every_rank"] and leg["ids_equal_unsplit_call"]
        assert leg["sumexp_max_rel_diff_to_unsplit_call"] <= 1e-6 and leg["ms_per_step"] > 0
