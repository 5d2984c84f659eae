"""Large shapes through every entry point: a vocabulary of 2^21 ids at the top of the 32-bit id
range, one sequence of three million tokens.  The oracle computes every output here too."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_03844_b200 as sbw
from paper_2609_03844_b200 import inputs
from gpu_util import KEY, assert_same_bits, host_bits, require_gpu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_vocabulary_of_two_million_ids_at_the_top_of_the_id_range(dtype):
    dev = require_gpu()
    B, V = 2, 1 << 21
    off = (1 << 32) - V                                        # the last id is 2^32 - 1
    x = inputs.logits_normal(B, V, 3.0, dtype, seed=3)
    ctx = inputs.uniform_tokens((B, 4), 1 << 31, seed=4)
    xo, co = host_bits(x), ctx.numpy()
    args = (KEY, 0.25, 2.0, sbw.SCHEME_SELFSALT)

    xd = x.to(dev)
    sbw.sbw_bias_logits(xd, ctx.to(dev), *args, vocab_offset=off)
    torch.cuda.synchronize()
    assert_same_bits(host_bits(xd), oracle.bias_logits(xo, V, co, *args, vocab_offset=off, threads=8))

    xd = x.to(dev)
    sbw.sbw_bias_logits_topk(xd, ctx.to(dev), *args, 40, vocab_offset=off)
    torch.cuda.synchronize()
    assert_same_bits(host_bits(xd), oracle.bias_logits_topk(xo, V, co, *args, 40, vocab_offset=off)[0])

    ids = torch.empty(B, dtype=torch.int32, device=dev)
    ws = torch.empty(sbw.sbw_sample_workspace_bytes(B, V), dtype=torch.uint8, device=dev)
    sbw.sbw_bias_sample(x.to(dev), ctx.to(dev), *args, 0.7, 9, 1, ids, ws, vocab_offset=off)
    torch.cuda.synchronize()
    want = oracle.bias_sample(xo, V, co, *args, 0.7, 9, 1, vocab_offset=off, threads=2)
    assert np.array_equal(ids.cpu().numpy(), want["tokens"])

    kept = torch.empty(B, dtype=torch.int32, device=dev)
    wsf = torch.empty(sbw.sbw_sample_filtered_workspace_bytes(dtype, B, V), dtype=torch.uint8, device=dev)
    for top_k, top_p in ((0, 0.9), (3000, 0.999)):
        sbw.sbw_bias_sample_filtered(x.to(dev), ctx.to(dev), *args, 0.7, top_k, top_p, 9, 1, ids, wsf, out_kept=kept,
                                     vocab_offset=off)
        torch.cuda.synchronize()
        want = oracle.bias_sample_filtered(xo, V, co, *args, 0.7, top_k, top_p, 9, 1, vocab_offset=off, threads=2)
        assert np.array_equal(kept.cpu().numpy(), want["kept"]) and np.array_equal(ids.cpu().numpy(), want["tokens"])
    # one id more than the filter's histogram counters hold
    with pytest.raises(sbw.SbwError) as e:
        sbw.sbw_bias_sample_filtered(torch.zeros(1, V + 8, device=dev), ctx[:1].to(dev), *args, 0.7, 0, 0.9, 9, 1,
                                     ids[:1], torch.empty(1 << 24, dtype=torch.uint8, device=dev))
    assert e.value.code == -2


def test_one_sequence_of_three_million_tokens():
    dev = require_gpu()
    L, W = 3_000_000, 2
    rng = np.random.default_rng(8)
    tok = rng.integers(0, 1500, size=L + 50).astype(np.int32)          # repeats are common: 2.25 M possible tuples
    lens = np.array([L, 50], dtype=np.int32)
    t, l = torch.from_numpy(tok).to(dev), torch.from_numpy(lens).to(dev)
    N, total = 2, t.numel()
    counts = torch.empty(N, dtype=torch.int32, device=dev)
    T = torch.empty(N, dtype=torch.int32, device=dev)
    z = torch.empty(N, dtype=torch.float64, device=dev)
    bits = torch.zeros(sbw.sbw_detect_bits_words(N, total), dtype=torch.int32, device=dev)
    ws = torch.empty(sbw.sbw_detect_workspace_bytes(N), dtype=torch.uint8, device=dev)
    sbw.sbw_detect_bits(t, l, KEY, 0.25, sbw.SCHEME_SELFSALT, counts, z, bits, out_T=T, workspace=ws, ctx_width=W)
    offs = ws[:8 * (N + 1)].view(torch.int64)
    scratch = torch.empty_like(bits)
    bc, bs = torch.empty_like(counts), torch.empty_like(counts)
    bz = torch.empty_like(z)
    sbw.sbw_window_z(bits, l, offs, total, 100000, 0.25, scratch, bc, bs, bz, ctx_width=W)
    uc, uT, uz = torch.empty_like(counts), torch.empty_like(counts), torch.empty_like(z)
    uws = torch.empty(sbw.sbw_detect_unique_workspace_bytes(N, total, L), dtype=torch.uint8, device=dev)
    sbw.sbw_detect_unique(t, l, L, KEY, 0.25, sbw.SCHEME_SELFSALT, uc, uz, uws, out_T=uT, ctx_width=W)
    torch.cuda.synchronize()
    oc, oT, oz = oracle.detect(tok, lens, KEY, 0.25, 1, ctx_width=W)
    assert np.array_equal(counts.cpu().numpy(), oc) and np.array_equal(T.cpu().numpy(), oT)
    assert np.max(np.abs(z.cpu().numpy() - oz)) <= 1e-9
    green = oracle.detect_bits(tok, lens, KEY, 0.25, 1, ctx_width=W)
    # the quadratic window and distinct-tuple oracles are too slow at this length: restate both with
    # numpy on the oracle's own per-token bits (cumulative sums; np.unique over packed tuples)
    y = green[W:L].astype(np.int64)
    c = np.concatenate([[0], np.cumsum(y)])
    sums = c[100000:] - c[:-100000]
    assert int(bc.cpu()[0]) == int(sums.max()) and int(bs.cpu()[0]) == int(np.argmax(sums))
    assert abs(float(bz.cpu()[0]) - oracle.zscore(int(sums.max()), 100000, 0.25)) <= 1e-9
    packed = tok[:L].astype(np.int64)
    tup = packed[2:] * 1500 * 1500 + packed[1:-1] * 1500 + packed[:-2]
    _, first = np.unique(tup, return_index=True)
    assert int(uT.cpu()[0]) == len(first) and int(uc.cpu()[0]) == int(y[first].sum())
    assert abs(float(uz.cpu()[0]) - oracle.zscore(int(y[first].sum()), len(first), 0.25)) <= 1e-9
    ouc, ouT, _ = oracle.detect_unique(tok[L:], lens[1:], KEY, 0.25, 1, ctx_width=W)
    assert (int(uc.cpu()[1]), int(uT.cpu()[1])) == (int(ouc[0]), int(ouT[0]))
