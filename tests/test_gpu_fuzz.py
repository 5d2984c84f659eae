"""Seeded random configurations through every entry point, GPU against the oracle: shapes with
ragged tails and padded rows, vocabulary offsets, context widths 1..8, both schemes and dtypes,
random gamma / delta / temperature / filters.  Integer results bit-exact, z within 1e-9."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_03844_b200 as sbw
from paper_2609_03844_b200 import inputs
from gpu_util import assert_same_bits, host_bits, require_gpu

pytestmark = pytest.mark.gpu


def _config(seed):
    rng = np.random.default_rng(1000 + seed)
    V = int(rng.choice([1, 2, 7, 8, 9, 31, 257, 1000, 4097, 12345, 33000]))
    cfg = dict(
        B=int(rng.integers(1, 9)), V=V, pad=int(rng.choice([0, 0, 1, 3, 8, 40])),
        dtype=[torch.float32, torch.bfloat16][int(rng.integers(0, 2))],
        W=int(rng.integers(1, 9)), scheme=int(rng.integers(0, 2)),
        gamma=float(rng.choice([0.01, 0.25, 0.5, 0.73, 0.99])),
        delta=float(rng.choice([0.0, 0.5, 2.0, 4.0, -1.5])),
        tau=float(rng.choice([0.3, 0.7, 1.0, 1.7])),
        off=int(rng.choice([0, 0, 5, 100000, 2 ** 31])),
        key=int(rng.integers(1, 2 ** 63)),
        top_k=int(rng.choice([0, 1, 5, 40, 300, 5000])), top_p=float(rng.choice([1.0, 0.8, 0.5, 0.95, 0.1])),
        sigma=float(rng.choice([0.1, 1.0, 4.0])),
    )
    return cfg, rng


@pytest.mark.parametrize("seed", range(24))
def test_logit_entry_points(seed):
    dev = require_gpu()
    c, rng = _config(seed)
    B, V, ld = c["B"], c["V"], c["V"] + c["pad"]
    x = inputs.logits_normal(B, ld, c["sigma"], c["dtype"], seed=seed)
    if seed % 5 == 0:
        x = torch.round(x)                                    # ties
    ctx = inputs.uniform_tokens((B, c["W"]), 200000, seed=seed + 50)
    args = (c["key"], c["gamma"], c["delta"], c["scheme"])
    xo, co = host_bits(x), ctx.numpy()

    # bias, in place; padding untouched
    xd = x.to(dev)
    sbw.sbw_bias_logits(xd, ctx.to(dev), *args, V=V, vocab_offset=c["off"])
    torch.cuda.synchronize()
    assert_same_bits(host_bits(xd), oracle.bias_logits(xo, V, co, *args, vocab_offset=c["off"]))

    # bias on the top-k candidates
    k = max(c["top_k"], 1)
    xd = x.to(dev)
    sbw.sbw_bias_logits_topk(xd, ctx.to(dev), *args, k, V=V, vocab_offset=c["off"])
    torch.cuda.synchronize()
    assert_same_bits(host_bits(xd), oracle.bias_logits_topk(xo, V, co, *args, k, vocab_offset=c["off"])[0])

    # fused sampler and its truncated variant
    ids = torch.empty(B, dtype=torch.int32, device=dev)
    ws = torch.empty(max(sbw.sbw_sample_workspace_bytes(B, V), 256), dtype=torch.uint8, device=dev)
    sbw.sbw_bias_sample(x.to(dev), ctx.to(dev), *args, c["tau"], 77, seed, ids, ws, V=V, vocab_offset=c["off"])
    torch.cuda.synchronize()
    want = oracle.bias_sample(xo, V, co, *args, c["tau"], 77, seed, vocab_offset=c["off"])
    assert np.array_equal(ids.cpu().numpy(), want["tokens"])
    kept = torch.empty(B, dtype=torch.int32, device=dev)
    wsf = torch.empty(max(sbw.sbw_sample_filtered_workspace_bytes(c["dtype"], B, V), 256), dtype=torch.uint8,
                      device=dev)
    sbw.sbw_bias_sample_filtered(x.to(dev), ctx.to(dev), *args, c["tau"], c["top_k"], c["top_p"], 77, seed, ids,
                                 wsf, out_kept=kept, V=V, vocab_offset=c["off"])
    torch.cuda.synchronize()
    want = oracle.bias_sample_filtered(xo, V, co, *args, c["tau"], c["top_k"], c["top_p"], 77, seed,
                                       vocab_offset=c["off"])
    assert np.array_equal(kept.cpu().numpy(), want["kept"]) and np.array_equal(ids.cpu().numpy(), want["tokens"])


@pytest.mark.parametrize("seed", range(16))
def test_sequence_entry_points(seed):
    dev = require_gpu()
    c, rng = _config(seed + 100)
    N = int(rng.integers(1, 70))
    alphabet = int(rng.choice([2, 6, 100, 128256]))
    lens = rng.integers(0, int(rng.choice([5, 40, 300, 2000])), size=N).astype(np.int32)
    tok = rng.integers(0, alphabet, size=int(lens.sum())).astype(np.int32)
    W, scheme, gamma, key = c["W"], c["scheme"], c["gamma"], c["key"]
    t, l = torch.from_numpy(tok).to(dev), torch.from_numpy(lens).to(dev)
    total = t.numel()
    counts = torch.empty(N, dtype=torch.int32, device=dev)
    T = torch.empty(N, dtype=torch.int32, device=dev)
    z = torch.empty(N, dtype=torch.float64, device=dev)
    bits = torch.zeros(sbw.sbw_detect_bits_words(N, total), dtype=torch.int32, device=dev)
    ws = torch.empty(sbw.sbw_detect_workspace_bytes(N), dtype=torch.uint8, device=dev)
    sbw.sbw_detect_bits(t, l, key, gamma, scheme, counts, z, bits, out_T=T, workspace=ws, ctx_width=W)
    torch.cuda.synchronize()
    oc, oT, oz = oracle.detect(tok, lens, key, gamma, scheme, ctx_width=W)
    assert np.array_equal(counts.cpu().numpy(), oc) and np.array_equal(T.cpu().numpy(), oT)
    assert np.max(np.abs(z.cpu().numpy() - oz), initial=0) <= 1e-9
    green = oracle.detect_bits(tok, lens, key, gamma, scheme, ctx_width=W)
    offs = ws[:8 * (N + 1)].view(torch.int64)

    window = int(rng.integers(1, 60))
    scratch = torch.empty_like(bits)
    bc, bs, bz = (torch.empty(N, dtype=torch.int32, device=dev), torch.empty(N, dtype=torch.int32, device=dev),
                  torch.empty(N, dtype=torch.float64, device=dev))
    sbw.sbw_window_z(bits, l, offs, total, window, gamma, scratch, bc, bs, bz, ctx_width=W)
    keep = torch.from_numpy(rng.integers(-2, 2100, size=N).astype(np.int32)).to(dev)
    pc, pz = torch.empty_like(counts), torch.empty_like(z)
    sbw.sbw_prefix_z(bits, l, offs, keep, total, gamma, pc, pz, ctx_width=W)
    uc, uT, uz = torch.empty_like(counts), torch.empty_like(counts), torch.empty_like(z)
    max_len = int(lens.max(initial=0))
    uws = torch.empty(max(sbw.sbw_detect_unique_workspace_bytes(N, total, max_len), 256), dtype=torch.uint8,
                      device=dev)
    sbw.sbw_detect_unique(t, l, max_len, key, gamma, scheme, uc, uz, uws, out_T=uT, ctx_width=W)
    labels = torch.from_numpy(rng.integers(0, 2, size=N).astype(np.uint8)).to(dev)
    auc = torch.empty(1, dtype=torch.float64, device=dev)
    stats = torch.empty(4, dtype=torch.int64, device=dev)
    rws = torch.empty(sbw.sbw_roc_auc_workspace_bytes(N), dtype=torch.uint8, device=dev)
    sbw.sbw_roc_auc(z, labels, auc, rws, out_stats=stats)
    torch.cuda.synchronize()

    wc, wst, wz = oracle.window_z(green, lens, window, gamma, ctx_width=W)
    assert np.array_equal(bc.cpu().numpy(), wc) and np.array_equal(bs.cpu().numpy(), wst)
    assert np.max(np.abs(bz.cpu().numpy() - wz), initial=0) <= 1e-9
    qc, _, qz = oracle.prefix_z(green, lens, keep.cpu().numpy(), gamma, ctx_width=W)
    assert np.array_equal(pc.cpu().numpy(), qc) and np.max(np.abs(pz.cpu().numpy() - qz), initial=0) <= 1e-9
    ouc, ouT, ouz = oracle.detect_unique(tok, lens, key, gamma, scheme, ctx_width=W, threads=4)
    assert np.array_equal(uc.cpu().numpy(), ouc) and np.array_equal(uT.cpu().numpy(), ouT)
    assert np.max(np.abs(uz.cpu().numpy() - ouz), initial=0) <= 1e-9
    oa, ost = oracle.roc_auc(z.cpu().numpy(), labels.cpu().numpy())
    assert np.array_equal(stats.cpu().numpy().astype(np.uint64), ost)
    a = float(auc.cpu()[0])
    assert (np.isnan(a) and np.isnan(oa)) or a == oa
