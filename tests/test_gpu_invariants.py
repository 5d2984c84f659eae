"""Invariants of the library that hold whatever the inputs: no device memory is allocated by any
entry point (the paper's Section 5.1 "in-place, zero allocation" and the 0 MB column of its memory
table, Appendix E), the softmax sum keeps its accuracy on rows built to stress it, and the
host-buffer entry point matches the oracle at the size the benchmark's end-to-end figure uses."""
import gc

import numpy as np
import pytest
import torch

import paper_2609_03844_b200 as sbw
from paper_2609_03844_b200 import binding, inputs
from gpu_util import KEY, assert_same_bits, host_bits, require_gpu


def _entry_point_calls(dev):
    """One closure per C entry point, every output and workspace allocated beforehand."""
    B, V = 16, 32000
    x32 = inputs.logits_normal(B, V, 4.0, torch.float32, seed=1, device=dev)
    x16 = inputs.logits_normal(B, V, 4.0, torch.bfloat16, seed=2, device=dev)
    ctx = inputs.uniform_tokens((B, 1), V, seed=3, device=dev)
    ids = torch.empty(B, dtype=torch.int32, device=dev)
    kept = torch.empty(B, dtype=torch.int32, device=dev)
    m, Z, p = (torch.empty(B, dtype=torch.float32, device=dev) for _ in range(3))
    ws = torch.empty(sbw.sbw_sample_workspace_bytes(B, V), dtype=torch.uint8, device=dev)
    wsf = torch.empty(sbw.sbw_sample_filtered_workspace_bytes(torch.bfloat16, B, V), dtype=torch.uint8, device=dev)
    summ = torch.empty((2, B, 8), dtype=torch.float32, device=dev)
    half = V // 2
    N = 300
    tokens, lengths = inputs.null_token_streams(N, 5, 400, V, seed=4, device=dev)
    total = tokens.numel()
    offsets = torch.zeros(N + 1, dtype=torch.int64, device=dev)
    offsets[1:] = torch.cumsum(lengths.to(torch.int64), 0)
    counts, T = (torch.empty(N, dtype=torch.int32, device=dev) for _ in range(2))
    start = torch.empty(N, dtype=torch.int32, device=dev)
    keep = torch.full((N,), 50, dtype=torch.int32, device=dev)
    z = torch.empty(N, dtype=torch.float64, device=dev)
    wsd = torch.empty(sbw.sbw_detect_workspace_bytes(N), dtype=torch.uint8, device=dev)
    wsu = torch.empty(sbw.sbw_detect_unique_workspace_bytes(N, total, 400), dtype=torch.uint8, device=dev)
    bits = torch.zeros(sbw.sbw_detect_bits_words(N, total), dtype=torch.int32, device=dev)
    scratch = torch.zeros_like(bits)
    labels = (torch.arange(N, device=dev) % 2).to(torch.uint8)
    auc = torch.empty(4, dtype=torch.float64, device=dev)
    wsr = torch.empty(sbw.sbw_roc_auc_workspace_bytes(N), dtype=torch.uint8, device=dev)
    roc_off = torch.tensor([0, 100, 200, 300], dtype=torch.int64, device=dev)
    hx = inputs.logits_normal(B, V, 4.0, torch.bfloat16, seed=5).pin_memory()
    hctx = inputs.uniform_tokens((B, 1), V, seed=6).pin_memory()
    staging = torch.empty(sbw.sbw_bias_logits_host_staging_bytes(torch.bfloat16, B, V, 1), dtype=torch.uint8, device=dev)
    S0, S1 = sbw.SCHEME_CONTEXT, sbw.SCHEME_SELFSALT
    return {
        "sbw_bias_logits": lambda i: (sbw.sbw_bias_logits(x32, ctx, KEY, 0.25, 2.0, S1),
                                      sbw.sbw_bias_logits(x16, ctx, KEY, 0.5, 2.0, S0)),
        "sbw_bias_logits_topk": lambda i: sbw.sbw_bias_logits_topk(x32, ctx, KEY, 0.25, 2.0, S1, 40),
        "sbw_bias_logits_host": lambda i: sbw.sbw_bias_logits_host(hx, hctx, KEY, 0.5, 2.0, S0, staging),
        "sbw_bias_sample": lambda i: (sbw.sbw_bias_sample(x16, ctx, KEY, 0.25, 2.0, S0, 0.7, 1, i, ids, ws, out_max=m,
                                                          out_sumexp=Z, out_prob=p),
                                      sbw.sbw_bias_sample(x32, ctx, KEY, 0.25, 2.0, S1, 0.7, 1, i, ids, ws)),
        "sbw_bias_sample_noalloc": lambda i: sbw.sbw_bias_sample_noalloc(x16, ctx, KEY, 0.25, 2.0, S0, 0.7, 1, i, ids,
                                                                         out_sumexp=Z),
        "sbw_bias_sample_shard + combine": lambda i: (
            sbw.sbw_bias_sample_shard(x16[:, :half], ctx, KEY, 0.25, 2.0, S0, 0.7, 1, i, summ[0], ids, ws, vocab_offset=0),
            sbw.sbw_bias_sample_shard(x16[:, half:], ctx, KEY, 0.25, 2.0, S0, 0.7, 1, i, summ[1], ids, ws,
                                      vocab_offset=half, ids_only=False),
            sbw.sbw_sample_combine(summ, 0.7, ids, out_sumexp=Z)),
        "sbw_bias_sample_filtered": lambda i: (
            sbw.sbw_bias_sample_filtered(x16, ctx, KEY, 0.25, 2.0, S0, 0.7, 0, 0.8, 1, i, ids, wsf, out_kept=kept),
            sbw.sbw_bias_sample_filtered(x16, ctx, KEY, 0.25, 2.0, S0, 0.7, 50, 1.0, 1, i, ids, wsf)),
        "sbw_detect": lambda i: (sbw.sbw_detect(tokens, lengths, KEY, 0.25, S0, counts, z, workspace=wsd, out_T=T),
                                 sbw.sbw_detect(tokens, lengths, KEY, 0.25, S1, counts, z, offsets=offsets)),
        "sbw_detect_bits, window, prefix": lambda i: (
            sbw.sbw_detect_bits(tokens, lengths, KEY, 0.25, S0, counts, z, bits, offsets=offsets),
            sbw.sbw_window_z(bits, lengths, offsets, total, 64, 0.25, scratch, counts, start, z),
            sbw.sbw_prefix_z(bits, lengths, offsets, keep, total, 0.25, counts, z)),
        "sbw_detect_unique": lambda i: sbw.sbw_detect_unique(tokens, lengths, 400, KEY, 0.25, S0, counts, z, wsu),
        "sbw_roc_auc": lambda i: (sbw.sbw_roc_auc(z, labels, auc, wsr),
                                  sbw.sbw_roc_auc_batched(z, labels, roc_off, auc)),
    }


@pytest.mark.gpu
def test_no_entry_point_allocates_device_memory():
    """Free device memory (cudaMemGetInfo) and torch's allocator are the same before and after a
    few hundred calls of every entry point.  Each call is made once beforehand: the first launch
    of a kernel loads its code, which is not the library allocating."""
    dev = require_gpu()
    calls = _entry_point_calls(dev)
    for fn in calls.values():
        fn(0)
    torch.cuda.synchronize()

    def one_pass():
        gc.collect()                                           # tensors left by earlier tests go now, not mid-pass
        free0, _ = torch.cuda.mem_get_info(dev)
        torch0 = torch.cuda.memory_allocated(dev), torch.cuda.memory_reserved(dev)
        for name, fn in calls.items():
            for i in range(200):
                fn(i + 1)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info(dev)
        return free0 - free1, torch0 == (torch.cuda.memory_allocated(dev), torch.cuda.memory_reserved(dev))

    # the GPU's free memory is a device-wide figure: one repeat in case something else moved it
    results = [one_pass()]
    if results[0][0] != 0:
        results.append(one_pass())
    assert all(same for _, same in results)                    # torch saw no allocation
    assert any(delta == 0 for delta, _ in results), results    # nor did the driver


@pytest.mark.gpu
@pytest.mark.parametrize("tau", [0.3, 0.7, 1.0])
def test_softmax_sum_on_rows_built_to_stress_it(oracle, tau):
    """Rows whose softmax mass sits far below the maximum, where every term's exponent is large and
    its fp32 rounding error does not average out: one dominant logit and 131071 logits 8 to 20
    units (and 8 tau to 20 tau units) below it, spread out, all equal, or on a few values."""
    dev = require_gpu()
    V = 131072
    g = torch.Generator().manual_seed(1234)
    rows = []
    for lo, hi in ((8.0, 20.0), (8.0 * tau, 20.0 * tau)):
        spread = 7.25 - (lo + (hi - lo) * torch.rand(V, generator=g))
        equal = torch.full((V,), 7.25 - 0.5 * (lo + hi) - 0.123456)
        few = 7.25 - torch.tensor([lo, 0.5 * (lo + hi), hi])[torch.randint(0, 3, (V,), generator=g)] - 0.0371
        for r in (spread, equal, few):
            r = r.clone()
            r[int(torch.randint(0, V, (1,), generator=g))] = 7.25
            rows.append(r)
    x = torch.stack(rows).to(torch.float32).contiguous()
    B = x.shape[0]
    ctx = inputs.uniform_tokens((B, 1), V, seed=77)
    for scheme, delta in ((sbw.SCHEME_CONTEXT, 2.0), (sbw.SCHEME_SELFSALT, 0.5), (sbw.SCHEME_CONTEXT, -1.0)):
        want = oracle.bias_sample(x.numpy(), V, ctx.numpy(), KEY, 0.25, delta, scheme, tau, 5, 9, threads=8)
        xd, cd = x.to(dev), ctx.to(dev)
        ids = torch.empty(B, dtype=torch.int32, device=dev)
        m, Z, p = (torch.empty(B, dtype=torch.float32, device=dev) for _ in range(3))
        ws = torch.empty(sbw.sbw_sample_workspace_bytes(B, V), dtype=torch.uint8, device=dev)
        sbw.sbw_bias_sample(xd, cd, KEY, 0.25, delta, scheme, tau, 5, 9, ids, ws, out_max=m, out_sumexp=Z, out_prob=p)
        torch.cuda.synchronize()
        assert np.array_equal(ids.cpu().numpy(), want["tokens"])
        assert np.array_equal(m.cpu().numpy().astype(np.float64), want["max"])
        rel = np.abs(Z.cpu().numpy().astype(np.float64) / want["sumexp"] - 1.0)
        assert rel.max() <= 1e-6, (scheme, delta, rel)
        ok = want["prob"] >= np.finfo(np.float32).tiny
        relp = np.abs(p.cpu().numpy().astype(np.float64)[ok] / want["prob"][ok] - 1.0)
        assert relp.size == 0 or relp.max() <= 1e-6, (scheme, delta, relp)


@pytest.mark.gpu
def test_host_entry_point_at_the_benchmark_shape(oracle):
    """sbw_bias_logits_host on the headline workload's shape (64 x 128256 bf16, context scheme,
    gamma 0.5, delta 2): the call the benchmark's end-to-end figure times."""
    dev = require_gpu()
    B, V = 64, 128256
    hx = inputs.logits_normal(B, V, 4.0, torch.bfloat16, seed=4711).pin_memory()
    hctx = inputs.uniform_tokens((B, 1), V, seed=4712).pin_memory()
    want = oracle.bias_logits(host_bits(hx), V, hctx.numpy(), KEY, 0.5, 2.0, 0, threads=8)
    staging = torch.empty(sbw.sbw_bias_logits_host_staging_bytes(torch.bfloat16, B, V, 1), dtype=torch.uint8, device=dev)
    sbw.sbw_bias_logits_host(hx, hctx, KEY, 0.5, 2.0, sbw.SCHEME_CONTEXT, staging)
    torch.cuda.synchronize()
    assert_same_bits(host_bits(hx), want)
    # a rejected call enqueues nothing: the host buffer keeps its bits
    before = host_bits(hx)
    with pytest.raises(sbw.SbwError):
        sbw.sbw_bias_logits_host(hx, hctx, KEY, 0.5, float("nan"), sbw.SCHEME_CONTEXT, staging)
    torch.cuda.synchronize()
    assert_same_bits(host_bits(hx), before)


@pytest.mark.gpu
def test_process_exits_cleanly_after_library_calls():
    """A process that used the library, synchronised and left ends with status 0 (the library is
    linked against the CUDA runtime torch loads; its teardown must not depend on unload order)."""
    import subprocess
    import sys
    from pathlib import Path

    require_gpu()
    root = Path(__file__).resolve().parent.parent
    code = ("import torch, paper_2609_03844_b200 as sbw\n"
            "from paper_2609_03844_b200 import inputs\n"
            "x = inputs.logits_normal(4, 4096, 4.0, torch.bfloat16, seed=1, device='cuda')\n"
            "c = inputs.uniform_tokens((4, 1), 4096, seed=2, device='cuda')\n"
            "ids = torch.empty(4, dtype=torch.int32, device='cuda')\n"
            "ws = torch.empty(sbw.sbw_sample_workspace_bytes(4, 4096), dtype=torch.uint8, device='cuda')\n"
            "sbw.sbw_bias_logits(x, c, 0x5EED, 0.5, 2.0, 0)\n"
            "sbw.sbw_bias_sample(x, c, 0x5EED, 0.25, 2.0, 1, 0.7, 1, 2, ids, ws)\n"
            "torch.cuda.synchronize()\n"
            "print(int(ids.min()) >= 0)\n")
    out = subprocess.run([sys.executable, "-c", code], cwd=root, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, (out.returncode, out.stderr[-1000:])
    assert out.stdout.strip().endswith("True")
