"""GPU parity of sbw_bias_sample against the CPU oracle: sampled ids bit-exact given the same
RNG counter, row maximum exact, softmax sum / sampled probability / full probabilities within
1e-6 relative of the oracle's fp64 values."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_03844_b200 as sbw
from paper_2609_03844_b200 import inputs
from gpu_util import KEY, host_bits, require_gpu

pytestmark = pytest.mark.gpu

SCHEMES = [sbw.SCHEME_CONTEXT, sbw.SCHEME_SELFSALT]
REL = 1e-6
FLT_MIN = 1.1754943508222875e-38


def _sample(x, V, ctx, key, gamma, delta, scheme, tau, seed, step, off=0, want_probs=False, view=None):
    dev = require_gpu()
    B = x.shape[0]
    x_dev = x.to(dev)
    target = x_dev if view is None else view(x_dev)
    before = host_bits(x_dev)
    out = {
        "tokens": torch.full((B,), -1, dtype=torch.int32, device=dev),
        "max": torch.zeros(B, dtype=torch.float32, device=dev),
        "sumexp": torch.zeros(B, dtype=torch.float32, device=dev),
        "prob": torch.zeros(B, dtype=torch.float32, device=dev),
        "probs": torch.zeros((B, V), dtype=torch.float32, device=dev) if want_probs else None,
    }
    ws = torch.empty(sbw.sbw_sample_workspace_bytes(B, V), dtype=torch.uint8, device=dev)
    sbw.sbw_bias_sample(target, ctx.to(dev), key, gamma, delta, scheme, tau, seed, step, out["tokens"], ws,
                        out_max=out["max"], out_sumexp=out["sumexp"], out_prob=out["prob"],
                        out_probs=out["probs"], V=V, vocab_offset=off)
    torch.cuda.synchronize()
    assert host_bits(x_dev).tobytes() == before.tobytes()           # logits are read-only
    return {k: (None if v is None else v.cpu().numpy()) for k, v in out.items()}


def _check(x, V, ctx, key, gamma, delta, scheme, tau, seed, step, off=0, want_probs=False, view=None):
    got = _sample(x, V, ctx, key, gamma, delta, scheme, tau, seed, step, off, want_probs, view)
    src = x if view is None else view(x).contiguous()
    want = oracle.bias_sample(host_bits(src), V, ctx.numpy(), key, gamma, delta, scheme, tau, seed, step,
                              vocab_offset=off, want_probs=want_probs, threads=8)
    assert np.array_equal(got["tokens"], want["tokens"])
    assert np.array_equal(got["max"].astype(np.float64), want["max"])
    assert np.max(np.abs(got["sumexp"] / want["sumexp"] - 1.0)) <= REL
    assert np.max(np.abs(got["prob"] / want["prob"] - 1.0)) <= REL
    if want_probs:
        normal = want["probs"] >= FLT_MIN
        rel = np.abs(got["probs"][normal] / want["probs"][normal] - 1.0)
        assert rel.max() <= REL
        assert np.all(got["probs"][~normal] < 2 * FLT_MIN)
    return got, want


def test_config1_shape_fp32_with_probs():
    x = inputs.logits_normal(1, 32000, 3.0, torch.float32, seed=0)
    ctx = inputs.uniform_tokens((1, 1), 32000, seed=1)
    for scheme in SCHEMES:
        _check(x, 32000, ctx, KEY, 0.25, 2.0, scheme, 0.7, 0xC4, 0, want_probs=True)


@pytest.mark.parametrize("scheme", SCHEMES)
@pytest.mark.parametrize("B", [1, 8, 32])
def test_config4_small_batches_split_rows(B, scheme):
    """V=128256 bf16 N(0, 4^2), tau 0.7: rows are split over many CTAs and merged by the last one."""
    x = inputs.logits_normal(B, 128256, 4.0, torch.bfloat16, seed=100 + B)
    ctx = inputs.uniform_tokens((B, 1), 128256, seed=200 + B)
    for step in (0, 1):
        _check(x, 128256, ctx, KEY, 0.25, 2.0, scheme, 0.7, 0xC4, step, want_probs=(B <= 8 and step == 0))


@pytest.mark.parametrize("gamma", [0.25, 0.5])
@pytest.mark.parametrize("delta", [0.5, 1.0, 2.0, 4.0])
def test_config4_gamma_delta_grid(gamma, delta):
    x = inputs.logits_normal(8, 128256, 4.0, torch.bfloat16, seed=300)
    ctx = inputs.uniform_tokens((8, 1), 128256, seed=301)
    for scheme in SCHEMES:
        _check(x, 128256, ctx, KEY, gamma, delta, scheme, 0.7, 0xC4, 5)


@pytest.mark.parametrize("B,scheme", [(128, sbw.SCHEME_CONTEXT), (128, sbw.SCHEME_SELFSALT),
                                      (512, sbw.SCHEME_CONTEXT), (1024, sbw.SCHEME_SELFSALT)])
def test_config4_large_batches(B, scheme):
    dev = require_gpu()
    x = inputs.logits_normal(B, 128256, 4.0, torch.bfloat16, seed=400 + B, device=dev).cpu()
    ctx = inputs.uniform_tokens((B, 1), 128256, seed=500 + B)
    _check(x, 128256, ctx, KEY, 0.5, 2.0, scheme, 0.7, 0xC4, (1 << 33) + 9)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("scheme", SCHEMES)
def test_ragged_unaligned_offset_and_wide_context(dtype, scheme):
    B, V = 5, 10007
    x = inputs.logits_normal(B, V + 9, 4.0, dtype, seed=600)
    ctx = inputs.uniform_tokens((B, 4), 151936, seed=601)
    _check(x, V, ctx, KEY, 0.25, 2.0, scheme, 0.7, 1, 2, off=3, want_probs=True)            # padded rows
    _check(x, V, ctx, KEY, 0.25, 2.0, scheme, 1.0, 1, 2, off=123456, view=lambda t: t[:, 1:V + 1])  # unaligned
    for v in (1, 3, 8, 9):
        _check(x[:, :v].contiguous(), v, ctx, KEY, 0.5, 1.0, scheme, 0.7, 1, 3, want_probs=True)


def test_zipf_spike_rows_fp32_selfsalt():
    """Config 3's logits (confident rows): the winner is usually a spiked id; statistics hold."""
    x = inputs.logits_normal(16, 151936, 4.0, torch.float32, seed=700)
    inputs.add_zipf_spike_(x, 151936, seed=701)
    ctx = inputs.uniform_tokens((16, 1), 151936, seed=702)
    _check(x, 151936, ctx, KEY, 0.25, 4.0, sbw.SCHEME_SELFSALT, 0.7, 0xC4, 1)


def test_masked_logits_ties_and_temperature_extremes():
    dev = require_gpu()
    V = 5000
    x = inputs.logits_normal(6, V, 4.0, torch.float32, seed=800)
    x[0, :] = float("-inf")                         # all masked: id 0
    x[1, :] = float("-inf")
    x[1, 4321] = 0.5                                 # a single survivor
    x[2, 100:4000] = float("-inf")                  # many masked
    x[3, :] = 1e30                                   # the Gumbel is absorbed: all scores tie -> lowest id
    ctx = inputs.uniform_tokens((6, 1), V, seed=801)
    got = _sample(x, V, ctx, KEY, 0.25, 2.0, sbw.SCHEME_CONTEXT, 0.7, 3, 4)
    want = oracle.bias_sample(host_bits(x), V, ctx.numpy(), KEY, 0.25, 2.0, 0, 0.7, 3, 4)
    assert np.array_equal(got["tokens"], want["tokens"])
    assert got["tokens"][0] == 0 and got["tokens"][1] == 4321 and got["tokens"][3] == 0
    rows = [1, 2, 4, 5]
    assert np.max(np.abs(got["sumexp"][rows] / want["sumexp"][rows] - 1)) <= REL
    assert np.max(np.abs(got["prob"][rows] / want["prob"][rows] - 1)) <= REL
    # cold and hot temperatures
    y = inputs.logits_normal(4, V, 4.0, torch.bfloat16, seed=802)
    for tau in (1e-3, 0.05, 5.0, 100.0):
        _check(y, V, ctx[:4], KEY, 0.25, 2.0, sbw.SCHEME_SELFSALT, tau, 3, 4)
    del dev


def test_sampled_tokens_feed_the_next_step():
    """A short autoregressive chain: each row's sampled id is its next context token."""
    dev = require_gpu()
    B, V, steps = 4, 32000, 6
    ctx = inputs.uniform_tokens((B, 1), V, seed=900)
    ctx_dev, ctx_host = ctx.to(dev), ctx.numpy().copy()
    ws = torch.empty(sbw.sbw_sample_workspace_bytes(B, V), dtype=torch.uint8, device=dev)
    for t in range(steps):
        x = inputs.logits_normal(B, V, 4.0, torch.bfloat16, seed=910 + t)
        nxt = torch.empty(B, dtype=torch.int32, device=dev)
        sbw.sbw_bias_sample(x.to(dev), ctx_dev, KEY, 0.25, 2.0, sbw.SCHEME_SELFSALT, 0.7, 0xC4, t, nxt, ws)
        want = oracle.bias_sample(host_bits(x), V, ctx_host, KEY, 0.25, 2.0, 1, 0.7, 0xC4, t)
        torch.cuda.synchronize()
        assert np.array_equal(nxt.cpu().numpy(), want["tokens"])
        ctx_dev = nxt.view(B, 1)
        ctx_host = want["tokens"].reshape(B, 1).copy()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("scheme", SCHEMES)
@pytest.mark.parametrize("delta", [0.5, 4.0, -1.5, 0.0])
def test_ids_only_calls_skip_the_green_test_where_it_cannot_matter(dtype, scheme, delta):
    """Without statistics outputs the kernel screens on the Gumbel words first and hashes only the
    candidates that could win with the largest possible bias: the ids must not change."""
    dev = require_gpu()
    for B, V, ld, tau in ((1, 128256, 128256, 0.7), (9, 20011, 20016, 1.3), (130, 5000, 5003, 0.3)):
        x = inputs.logits_normal(B, ld, 3.0, dtype, seed=7 + B)
        ctx = inputs.uniform_tokens((B, 2), V, seed=8 + B)
        xd, cd = x.to(dev), ctx.to(dev)
        ws = torch.empty(sbw.sbw_sample_workspace_bytes(B, V), dtype=torch.uint8, device=dev)
        ids = torch.empty(B, dtype=torch.int32, device=dev)
        ids_stats = torch.empty(B, dtype=torch.int32, device=dev)
        m = torch.empty(B, dtype=torch.float32, device=dev)
        for step in range(3):
            sbw.sbw_bias_sample(xd, cd, KEY, 0.25, delta, scheme, tau, 3, step, ids, ws, V=V, vocab_offset=11)
            sbw.sbw_bias_sample(xd, cd, KEY, 0.25, delta, scheme, tau, 3, step, ids_stats, ws, out_max=m, V=V,
                                vocab_offset=11)
            torch.cuda.synchronize()
            want = oracle.bias_sample(host_bits(x), V, ctx.numpy(), KEY, 0.25, delta, scheme, tau, 3, step,
                                      vocab_offset=11, threads=8)
            assert np.array_equal(ids.cpu().numpy(), want["tokens"])
            assert np.array_equal(ids_stats.cpu().numpy(), want["tokens"])


@pytest.mark.parametrize("dtype,base", [(torch.bfloat16, 256.0), (torch.float32, 16777216.0)])
def test_ids_only_screen_allows_for_the_rounding_of_the_biased_sum(dtype, base):
    """Logits next to a power of two, where l + delta rounds up by half a spacing: the screen's
    bound on the biased value must cover that."""
    dev = require_gpu()
    B, V = 4, 6000
    rng = np.random.default_rng(5)
    step = base / 256.0
    x = torch.from_numpy(base + step * rng.integers(-6, 3, size=(B, V))).to(dtype)
    ctx = inputs.uniform_tokens((B, 1), V, seed=6)
    xd, cd = x.to(dev), ctx.to(dev)
    ws = torch.empty(sbw.sbw_sample_workspace_bytes(B, V), dtype=torch.uint8, device=dev)
    ids = torch.empty(B, dtype=torch.int32, device=dev)
    tau = float(step)                                          # scores then differ by O(1) between neighbours
    for delta in (1.0, 3.0):
        for step_no in range(12):
            sbw.sbw_bias_sample(xd, cd, KEY, 0.5, delta * step, 0, tau, 3, step_no, ids, ws)
            torch.cuda.synchronize()
            want = oracle.bias_sample(host_bits(x), V, ctx.numpy(), KEY, 0.5, delta * step, 0, tau, 3, step_no)
            assert np.array_equal(ids.cpu().numpy(), want["tokens"])


def test_config4_all_96_combinations():
    """Config 4 in full: B in {1, 8, 32, 128, 512, 1024} x both schemes x gamma in {.25, .5} x delta in
    {.5, 1, 2, 4}, V = 128256 bf16, tau 0.7.  The batches are the leading rows of one tensor, so one
    oracle pass per (scheme, gamma, delta) serves all six batch sizes; ids bit-exact from both
    kernels (with and without statistics), m exact, Z and p within 1e-6."""
    import os

    dev = require_gpu()
    threads = min(32, os.cpu_count() or 8)
    V, Bmax, tau = 128256, 1024, 0.7
    x = inputs.logits_normal(Bmax, V, 4.0, torch.bfloat16, seed=0xC4, device=dev)
    ctx = inputs.uniform_tokens((Bmax, 1), V, seed=0xC5, device=dev)
    xh, ch = host_bits(x), ctx.cpu().numpy()
    ws = torch.empty(sbw.sbw_sample_workspace_bytes(Bmax, V), dtype=torch.uint8, device=dev)
    ids, ids_only = (torch.empty(Bmax, dtype=torch.int32, device=dev) for _ in range(2))
    m, Z, p = (torch.empty(Bmax, dtype=torch.float32, device=dev) for _ in range(3))
    step = 0
    for scheme in SCHEMES:
        for gamma in (0.25, 0.5):
            for delta in (0.5, 1.0, 2.0, 4.0):
                step += 1
                want = oracle.bias_sample(xh, V, ch, KEY, gamma, delta, scheme, tau, 0xC4, step, threads=threads)
                for B in (1, 8, 32, 128, 512, 1024):
                    sbw.sbw_bias_sample(x[:B], ctx[:B], KEY, gamma, delta, scheme, tau, 0xC4, step, ids[:B], ws,
                                        out_max=m[:B], out_sumexp=Z[:B], out_prob=p[:B])
                    sbw.sbw_bias_sample(x[:B], ctx[:B], KEY, gamma, delta, scheme, tau, 0xC4, step, ids_only[:B], ws)
                    torch.cuda.synchronize()
                    tag = (scheme, gamma, delta, B)
                    assert np.array_equal(ids[:B].cpu().numpy(), want["tokens"][:B]), tag
                    assert np.array_equal(ids_only[:B].cpu().numpy(), want["tokens"][:B]), tag
                    assert np.array_equal(m[:B].cpu().numpy().astype(np.float64), want["max"][:B]), tag
                    assert np.max(np.abs(Z[:B].cpu().numpy() / want["sumexp"][:B] - 1.0)) <= REL, tag
                    assert np.max(np.abs(p[:B].cpu().numpy() / want["prob"][:B] - 1.0)) <= REL, tag
