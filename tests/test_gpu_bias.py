"""GPU parity of sbw_bias_logits (Eq. 1 + Eq. 2) against the CPU oracle: biased logits must be
bit-identical, element by element, on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_03844_b200 as sbw
from paper_2609_03844_b200 import inputs
from gpu_util import KEY, assert_same_bits, host_bits, require_gpu

pytestmark = pytest.mark.gpu

SCHEMES = [sbw.SCHEME_CONTEXT, sbw.SCHEME_SELFSALT]
DTYPES = [torch.float32, torch.bfloat16]


def _run(x_host: torch.Tensor, V, ctx_host: torch.Tensor, key, gamma, delta, scheme, off=0,
         view=None):
    """Runs the CUDA path on a device copy and the oracle on the host bytes; returns both."""
    dev = require_gpu()
    x_dev = x_host.to(dev)
    target = x_dev if view is None else view(x_dev)
    host_view = x_host if view is None else view(x_host)
    sbw.sbw_bias_logits(target, ctx_host.to(dev), key, gamma, delta, scheme, V=V, vocab_offset=off)
    torch.cuda.synchronize()
    want = oracle.bias_logits(host_bits(host_view.contiguous()) if view is not None else host_bits(x_host),
                              V, ctx_host.numpy(), key, gamma, delta, scheme, vocab_offset=off, threads=8)
    got_full = host_bits(x_dev)
    got = host_bits(target.contiguous()) if view is not None else got_full
    return got, want, got_full


def test_config1_fp32_context():
    """B=1, V=32000, fp32 N(0, 3^2) from seed 0, one context token, key 0x5EED, gamma .25, delta 2."""
    x = inputs.logits_normal(1, 32000, 3.0, torch.float32, seed=0)
    ctx = inputs.uniform_tokens((1, 1), 32000, seed=1)
    got, want, _ = _run(x, 32000, ctx, KEY, 0.25, 2.0, sbw.SCHEME_CONTEXT)
    assert_same_bits(got, want)
    changed = (got != host_bits(x)).mean()
    assert 0.23 < changed < 0.27


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("scheme", SCHEMES)
@pytest.mark.parametrize("W", [1, 4])
def test_several_tiles_ragged_tail_padding_offset(dtype, scheme, W):
    """Rows span several CTAs' shares, V is not a multiple of the vector width, ld > V."""
    B, V, ld, off = 37, 10007, 10016, 123457
    x = inputs.logits_normal(B, V, 4.0, dtype, seed=2, ld=ld)
    ctx = inputs.uniform_tokens((B, W), 151936, seed=3)
    got, want, _ = _run(x, V, ctx, KEY, 0.5, 2.0, scheme, off=off)
    assert_same_bits(got, want)
    assert np.array_equal(got[:, V:], host_bits(x)[:, V:])          # padding untouched


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("scheme", SCHEMES)
def test_unaligned_rows_take_the_scalar_path(dtype, scheme):
    """Odd row stride and a base pointer that is not 16-byte aligned (a column slice)."""
    B, V = 9, 1001
    x = inputs.logits_normal(B, V + 3, 4.0, dtype, seed=4)
    ctx = inputs.uniform_tokens((B, 1), 50000, seed=5)
    got, want, full = _run(x, V, ctx, KEY, 0.25, 1.0, scheme, view=lambda t: t[:, 1:V + 1])
    assert_same_bits(got, want)
    ref = host_bits(x)
    assert np.array_equal(full[:, 0], ref[:, 0]) and np.array_equal(full[:, V + 1:], ref[:, V + 1:])


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("V", [1, 3, 7, 8, 9, 31, 33])
def test_tiny_vocabularies_and_empty_batch(dtype, V):
    x = inputs.logits_normal(5, V, 4.0, dtype, seed=6 + V)
    ctx = inputs.uniform_tokens((5, 1), 1000, seed=7)
    for scheme in SCHEMES:
        got, want, _ = _run(x, V, ctx, KEY, 0.5, 2.0, scheme)
        assert_same_bits(got, want)
    dev = require_gpu()
    empty = torch.empty((0, V), dtype=dtype, device=dev)
    sbw.sbw_bias_logits(empty, torch.empty((0, 1), dtype=torch.int32, device=dev), KEY, 0.5, 2.0, 0, V=V)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("delta", [0.0, -1.5, 0.3, 4.0, 1e-3])
def test_delta_values_and_special_logits(dtype, delta):
    """-0.0, +-inf, subnormals, huge values, NaN (payload not compared); delta = 0 changes no bit."""
    B, V = 4, 4096
    x = inputs.logits_normal(B, V, 4.0, dtype, seed=8)
    specials = torch.tensor([0.0, -0.0, float("inf"), float("-inf"), 1e-40, -1e-40, 3e38, -3e38,
                             float("nan"), 1.0, -2.0, 65504.0], dtype=torch.float32).to(dtype)
    for b in range(B):
        x[b, b * 100:b * 100 + len(specials)] = specials
        x[b, 2000 + b:2000 + b + 24:2] = specials
    ctx = inputs.uniform_tokens((B, 1), 32000, seed=9)
    for scheme in SCHEMES:
        got, want, _ = _run(x, V, ctx, KEY, 0.5, delta, scheme)
        assert_same_bits(got, want, allow_nan_payload=True)
        if delta == 0.0:
            assert got.tobytes() == host_bits(x).tobytes()


def test_config2_shape_one_step_bf16():
    """B=64, V=128256 bf16 N(0, 4^2), context scheme, gamma .5, delta 2 -- every element."""
    dev = require_gpu()
    x = inputs.logits_normal(64, 128256, 4.0, torch.bfloat16, seed=20, device=dev)
    ctx = inputs.uniform_tokens((64, 1), 128256, seed=21, device=dev)
    before = host_bits(x)
    sbw.sbw_bias_logits(x, ctx, KEY, 0.5, 2.0, sbw.SCHEME_CONTEXT)
    torch.cuda.synchronize()
    want = oracle.bias_logits(before, 128256, ctx.cpu().numpy(), KEY, 0.5, 2.0,
                              oracle.SCHEME_CONTEXT, threads=8)
    assert_same_bits(host_bits(x), want)


def test_config2_all_256_decode_steps():
    """Config 2 in full: 256 consecutive decode steps, each on its own (64, 128256) bf16 tensor and
    context column, launched back to back as the benchmark does; every one of the 2.1e9 biased
    logits is compared with the oracle (16 steps resident at a time)."""
    import os

    dev = require_gpu()
    threads = min(32, os.cpu_count() or 8)
    for first in range(0, 256, 16):
        xs = [inputs.logits_normal(64, 128256, 4.0, torch.bfloat16, seed=5000 + t, device=dev)
              for t in range(first, first + 16)]
        cs = [inputs.uniform_tokens((64, 1), 128256, seed=6000 + t, device=dev) for t in range(first, first + 16)]
        before = [host_bits(x) for x in xs]
        for x, c in zip(xs, cs):
            sbw.sbw_bias_logits(x, c, KEY, 0.5, 2.0, sbw.SCHEME_CONTEXT)
        torch.cuda.synchronize()
        for x, c, b in zip(xs, cs, before):
            want = oracle.bias_logits(b, 128256, c.cpu().numpy(), KEY, 0.5, 2.0, oracle.SCHEME_CONTEXT, threads=threads)
            assert host_bits(x).tobytes() == want.tobytes()


def test_config3_shape_one_step_fp32_selfsalt_with_zipf_spike():
    """B=256, V=151936 fp32 N(0, 4^2) + Zipf(1.1) spike on 50 ids per row, self-salt, gamma .25,
    delta 4 -- every element."""
    dev = require_gpu()
    x = inputs.logits_normal(256, 151936, 4.0, torch.float32, seed=30, device=dev)
    inputs.add_zipf_spike_(x, 151936, seed=31)
    ctx = inputs.uniform_tokens((256, 1), 151936, seed=32, device=dev)
    before = host_bits(x)
    sbw.sbw_bias_logits(x, ctx, KEY, 0.25, 4.0, sbw.SCHEME_SELFSALT)
    torch.cuda.synchronize()
    want = oracle.bias_logits(before, 151936, ctx.cpu().numpy(), KEY, 0.25, 4.0,
                              oracle.SCHEME_SELFSALT, threads=8)
    assert_same_bits(host_bits(x), want)


def test_config3_sixteen_of_the_128_decode_steps():
    """Config 3 over a rotating pool: steps 0, 8, ..., 120 of the 128-step sequence (each its own
    (256, 151936) fp32 tensor with its Zipf spike and context column), every logit compared."""
    import os

    dev = require_gpu()
    threads = min(32, os.cpu_count() or 8)
    for t in range(0, 128, 8):
        x = inputs.logits_normal(256, 151936, 4.0, torch.float32, seed=7000 + t, device=dev)
        inputs.add_zipf_spike_(x, 151936, seed=7500 + t)
        ctx = inputs.uniform_tokens((256, 1), 151936, seed=8000 + t, device=dev)
        before = host_bits(x)
        sbw.sbw_bias_logits(x, ctx, KEY, 0.25, 4.0, sbw.SCHEME_SELFSALT)
        torch.cuda.synchronize()
        want = oracle.bias_logits(before, 151936, ctx.cpu().numpy(), KEY, 0.25, 4.0, oracle.SCHEME_SELFSALT,
                                  threads=threads)
        assert host_bits(x).tobytes() == want.tobytes(), t


def test_consecutive_steps_on_a_side_stream_and_other_keys():
    """Several decode steps enqueued back to back on a non-default stream, 64-bit keys."""
    dev = require_gpu()
    stream = torch.cuda.Stream()
    steps = []
    with torch.cuda.stream(stream):
        for t in range(4):
            x = inputs.logits_normal(16, 32000, 4.0, torch.bfloat16, seed=40 + t, device=dev)
            ctx = inputs.uniform_tokens((16, 1), 32000, seed=50 + t, device=dev)
            steps.append((x, host_bits(x), ctx))
        stream.synchronize()
        for t, (x, _, ctx) in enumerate(steps):
            sbw.sbw_bias_logits(x, ctx, 0xFEDCBA9876543211 + t, 0.25, 1.0, t % 2, stream=stream)
    stream.synchronize()
    for t, (x, before, ctx) in enumerate(steps):
        want = oracle.bias_logits(before, 32000, ctx.cpu().numpy(), 0xFEDCBA9876543211 + t, 0.25,
                                  1.0, t % 2, threads=8)
        assert_same_bits(host_bits(x), want)


def test_host_buffer_entry_point():
    dev = require_gpu()
    B, V = 8, 32000
    x = inputs.logits_normal(B, V, 4.0, torch.bfloat16, seed=60).pin_memory()
    ctx = inputs.uniform_tokens((B, 1), V, seed=61).pin_memory()
    before = host_bits(x)
    nbytes = sbw.sbw_bias_logits_host_staging_bytes(torch.bfloat16, B, V, 1)
    staging = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    sbw.sbw_bias_logits_host(x, ctx, KEY, 0.5, 2.0, sbw.SCHEME_CONTEXT, staging)
    torch.cuda.synchronize()
    want = oracle.bias_logits(before, V, ctx.numpy(), KEY, 0.5, 2.0, oracle.SCHEME_CONTEXT)
    assert_same_bits(host_bits(x), want)


def test_cuda_graph_replay_and_dependent_steps_keep_stream_order():
    """The launch configuration the benchmark times: decode steps captured in one CUDA graph and
    replayed.  The kernels use programmatic dependent launch, so this also checks that a step
    which depends on the previous one (same buffer, biased twice; context tokens produced by a
    kernel that runs just before) still sees its predecessor's writes."""
    dev = require_gpu()
    B, V, steps = 64, 128256, 6
    xs = [inputs.logits_normal(B, V, 4.0, torch.bfloat16, seed=1200 + t, device=dev) for t in range(steps)]
    ctxs = [inputs.uniform_tokens((B, 1), V, seed=1300 + t, device=dev) for t in range(steps)]
    before = [host_bits(x) for x in xs]
    same = inputs.logits_normal(B, V, 4.0, torch.float32, seed=1400, device=dev)
    same_before = host_bits(same)
    ctx_src = inputs.uniform_tokens((B, 1), V, seed=1401, device=dev)
    ctx_dst = torch.zeros_like(ctx_src)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for t in range(2):                       # warm-up outside capture (first-call set-up)
            sbw.sbw_bias_logits(torch.zeros((2, 64), dtype=torch.bfloat16, device=dev),
                                torch.zeros((2, 1), dtype=torch.int32, device=dev), KEY, 0.5, 2.0, t)
            sbw.sbw_bias_logits(torch.zeros((2, 64), dtype=torch.float32, device=dev),
                                torch.zeros((2, 1), dtype=torch.int32, device=dev), KEY, 0.5, 2.0, t)
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for t in range(steps):
                sbw.sbw_bias_logits(xs[t], ctxs[t], KEY, 0.5, 2.0, sbw.SCHEME_CONTEXT, stream=side)
            ctx_dst.copy_(ctx_src + 0)           # a torch kernel writes the context tokens ...
            for rep in range(3):                 # ... that three dependent in-place steps read
                sbw.sbw_bias_logits(same, ctx_dst, KEY, 0.25, 1.5, rep % 2, stream=side)
        graph.replay()
    side.synchronize()
    torch.cuda.synchronize()
    for t in range(steps):
        want = oracle.bias_logits(before[t], V, ctxs[t].cpu().numpy(), KEY, 0.5, 2.0, oracle.SCHEME_CONTEXT,
                                  threads=8)
        assert_same_bits(host_bits(xs[t]), want)
    want = same_before
    for rep in range(3):
        want = oracle.bias_logits(want, V, ctx_src.cpu().numpy(), KEY, 0.25, 1.5, rep % 2, threads=8)
    assert_same_bits(host_bits(same), want)
