"""GPU parity of sbw_bias_logits_topk (the paper's SBW-ss: only the top-k candidates of a row are
tested and biased) against the CPU oracle: every bit of the row."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_03844_b200 as sbw
from paper_2609_03844_b200 import inputs
from gpu_util import KEY, assert_same_bits, host_bits, require_gpu

pytestmark = pytest.mark.gpu
SCHEMES = [sbw.SCHEME_CONTEXT, sbw.SCHEME_SELFSALT]


def _check(x, V, ctx, key, gamma, delta, scheme, k, off=0, view=None, nan_payload=False):
    dev = require_gpu()
    x_dev = x.to(dev)
    target = x_dev if view is None else view(x_dev)
    src = x if view is None else view(x).contiguous()
    sbw.sbw_bias_logits_topk(target, ctx.to(dev), key, gamma, delta, scheme, k, V=V, vocab_offset=off)
    torch.cuda.synchronize()
    want, sel = oracle.bias_logits_topk(host_bits(src), V, ctx.numpy(), key, gamma, delta, scheme, k,
                                        vocab_offset=off)
    got = host_bits(target.contiguous()) if view is not None else host_bits(x_dev)
    assert_same_bits(got, want, allow_nan_payload=nan_payload)
    return got, sel


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("scheme", SCHEMES)
def test_top40_on_full_vocabulary_rows(dtype, scheme):
    """V=151936 (fp32) / 128256 (bf16, many tied values near the top), context width 4, k = 40."""
    V = 151936 if dtype == torch.float32 else 128256
    x = inputs.logits_normal(48, V, 4.0, dtype, seed=70)
    inputs.add_zipf_spike_(x, V, seed=71)
    ctx = inputs.uniform_tokens((48, 4), V, seed=72)
    got, sel = _check(x, V, ctx, KEY, 0.25, 2.0, scheme, 40)
    changed = (got != host_bits(x)).sum(axis=1)
    assert np.all(changed <= 40) and 100 < changed.sum() < 48 * 25      # about gamma * 40 per row


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("k", [1, 7, 40, 128, 129, 300])
def test_various_k_ragged_rows_offset_and_unaligned(dtype, k):
    B, V = 5, 10007
    x = inputs.logits_normal(B, V + 9, 4.0, dtype, seed=73)
    ctx = inputs.uniform_tokens((B, 1), 50000, seed=74)
    _check(x, V, ctx, KEY, 0.5, 2.0, sbw.SCHEME_SELFSALT, k, off=1234)                       # padded rows
    _check(x, V, ctx, KEY, 0.5, -1.5, sbw.SCHEME_SELFSALT, k, view=lambda t: t[:, 1:V + 1])  # unaligned


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_degenerate_rows_take_the_exact_fallback(dtype):
    """Constant rows, two-valued rows, masked rows (-inf), zeros of both signs, NaNs: ties decide."""
    V = 3000
    x = inputs.logits_normal(8, V, 4.0, dtype, seed=75)
    x[0, :] = 1.25
    x[1, :] = float("-inf")
    x[1, 17] = 0.5
    x[2, ::2] = 3.0
    x[2, 1::2] = -3.0
    x[3, :] = 0.0
    x[3, 5::7] = -0.0
    x[4, 100:2900] = float("-inf")
    x[5, 10] = float("nan")
    x[5, 20] = float("inf")
    x[6, :50] = 9.0
    ctx = inputs.uniform_tokens((8, 1), V, seed=76)
    for k in (1, 40, 200):
        for delta in (2.0, -2.0):
            _check(x, V, ctx, KEY, 0.5, delta, sbw.SCHEME_SELFSALT, k)


def test_k_at_least_v_is_the_full_vocabulary_scheme_and_small_vocabularies():
    dev = require_gpu()
    for V in (1, 3, 8, 33):
        x = inputs.logits_normal(4, V, 4.0, torch.float32, seed=77 + V)
        ctx = inputs.uniform_tokens((4, 1), 1000, seed=78)
        for k in (1, 2, V, V + 10):
            _check(x, V, ctx, KEY, 0.5, 1.0, sbw.SCHEME_SELFSALT, k)
    x = inputs.logits_normal(3, 4096, 4.0, torch.bfloat16, seed=79)
    ctx = inputs.uniform_tokens((3, 1), 4096, seed=80)
    a = x.to(dev)
    b = x.to(dev)
    sbw.sbw_bias_logits_topk(a, ctx.to(dev), KEY, 0.25, 2.0, 1, 5000)
    sbw.sbw_bias_logits(b, ctx.to(dev), KEY, 0.25, 2.0, 1)
    torch.cuda.synchronize()
    assert host_bits(a).tobytes() == host_bits(b).tobytes()
    L = sbw.lib()
    assert L.sbw_bias_logits_topk(a.data_ptr(), 1, 3, 4096, 4096, 0, ctx.to(dev).data_ptr(), 1, KEY, 0.25, 2.0, 1,
                                  0, None) == -1


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("k", [40, 128, 200])
def test_batches_larger_than_the_sm_count(dtype, k):
    """More rows than SMs selects the 512-thread kernel (k <= 128) -- same results, incl. ties."""
    B, V = 200, 20011
    x = inputs.logits_normal(B, V, 4.0, dtype, seed=81)
    x[3, :] = 2.5
    x[7, 1000:] = float("-inf")
    ctx = inputs.uniform_tokens((B, 4), V, seed=82)
    _check(x, V, ctx, KEY, 0.25, 2.0, sbw.SCHEME_SELFSALT, k)


@pytest.mark.parametrize("B", [1, 37, 38, 74, 75, 148, 149])
def test_every_cluster_size(B):
    """Small batches give a row to a cluster of 8, 4 or 2 CTAs; ties, flat rows and a ragged tail included."""
    V = 20011
    x = inputs.logits_normal(B, V, 4.0, torch.float32, seed=90 + B)
    x[0, :] = 1.25
    if B > 2:
        x[2, 5000:15000] = 9.0
    ctx = inputs.uniform_tokens((B, 1), V, seed=91)
    _check(x, V, ctx, KEY, 0.25, 2.0, sbw.SCHEME_SELFSALT, 40)
    _check(x.to(torch.bfloat16), V, ctx, KEY, 0.25, 2.0, sbw.SCHEME_CONTEXT, 128)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B,V,ld", [(149, 20011, 20016), (300, 4096, 4096), (700, 8192, 8200), (297, 65539, 65544),
                                    (310, 36869, 36872)])
def test_large_batches_of_aligned_rows(dtype, B, V, ld):
    """More rows than SMs with 16-byte aligned rows (the vector-wise passes): ragged ends (a tail shorter
    than 16 bytes), widths that are exact multiples of the per-trip columns, several rows per CTA,
    degenerate rows that take the fallback, the largest logit in the ragged tail."""
    x = inputs.logits_normal(B, ld, 4.0, dtype, seed=95 + B)
    x[3, :] = 2.5
    x[7, 1000:] = float("-inf")
    x[B - 1, ::3] = 7.0
    x[B - 2, V - 1] = 50.0                    # the largest logit in the ragged tail
    ctx = inputs.uniform_tokens((B, 2), V, seed=96)
    for k, scheme in ((40, sbw.SCHEME_SELFSALT), (128, sbw.SCHEME_CONTEXT), (1, sbw.SCHEME_SELFSALT)):
        _check(x, V, ctx, KEY, 0.25, 2.0, scheme, k, view=lambda t: t[:, :V])


def test_large_batches_of_full_vocabulary_rows():
    """The headline shapes of the scheme, 256 and 400 rows: V = 151936 fp32 and 128256 bf16."""
    for dtype, V, B in ((torch.float32, 151936, 256), (torch.bfloat16, 128256, 400)):
        x = inputs.logits_normal(B, V, 4.0, dtype, seed=97)
        inputs.add_zipf_spike_(x, V, seed=98)
        ctx = inputs.uniform_tokens((B, 1), V, seed=99)
        _check(x, V, ctx, KEY, 0.25, 4.0, sbw.SCHEME_SELFSALT, 40)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B", [9, 150])
def test_special_values_in_the_vector_passes(dtype, B):
    """NaNs of both signs, infinities, zeros of both signs, subnormals and huge values scattered over aligned
    rows (a cluster per row at B = 9, one CTA per row at B = 150): the order codes of whole vectors must
    rank them like the oracle's total order on bit patterns."""
    V = 8192
    x = inputs.logits_normal(B, V, 4.0, dtype, seed=120 + B)
    specials = torch.tensor([float("nan"), -float("nan"), float("inf"), float("-inf"), 0.0, -0.0, 1e-40, -1e-40,
                             3e38, -3e38], dtype=torch.float32).to(dtype)
    g = torch.Generator().manual_seed(121)
    rows = torch.randint(0, B, (400,), generator=g)
    cols = torch.randint(0, V, (400,), generator=g)
    x[rows, cols] = specials[torch.randint(0, len(specials), (400,), generator=g)]
    ctx = inputs.uniform_tokens((B, 1), V, seed=122)
    for k, delta in ((40, 2.0), (128, -1.0), (3, 8.0)):
        _check(x, V, ctx, KEY, 0.5, delta, sbw.SCHEME_SELFSALT, k, nan_payload=True)
