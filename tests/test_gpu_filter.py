"""GPU parity of sbw_bias_sample_filtered against the oracle: sampled ids and kept counts
bit-exact (the truncation is integer arithmetic on both sides)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_03844_b200 as sbw
from paper_2609_03844_b200 import inputs
from gpu_util import KEY, require_gpu

pytestmark = pytest.mark.gpu


def _run(x, ctx, scheme, tau, top_k, top_p, step, gamma=0.25, delta=2.0, V=None, vocab_offset=0):
    dev = require_gpu()
    xd, cd = x.to(dev), ctx.to(dev)
    B = x.shape[0]
    V = V or x.shape[1]
    ws = torch.empty(max(sbw.sbw_sample_filtered_workspace_bytes(x.dtype, B, V), 256), dtype=torch.uint8, device=dev)
    ids = torch.full((B,), -9, dtype=torch.int32, device=dev)
    kept = torch.full((B,), -9, dtype=torch.int32, device=dev)
    before = xd.clone()
    sbw.sbw_bias_sample_filtered(xd, cd, KEY, gamma, delta, scheme, tau, top_k, top_p, 0xC0FFEE, step, ids, ws,
                                 out_kept=kept, V=V, vocab_offset=vocab_offset)
    torch.cuda.synchronize()
    assert torch.equal(xd.view(torch.uint8), before.view(torch.uint8))       # the logits are an input
    return ids.cpu().numpy(), kept.cpu().numpy()


def _check(x, ctx, scheme, tau, top_k, top_p, step=0, gamma=0.25, delta=2.0, V=None, vocab_offset=0):
    ids, kept = _run(x, ctx, scheme, tau, top_k, top_p, step, gamma, delta, V, vocab_offset)
    V = V or x.shape[1]
    want = oracle.bias_sample_filtered(inputs.as_oracle_array(x), V, ctx.numpy(), KEY, gamma, delta, scheme, tau,
                                       top_k, top_p, 0xC0FFEE, step, vocab_offset=vocab_offset, threads=8)
    assert np.array_equal(kept, want["kept"]), (kept[:8], want["kept"][:8])
    assert np.array_equal(ids, want["tokens"])
    return kept


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("scheme", [sbw.SCHEME_CONTEXT, sbw.SCHEME_SELFSALT])
@pytest.mark.parametrize("top_k,top_p", [(0, 0.8), (50, 1.0), (300, 0.9), (0, 0.999), (0, 0.05), (5000, 0.95)])
def test_matches_oracle(dtype, scheme, top_k, top_p):
    B, V = 9, 20011
    x = inputs.logits_normal(B, V, 1.5, dtype, seed=41)
    ctx = inputs.uniform_tokens((B, 1), V, seed=42)
    for step in range(2):
        _check(x, ctx, scheme, 0.7, top_k, top_p, step)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_flat_rows_and_large_kept_sets(dtype):
    """Narrow logits: thousands of candidates stay, the boundary lies deep in the order."""
    B, V = 6, 50000
    x = inputs.logits_normal(B, V, 0.05, dtype, seed=51)
    ctx = inputs.uniform_tokens((B, 1), V, seed=52)
    kept = _check(x, ctx, sbw.SCHEME_CONTEXT, 1.0, 0, 0.8, delta=0.25)
    assert kept.min() > 5000
    _check(x, ctx, sbw.SCHEME_CONTEXT, 1.0, 30000, 0.5, delta=0.25)
    _check(x, ctx, sbw.SCHEME_CONTEXT, 1.0, 2500, 1.0, delta=0.25)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_ties(dtype):
    """Equal logits everywhere: every cut falls inside a group of ties and goes by column."""
    B, V = 5, 30000
    x = torch.zeros(B, V, dtype=dtype)
    x[1, ::3] = 1.0
    x[2, 100:20000] = 2.0
    x[3] = torch.round(inputs.logits_normal(1, V, 2.0, torch.float32, seed=5)[0]).to(dtype)
    x[4, 7] = 30.0
    ctx = inputs.uniform_tokens((B, 1), V, seed=62)
    for top_k, top_p in ((0, 0.5), (0, 0.9), (2500, 1.0), (12345, 1.0), (12345, 0.3), (1, 1.0), (0, 1e-9)):
        _check(x, ctx, sbw.SCHEME_SELFSALT, 0.7, top_k, top_p, delta=0.0)
        _check(x, ctx, sbw.SCHEME_SELFSALT, 0.7, top_k, top_p, delta=1.0)


def test_filters_off_equals_the_plain_sampler():
    dev = require_gpu()
    B, V = 7, 128256
    x = inputs.logits_normal(B, V, 4.0, torch.bfloat16, seed=71).to(dev)
    ctx = inputs.uniform_tokens((B, 1), V, seed=72).to(dev)
    ws = torch.empty(sbw.sbw_sample_filtered_workspace_bytes(x.dtype, B, V), dtype=torch.uint8, device=dev)
    ws2 = torch.empty(sbw.sbw_sample_workspace_bytes(B, V), dtype=torch.uint8, device=dev)
    a = torch.empty(B, dtype=torch.int32, device=dev)
    b = torch.empty(B, dtype=torch.int32, device=dev)
    kept = torch.empty(B, dtype=torch.int32, device=dev)
    for step in range(3):
        sbw.sbw_bias_sample_filtered(x, ctx, KEY, 0.25, 2.0, 1, 0.7, 0, 1.0, 5, step, a, ws, out_kept=kept)
        sbw.sbw_bias_sample(x, ctx, KEY, 0.25, 2.0, 1, 0.7, 5, step, b, ws2)
        torch.cuda.synchronize()
        assert torch.equal(a, b) and (kept == V).all()


def test_ragged_shapes_strides_and_offsets():
    B, V, ld = 3, 4099, 4200
    x = inputs.logits_normal(B, ld, 2.0, torch.float32, seed=81)
    ctx = inputs.uniform_tokens((B, 4), 100000, seed=82)
    _check(x, ctx, sbw.SCHEME_SELFSALT, 0.9, 40, 0.8, V=V, vocab_offset=50000)
    xb = inputs.logits_normal(B, ld, 2.0, torch.bfloat16, seed=83)
    _check(xb, ctx, sbw.SCHEME_CONTEXT, 0.9, 0, 0.8, V=V, vocab_offset=50000)
    one = inputs.logits_normal(2, 1, 2.0, torch.float32, seed=84)
    _check(one, ctx[:2], sbw.SCHEME_CONTEXT, 0.9, 0, 0.8)


def test_full_size_rows_on_sampled_rows():
    """The benchmark's shape: B = 64, V = 128256, bf16, temperature 0.7, top_p 0.8."""
    B, V = 64, 128256
    x = inputs.logits_normal(B, V, 4.0, torch.bfloat16, seed=91)
    ctx = inputs.uniform_tokens((B, 1), V, seed=92)
    ids, kept = _run(x, ctx, sbw.SCHEME_CONTEXT, 0.7, 0, 0.8, 3)
    rows = [0, 17, 63]
    want = oracle.bias_sample_filtered(inputs.as_oracle_array(x[rows]), V, ctx[rows].numpy(), KEY, 0.25, 2.0, 0, 0.7,
                                       0, 0.8, 0xC0FFEE, 3, threads=3)
    # the oracle numbers rows from 0: compare the kept counts (row-independent) and, for row 0, the id
    assert np.array_equal(kept[rows], want["kept"]) and ids[0] == want["tokens"][0]


def test_argument_checks():
    dev = require_gpu()
    x = torch.zeros(2, 64, device=dev)
    ctx = torch.zeros(2, 1, dtype=torch.int32, device=dev)
    ids = torch.empty(2, dtype=torch.int32, device=dev)
    ws = torch.empty(4096, dtype=torch.uint8, device=dev)
    for kw in (dict(top_p=0.0), dict(top_p=float("nan")), dict(top_k=-1), dict(temperature=0.0)):
        args = dict(temperature=0.7, top_k=0, top_p=0.8)
        args.update(kw)
        with pytest.raises(sbw.SbwError) as e:
            sbw.sbw_bias_sample_filtered(x, ctx, KEY, 0.25, 2.0, 0, args["temperature"], args["top_k"], args["top_p"],
                                         1, 0, ids, ws)
        assert e.value.code == -1
    with pytest.raises(sbw.SbwError) as e:
        sbw.sbw_bias_sample_filtered(x, ctx, KEY, 0.25, 2.0, 0, 0.7, 0, 0.8, 1, 0, ids, ws[:16])
    assert e.value.code == -3


@pytest.mark.parametrize("B", [37, 38, 74, 75, 148, 149, 300])
def test_every_cluster_size(B):
    """Small batches split a row over 8, 4 or 2 CTAs; larger ones take one CTA per row."""
    V = 6007
    x = inputs.logits_normal(B, V, 1.5, torch.bfloat16, seed=300 + B)
    x[1] = 0.0                                                  # a flat row: the list overflows, radix path
    x[2, :3000] = 3.0                                           # a big group of ties at the top
    ctx = inputs.uniform_tokens((B, 1), V, seed=400 + B)
    _check(x, ctx, sbw.SCHEME_CONTEXT, 0.7, 0, 0.8)
    _check(x, ctx, sbw.SCHEME_SELFSALT, 0.7, 40, 0.9)
    _check(x, ctx, sbw.SCHEME_CONTEXT, 1.0, 700, 1.0)
    _check(x.float(), ctx, sbw.SCHEME_CONTEXT, 0.7, 0, 0.97)


@pytest.mark.parametrize("dtype,base", [(torch.bfloat16, 256.0), (torch.float32, 16777216.0)])
@pytest.mark.parametrize("delta", [1.0, 2.0, 3.0, -1.0])
def test_rounding_of_the_biased_sum_at_the_cut(dtype, base, delta):
    """Logits around a power of two where the spacing of the type doubles: l + delta rounds (ties to
    even), biased values collapse onto each other, and the k-th largest biased logit is reached by
    columns whose exact sum lies below it.  The candidate threshold has to keep all of them."""
    B, V = 6, 9000
    rng = np.random.default_rng(int(base) % 97 + int(delta * 4) + 20)
    step = base / 256.0                                        # spacing below `base`
    grid = base + step * rng.integers(-40, 12, size=(B, V))    # above `base` every other value is not representable
    x = torch.from_numpy(grid).to(dtype)
    x[:, ::7] = x[:, ::7] - 50 * step                          # a bulk below the interesting range
    # rows 3..5: only some 600 columns stay near the top, so that the candidates fit the list
    sparse = torch.from_numpy(rng.random((3, V)) < 0.93)
    x[3:][sparse] = x[3:][sparse] - 1000 * step
    ctx = inputs.uniform_tokens((B, 1), V, seed=3)
    for top_k in (5, 50, 300):
        _check(x, ctx, sbw.SCHEME_CONTEXT, 1.0, top_k, 1.0, delta=delta * step, gamma=0.5)
        _check(x, ctx, sbw.SCHEME_SELFSALT, 1.0, top_k, 0.7, delta=delta * step, gamma=0.5)


@pytest.mark.parametrize("B", [6, 300])
def test_bf16_weight_table_windows(B):
    """bf16 top-p totals come from a per-row table over two windows of codes (below the maximum, above the
    lowest weighted code) with everything else evaluated directly: rows whose logits are all negative, all tiny,
    spread over many binades, subnormal, or concentrated on a few codes must still give the oracle's kept sets."""
    V = 12000
    x = inputs.logits_normal(B, V, 4.0, torch.bfloat16, seed=130 + B)
    x[0] = x[0] - 40.0                                   # every logit negative: the maximum is a negative code
    x[1] = x[1] * 1e-20                                  # tiny magnitudes of both signs
    x[2] = torch.exp2(torch.linspace(-120.0, 4.0, V)).to(torch.bfloat16) * torch.sign(x[2].float()).to(torch.bfloat16)
    x[3] = x[3] * 1e-39                                  # subnormals and zeros of both signs
    x[4] = torch.round(x[4] / 4) * 4                     # a handful of distinct codes
    x[5, :] = -3.0
    x[5, ::7] = 2.5
    ctx = inputs.uniform_tokens((B, 1), V, seed=131)
    for tau, top_p, delta in ((0.7, 0.8, 2.0), (0.05, 0.99, 2.0), (3.0, 0.5, -1.0), (1.0, 0.9999, 0.25)):
        _check(x, ctx, sbw.SCHEME_CONTEXT, tau, 0, top_p, delta=delta)
