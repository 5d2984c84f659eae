"""GPU parity of sbw_detect (membership per token, Eq. 5) against the CPU oracle: green counts
and T bit-exact, z within 1e-9 absolute in fp64."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_03844_b200 as sbw
from paper_2609_03844_b200 import inputs
from gpu_util import KEY, require_gpu

pytestmark = pytest.mark.gpu

SCHEMES = [sbw.SCHEME_CONTEXT, sbw.SCHEME_SELFSALT]


def _detect(tokens, lengths, key, gamma, scheme, W=1, with_offsets=False):
    dev = require_gpu()
    tok, lens = tokens.to(dev), lengths.to(dev)
    N = lens.numel()
    counts = torch.full((N,), -7, dtype=torch.int32, device=dev)
    T = torch.full((N,), -7, dtype=torch.int32, device=dev)
    z = torch.full((N,), 99.0, dtype=torch.float64, device=dev)
    offsets = ws = None
    if with_offsets:
        offsets = torch.zeros(N + 1, dtype=torch.int64, device=dev)
        offsets[1:] = torch.cumsum(lens.clamp(min=0).to(torch.int64), 0)
    else:
        ws = torch.empty(max(sbw.sbw_detect_workspace_bytes(N), 1), dtype=torch.uint8, device=dev)
    sbw.sbw_detect(tok, lens, key, gamma, scheme, counts, z, out_T=T, offsets=offsets, workspace=ws,
                   ctx_width=W)
    torch.cuda.synchronize()
    return counts.cpu().numpy(), T.cpu().numpy(), z.cpu().numpy()


def _compare(tokens, lengths, key, gamma, scheme, W=1, with_offsets=False):
    c, T, z = _detect(tokens, lengths, key, gamma, scheme, W, with_offsets)
    oc, oT, oz = oracle.detect(tokens.numpy(), lengths.numpy(), key, gamma, scheme, ctx_width=W, threads=8)
    assert np.array_equal(c, oc)
    assert np.array_equal(T, oT)
    assert np.max(np.abs(z - oz), initial=0.0) <= 1e-9
    return c, T, z


def test_config1_one_sequence_of_200():
    tokens = inputs.uniform_tokens((200,), 32000, seed=70)
    lengths = torch.tensor([200], dtype=torch.int32)
    for scheme in SCHEMES:
        c, T, z = _compare(tokens, lengths, KEY, 0.25, scheme)
        assert T[0] == 199


@pytest.mark.parametrize("scheme", SCHEMES)
@pytest.mark.parametrize("W", [1, 4])
@pytest.mark.parametrize("with_offsets", [False, True])
def test_ragged_batch_with_empty_and_short_sequences(scheme, W, with_offsets):
    """Lengths 0..300 (some shorter than the context width, several warp trips, ragged tails);
    more sequences than one scan tile."""
    tokens, lengths = inputs.null_token_streams(3000, 0, 300, 128256, seed=71)
    lengths[:8] = torch.tensor([0, 1, 2, 3, 4, 5, 64, 65], dtype=torch.int32)
    tokens = inputs.uniform_tokens((int(lengths.sum()),), 128256, seed=72)
    _compare(tokens, lengths, KEY, 0.25, scheme, W=W, with_offsets=with_offsets)


def test_single_long_sequence_and_arbitrary_ids():
    """One 100k-token sequence; ids are arbitrary 32-bit patterns, negatives included."""
    g = torch.Generator().manual_seed(73)
    tokens = torch.randint(-2**31, 2**31 - 1, (100000,), generator=g, dtype=torch.int64).to(torch.int32)
    lengths = torch.tensor([100000], dtype=torch.int32)
    for scheme in SCHEMES:
        _compare(tokens, lengths, 0xFEDCBA9876543211, 0.5, scheme)


def test_sequences_past_the_end_of_the_buffer_are_clipped():
    """total_tokens bounds every read: a length that overruns the buffer is scored up to it."""
    dev = require_gpu()
    tokens = inputs.uniform_tokens((150,), 32000, seed=74)
    lengths = torch.tensor([100, 100, 100], dtype=torch.int32)       # claims 300 > 150
    c, T, z = _detect(tokens, lengths, KEY, 0.25, sbw.SCHEME_CONTEXT)
    oc, oT, oz = oracle.detect(tokens.numpy(), np.array([100, 50, 0], dtype=np.int32), KEY, 0.25, 0)
    assert np.array_equal(c, oc) and np.array_equal(T, oT) and np.allclose(z, oz, atol=1e-9)
    del dev


@pytest.mark.parametrize("scheme", SCHEMES)
def test_config5_null_half_full_size(scheme):
    """100000 sequences, lengths uniform in [64, 1024], V=128256, uniform ids: all counts and z."""
    dev = require_gpu()
    tokens, lengths = inputs.null_token_streams(100000, 64, 1024, 128256, seed=75, device=dev)
    c, T, z = _compare(tokens.cpu(), lengths.cpu(), KEY, 0.25, scheme)
    assert abs(z.mean()) < 0.02 and abs(z.var() - 1.0) < 0.03          # null law of Eq. 5


@pytest.mark.parametrize("N", [1, 3, 64, 296, 297, 592, 593, 1184, 1185])
def test_few_sequences_take_a_cta_each(N):
    """Below a few thousand sequences a CTA (32, 16 or 8 warps) scores each sequence, its warps taking the
    128-token trips in turn; the batch sizes sit on both sides of every switch.  Lengths from 0 to beyond
    many trips, ragged tails, both schemes, widths 1 and 3."""
    tokens, lengths = inputs.null_token_streams(N, 0, 9000 if N <= 64 else 1500, 128256, seed=75 + N)
    lengths[0] = 0 if N > 1 else 7777
    tokens = inputs.uniform_tokens((int(lengths.sum()),), 128256, seed=76)
    for scheme, W in ((sbw.SCHEME_CONTEXT, 1), (sbw.SCHEME_SELFSALT, 3)):
        _compare(tokens, lengths, KEY, 0.25, scheme, W=W)
