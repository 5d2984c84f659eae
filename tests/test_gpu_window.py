"""GPU parity of sbw_detect_bits and sbw_window_z against the oracle: every stored green bit, and
the best window (count and start bit-exact, z within 1e-9)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_03844_b200 as sbw
from paper_2609_03844_b200 import inputs
from gpu_util import KEY, require_gpu

pytestmark = pytest.mark.gpu


def _run(tokens, lengths, scheme, W, window, gamma=0.25, given_offsets=False):
    dev = require_gpu()
    tok, lens = tokens.to(dev), lengths.to(dev)
    N, total = lens.numel(), tok.numel()
    words = sbw.sbw_detect_bits_words(N, total)
    bits = torch.full((words,), 0x5A5A5A5A, dtype=torch.int32, device=dev)
    counts = torch.empty(N, dtype=torch.int32, device=dev)
    z = torch.empty(N, dtype=torch.float64, device=dev)
    ws = torch.empty(max(sbw.sbw_detect_workspace_bytes(N), 8), dtype=torch.uint8, device=dev)
    offsets = None
    if given_offsets:
        offsets = torch.zeros(N + 1, dtype=torch.int64, device=dev)
        offsets[1:] = torch.cumsum(lens.clamp(min=0).to(torch.int64), 0)
    sbw.sbw_detect_bits(tok, lens, KEY, gamma, scheme, counts, z, bits, offsets=offsets, workspace=ws, ctx_width=W)
    # when the library scanned the lengths itself, the offsets are at the start of the workspace
    offs = offsets if given_offsets else ws[:8 * (N + 1)].view(torch.int64)
    scratch = torch.empty(words, dtype=torch.int32, device=dev)
    bc = torch.empty(N, dtype=torch.int32, device=dev)
    bs = torch.empty(N, dtype=torch.int32, device=dev)
    bz = torch.empty(N, dtype=torch.float64, device=dev)
    sbw.sbw_window_z(bits, lens, offs, total, window, gamma, scratch, bc, bs, bz, ctx_width=W)
    torch.cuda.synchronize()
    return (bits.cpu().numpy().view(np.uint32), counts.cpu().numpy(), z.cpu().numpy(), bc.cpu().numpy(),
            bs.cpu().numpy(), bz.cpu().numpy())


def _check(tokens, lengths, scheme, W, window, **kw):
    bits, counts, z, bc, bs, bz = _run(tokens, lengths, scheme, W, window, **kw)
    tok, lens = tokens.numpy(), lengths.numpy()
    green = oracle.detect_bits(tok, lens, KEY, 0.25, scheme, ctx_width=W)
    oc, _, oz = oracle.detect(tok, lens, KEY, 0.25, scheme, ctx_width=W)
    assert np.array_equal(counts, oc) and np.max(np.abs(z - oz), initial=0) <= 1e-9
    off = np.concatenate([[0], np.cumsum(np.maximum(lens, 0))])
    for s in range(len(lens)):
        L = max(int(lens[s]), 0)
        y = green[off[s] + min(W, L):off[s + 1]]
        T = len(y)
        nwords = (T + 31) // 32
        start = (off[s] >> 5) + 2 * s
        want = np.zeros(nwords * 32, dtype=np.uint8)
        want[:T] = y
        packed = np.packbits(want.reshape(-1, 32)[:, ::-1], axis=1).view(">u4").astype(np.uint32).ravel() \
            if nwords else np.zeros(0, dtype=np.uint32)
        assert np.array_equal(bits[start:start + nwords], packed), s
    wc, wst, wz = oracle.window_z(green, lens, window, 0.25, ctx_width=W)
    assert np.array_equal(bc, wc) and np.array_equal(bs, wst)
    assert np.max(np.abs(bz - wz), initial=0) <= 1e-9


@pytest.mark.parametrize("scheme", [sbw.SCHEME_CONTEXT, sbw.SCHEME_SELFSALT])
@pytest.mark.parametrize("W", [1, 4])
@pytest.mark.parametrize("window", [1, 32, 50, 200])
def test_bits_and_best_window_on_a_ragged_batch(scheme, W, window):
    tokens, lengths = inputs.null_token_streams(700, 0, 400, 128256, seed=2000)
    lengths[:10] = torch.tensor([0, 1, 2, 4, 5, 33, 34, 64, 65, 129], dtype=torch.int32)
    tokens = inputs.uniform_tokens((int(lengths.sum()),), 128256, seed=2001)
    _check(tokens, lengths, scheme, W, window, given_offsets=(window == 50))


def test_partly_watermarked_text_is_found_by_its_window():
    """A null stream with a 100-token stretch written under the watermark (every token chosen
    green under the context scheme): the whole-text z is diluted, the 100-token window is not."""
    rng = np.random.default_rng(7)
    V, L = 32000, 900
    seq = rng.integers(0, V, size=L).astype(np.int32)
    thr = oracle.threshold(0.25)
    for t in range(400, 500):
        r = oracle.seed_context(KEY, [int(seq[t - 1])])
        v = int(rng.integers(0, V))
        while not oracle.green(r, v, thr):
            v = int(rng.integers(0, V))
        seq[t] = v
    tokens = torch.from_numpy(seq)
    lengths = torch.tensor([L], dtype=torch.int32)
    _check(tokens, lengths, sbw.SCHEME_CONTEXT, 1, 100)
    bits, counts, z, bc, bs, bz = _run(tokens, lengths, sbw.SCHEME_CONTEXT, 1, 100)
    assert bc[0] >= 100 and 390 <= bs[0] <= 400 and bz[0] > 15 and z[0] < bz[0]
