"""Pins for the oracle's per-token indicators and windowed detection: the indicators against the
counts of the plain detector and the big-integer restatement, the best window against numpy's
convolution, and Eq. 5 on the window against its closed form."""
import math

import numpy as np
import pytest

from oracle import py_ref
from paper_2609_03844_b200 import inputs

KEY = 0x5EED


@pytest.mark.parametrize("scheme_name", ["context", "selfsalt"])
@pytest.mark.parametrize("W", [1, 4])
def test_bits_sum_to_the_detector_counts_and_match_bigint(oracle, scheme_name, W):
    scheme = oracle.SCHEME_SELFSALT if scheme_name == "selfsalt" else oracle.SCHEME_CONTEXT
    tokens, lengths = inputs.null_token_streams(60, 0, 80, 32000, seed=90)
    tok, lens = tokens.numpy(), lengths.numpy()
    green = oracle.detect_bits(tok, lens, KEY, 0.25, scheme, ctx_width=W)
    counts, T, _ = oracle.detect(tok, lens, KEY, 0.25, scheme, ctx_width=W)
    off = np.concatenate([[0], np.cumsum(lens)])
    for s in range(len(lens)):
        seg = green[off[s]:off[s + 1]]
        assert seg.sum() == counts[s] and not seg[:W].any()
        if s < 8:
            thr = py_ref.threshold(0.25)
            seq = [int(t) for t in tok[off[s]:off[s + 1]]]
            for t in range(W, len(seq)):
                r = (py_ref.seed_selfsalt(KEY, seq[t - W:t], seq[t]) if scheme_name == "selfsalt"
                     else py_ref.seed_context(KEY, seq[t - W:t]))
                assert seg[t] == py_ref.green(r, seq[t], thr)


@pytest.mark.parametrize("window", [1, 5, 32, 33, 64, 500])
def test_best_window_matches_numpy_convolution(oracle, window):
    rng = np.random.default_rng(91 + window)
    lens = rng.integers(0, 200, size=80).astype(np.int32)
    lens[:4] = [0, 1, 2, window + 1]
    green = (rng.random(int(lens.sum())) < 0.3).astype(np.uint8)
    off = np.concatenate([[0], np.cumsum(lens)])
    for s in range(len(lens)):
        green[off[s]:off[s] + min(1, lens[s])] = 0               # unscored first token
    bc, bs, bz = oracle.window_z(green, lens, window, 0.25, ctx_width=1)
    for s in range(len(lens)):
        y = green[off[s] + min(1, lens[s]):off[s + 1]].astype(np.int64)
        T = len(y)
        w = min(window, T)
        if T == 0:
            assert (bc[s], bs[s], bz[s]) == (0, 0, 0.0)
            continue
        sums = np.convolve(y, np.ones(w, dtype=np.int64), mode="valid")
        assert bc[s] == sums.max() and bs[s] == int(np.argmax(sums))      # argmax: first maximum
        assert bz[s] == pytest.approx((sums.max() - 0.25 * w) / math.sqrt(w * 0.25 * 0.75), abs=1e-12)


def test_window_at_least_as_long_as_the_text_is_plain_detection(oracle):
    tokens, lengths = inputs.null_token_streams(40, 0, 120, 32000, seed=92)
    tok, lens = tokens.numpy(), lengths.numpy()
    green = oracle.detect_bits(tok, lens, KEY, 0.5, oracle.SCHEME_CONTEXT)
    counts, T, z = oracle.detect(tok, lens, KEY, 0.5, oracle.SCHEME_CONTEXT)
    bc, bs, bz = oracle.window_z(green, lens, 10 ** 6, 0.5)
    assert np.array_equal(bc, counts) and not bs.any() and np.array_equal(bz, z)
