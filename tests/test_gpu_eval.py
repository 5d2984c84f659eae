"""GPU parity of the evaluation steps around detection -- distinct-tuple scoring, truncated text,
ROC-AUC -- against the oracle: integer results bit-exact, z within 1e-9, AUC bit-exact (it is one
division of exact integers on both sides)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_03844_b200 as sbw
from paper_2609_03844_b200 import inputs
from gpu_util import KEY, require_gpu

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------ distinct tuples ----
def _unique(tok, lens, scheme, W, max_length, gamma=0.25):
    dev = require_gpu()
    t, l = torch.as_tensor(tok, dtype=torch.int32).to(dev), torch.as_tensor(lens, dtype=torch.int32).to(dev)
    N = l.numel()
    ws = torch.empty(max(sbw.sbw_detect_unique_workspace_bytes(N, t.numel(), max_length), 256),
                     dtype=torch.uint8, device=dev)
    counts = torch.full((N,), -7, dtype=torch.int32, device=dev)
    T = torch.full((N,), -7, dtype=torch.int32, device=dev)
    z = torch.full((N,), 99.0, dtype=torch.float64, device=dev)
    sbw.sbw_detect_unique(t, l, max_length, KEY, gamma, scheme, counts, z, ws, out_T=T, ctx_width=W)
    torch.cuda.synchronize()
    return counts.cpu().numpy(), T.cpu().numpy(), z.cpu().numpy()


def _check_unique(tok, lens, scheme, W, max_length=None):
    tok, lens = np.asarray(tok, dtype=np.int32), np.asarray(lens, dtype=np.int32)
    if max_length is None:
        max_length = int(max(lens.max(initial=0), 0))
    c, T, z = _unique(tok, lens, scheme, W, max_length)
    oc, oT, oz = oracle.detect_unique(tok, lens, KEY, 0.25, scheme, ctx_width=W, threads=8)
    assert np.array_equal(c, oc) and np.array_equal(T, oT)
    assert np.max(np.abs(z - oz), initial=0) <= 1e-9


@pytest.mark.parametrize("scheme", [sbw.SCHEME_CONTEXT, sbw.SCHEME_SELFSALT])
@pytest.mark.parametrize("W", [1, 3, 4])
def test_repetitive_text(scheme, W):
    rng = np.random.default_rng(100 + W)
    lens = rng.integers(0, 700, size=300).astype(np.int32)
    lens[:4] = [0, W, W + 1, 1]
    # small alphabets of different sizes: from almost no distinct tuples to almost all distinct
    parts = [rng.integers(0, int(a), size=int(n)) for n, a in zip(lens, rng.choice([2, 5, 40, 3000], size=300))]
    _check_unique(np.concatenate(parts), lens, scheme, W)


@pytest.mark.parametrize("scheme", [sbw.SCHEME_CONTEXT, sbw.SCHEME_SELFSALT])
def test_without_repeats_it_is_the_plain_detector(scheme):
    dev = require_gpu()
    tok, lens = inputs.null_token_streams(500, 64, 1024, 128256, seed=5)
    c, T, z = _unique(tok.numpy(), lens.numpy(), scheme, 1, 1024)
    oc, oT, oz = oracle.detect_unique(tok.numpy(), lens.numpy(), KEY, 0.25, scheme, threads=8)
    assert np.array_equal(c, oc) and np.array_equal(T, oT) and np.max(np.abs(z - oz)) <= 1e-9
    pc, pT, _ = oracle.detect(tok.numpy(), lens.numpy(), KEY, 0.25, scheme, threads=8)
    assert (oT <= pT).all() and (pT - oT).sum() < 0.01 * pT.sum()      # uniform ids over 128K: hardly any repeat


@pytest.mark.parametrize("W", [1, 4])
def test_long_sequences_use_the_workspace_table(W):
    rng = np.random.default_rng(7)
    lens = np.array([1536 + W, 1537 + W, 5000, 300, 9000, 0, 2049], dtype=np.int32)
    parts = [rng.integers(0, a, size=int(n)) for n, a in zip(lens, [50, 50, 30, 10, 100000, 5, 70])]
    _check_unique(np.concatenate(parts), lens, sbw.SCHEME_SELFSALT, W)


def test_sequence_longer_than_declared_is_flagged_not_scored():
    rng = np.random.default_rng(8)
    lens = np.array([100, 4000, 200], dtype=np.int32)
    tok = rng.integers(0, 20, size=int(lens.sum())).astype(np.int32)
    c, T, z = _unique(tok, lens, sbw.SCHEME_CONTEXT, 1, max_length=1000)     # a lie about sequence 1
    oc, oT, oz = oracle.detect_unique(tok, lens, KEY, 0.25, 0)
    assert (c[1], T[1]) == (-1, -1) and np.isnan(z[1])
    assert (c[0], T[0], c[2], T[2]) == (oc[0], oT[0], oc[2], oT[2])


def test_unique_workspace_is_checked():
    dev = require_gpu()
    t = torch.zeros(100, dtype=torch.int32, device=dev)
    l = torch.full((2,), 50, dtype=torch.int32, device=dev)
    c = torch.empty(2, dtype=torch.int32, device=dev)
    z = torch.empty(2, dtype=torch.float64, device=dev)
    with pytest.raises(sbw.SbwError) as e:
        sbw.sbw_detect_unique(t, l, 50, KEY, 0.25, 0, c, z, torch.empty(8, dtype=torch.uint8, device=dev))
    assert e.value.code == -3
    assert sbw.sbw_detect_unique_workspace_bytes(2, 100, 5000) >= 16 * 100


# ------------------------------------------------------------------ truncated text ----
@pytest.mark.parametrize("W", [1, 4])
def test_prefix_z(W):
    dev = require_gpu()
    rng = np.random.default_rng(31)
    lens = rng.integers(0, 900, size=400).astype(np.int32)
    tok = rng.integers(0, 128256, size=int(lens.sum())).astype(np.int32)
    keep = rng.integers(-5, 1000, size=400).astype(np.int32)
    keep[:6] = [0, 1, W, W + 1, 33 + W, 32 + W]
    t, l, k = (torch.from_numpy(a).to(dev) for a in (tok, lens, keep))
    N, total = l.numel(), t.numel()
    bits = torch.zeros(sbw.sbw_detect_bits_words(N, total), dtype=torch.int32, device=dev)
    counts = torch.empty(N, dtype=torch.int32, device=dev)
    z = torch.empty(N, dtype=torch.float64, device=dev)
    ws = torch.empty(sbw.sbw_detect_workspace_bytes(N), dtype=torch.uint8, device=dev)
    sbw.sbw_detect_bits(t, l, KEY, 0.25, sbw.SCHEME_SELFSALT, counts, z, bits, workspace=ws, ctx_width=W)
    offs = ws[:8 * (N + 1)].view(torch.int64)
    pc = torch.empty(N, dtype=torch.int32, device=dev)
    pT = torch.empty(N, dtype=torch.int32, device=dev)
    pz = torch.empty(N, dtype=torch.float64, device=dev)
    sbw.sbw_prefix_z(bits, l, offs, k, total, 0.25, pc, pz, out_T=pT, ctx_width=W)
    torch.cuda.synchronize()
    green = oracle.detect_bits(tok, lens, KEY, 0.25, oracle.SCHEME_SELFSALT, ctx_width=W)
    oc, oT, oz = oracle.prefix_z(green, lens, keep, 0.25, ctx_width=W)
    assert np.array_equal(pc.cpu().numpy(), oc) and np.array_equal(pT.cpu().numpy(), oT)
    assert np.max(np.abs(pz.cpu().numpy() - oz)) <= 1e-9


# ------------------------------------------------------------------ ROC-AUC ----
def _auc(z, y):
    dev = require_gpu()
    zz = torch.as_tensor(np.asarray(z, dtype=np.float64)).to(dev)
    yy = torch.as_tensor(np.asarray(y, dtype=np.uint8)).to(dev)
    ws = torch.empty(sbw.sbw_roc_auc_workspace_bytes(zz.numel()), dtype=torch.uint8, device=dev)
    auc = torch.full((1,), 7.0, dtype=torch.float64, device=dev)
    stats = torch.full((4,), -1, dtype=torch.int64, device=dev)
    sbw.sbw_roc_auc(zz, yy, auc, ws, out_stats=stats)
    torch.cuda.synchronize()
    return float(auc.cpu()[0]), stats.cpu().numpy().astype(np.uint64)


@pytest.mark.parametrize("n", [1, 2, 33, 1024, 1025, 5000, 40000])
def test_auc_matches_the_pair_count(n):
    rng = np.random.default_rng(n)
    y = (rng.random(n) < 0.45).astype(np.uint8)
    z = rng.normal(size=n) + 0.8 * y
    z[::5] = np.round(z[::5] * 2) / 2                    # ties
    z[::97] = np.nan
    z[1::89] = -0.0
    z[2::83] = 0.0
    a, st = _auc(z, y)
    oa, ost = oracle.roc_auc(z, y, threads=8)
    assert np.array_equal(st, ost)
    assert (np.isnan(a) and np.isnan(oa)) or a == oa


def test_auc_degenerate_inputs():
    assert np.isnan(_auc([], [])[0])
    assert np.isnan(_auc([1.0, 2.0], [1, 1])[0])
    assert np.isnan(_auc([np.nan, 2.0], [0, 1])[0])
    assert _auc([3, 4, 1, 2], [1, 1, 0, 0])[0] == 1.0
    assert _auc([1, 2, 3, 4], [1, 1, 0, 0])[0] == 0.0
    assert _auc([5, 5, 5], [1, 0, 0])[0] == 0.5
    assert _auc([0.0, -0.0], [1, 0])[0] == 0.5
    # very unbalanced classes: one tile of one class against many of the other
    z = np.linspace(-1, 1, 30001)
    y = np.zeros(30001, dtype=np.uint8)
    y[15000] = 1
    a, st = _auc(z, y)
    assert a == oracle.roc_auc(z, y, threads=8)[0] and st.tolist() == [15000, 0, 1, 30000]


def test_auc_of_detector_scores():
    """z from the detection kernel on null and on strongly watermarked streams, then their AUC."""
    dev = require_gpu()
    N, L, V = 600, 120, 128256
    lens = torch.full((N,), L, dtype=torch.int32)
    tok = inputs.uniform_tokens((N, L), V, seed=77).numpy().astype(np.int32).copy()
    # second half: every scored token replaced by a green one with probability 0.3
    thr = oracle.threshold(0.25)
    rng = np.random.default_rng(5)
    for s in range(N // 2, N):
        for t in range(1, L):
            if rng.random() < 0.3:
                v = int(tok[s, t])
                while not oracle.green(oracle.seed_context(KEY, [int(tok[s, t - 1])]), v, thr):
                    v = (v + 1) % V
                tok[s, t] = v
    flat = torch.from_numpy(tok.ravel()).to(dev)
    counts = torch.empty(N, dtype=torch.int32, device=dev)
    z = torch.empty(N, dtype=torch.float64, device=dev)
    ws = torch.empty(sbw.sbw_detect_workspace_bytes(N), dtype=torch.uint8, device=dev)
    sbw.sbw_detect(flat, lens.to(dev), KEY, 0.25, sbw.SCHEME_CONTEXT, counts, z, workspace=ws)
    y = torch.zeros(N, dtype=torch.uint8, device=dev)
    y[N // 2:] = 1
    auc = torch.empty(1, dtype=torch.float64, device=dev)
    ws2 = torch.empty(sbw.sbw_roc_auc_workspace_bytes(N), dtype=torch.uint8, device=dev)
    sbw.sbw_roc_auc(z, y, auc, ws2)
    torch.cuda.synchronize()
    _, _, oz = oracle.detect(tok.ravel(), lens.numpy(), KEY, 0.25, 0)
    assert np.max(np.abs(z.cpu().numpy() - oz)) <= 1e-9
    want = oracle.roc_auc(z.cpu().numpy(), y.cpu().numpy())[0]
    assert float(auc.cpu()[0]) == want and want > 0.95
    assert abs(want - oracle.roc_auc(oz, y.cpu().numpy())[0]) < 1e-6


def test_batched_auc_equals_one_call_per_slice():
    """Table-4 shape: one AUC per configuration, 500 + 500 scores each, plus ragged and empty slices."""
    dev = require_gpu()
    rng = np.random.default_rng(55)
    sizes = [1000] * 16 + [0, 1, 2, 2047, 2048, 2049, 5000, 12000]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    n = int(off[-1])
    y = (rng.random(n) < 0.5).astype(np.uint8)
    z = rng.normal(size=n) + 1.1 * y
    z[::11] = np.round(z[::11])
    z[::501] = np.nan
    y[off[20]:off[21]] = 1                                     # a slice with one class only
    M = len(sizes)
    auc = torch.full((M,), 7.0, dtype=torch.float64, device=dev)
    stats = torch.full((4 * M,), -1, dtype=torch.int64, device=dev)
    sbw.sbw_roc_auc_batched(torch.from_numpy(z).to(dev), torch.from_numpy(y).to(dev), torch.from_numpy(off).to(dev),
                            auc, out_stats=stats)
    torch.cuda.synchronize()
    got, gst = auc.cpu().numpy(), stats.cpu().numpy().astype(np.uint64).reshape(M, 4)
    for i in range(M):
        want, wst = oracle.roc_auc(z[off[i]:off[i + 1]], y[off[i]:off[i + 1]], threads=4)
        assert np.array_equal(gst[i], wst), i
        assert (np.isnan(got[i]) and np.isnan(want)) or got[i] == want, i
