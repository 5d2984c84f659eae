"""Pins for the oracle's evaluation steps around detection: distinct-tuple scoring, truncated
text, ROC-AUC (Section 4.3).  Each is checked against something that is not the oracle's own
formula: Python sets, slices fed to the plain detector, scikit-learn, exact rationals, closed forms."""
from fractions import Fraction

import numpy as np
import pytest
from scipy.stats import norm

import oracle
from paper_2609_03844_b200 import inputs

KEY = 0x5EED


def _flat(seqs):
    lens = np.array([len(s) for s in seqs], dtype=np.int32)
    tok = np.concatenate([np.asarray(s, dtype=np.int32) for s in seqs]) if seqs else np.zeros(0, np.int32)
    return tok, lens


# ---------------------------------------------------------------- distinct tuples ----
@pytest.mark.parametrize("scheme", [oracle.SCHEME_CONTEXT, oracle.SCHEME_SELFSALT])
@pytest.mark.parametrize("W", [1, 2, 4])
def test_unique_matches_a_python_set_of_tuples(scheme, W):
    rng = np.random.default_rng(5 + W)
    # a small alphabet makes repeats common
    seqs = [rng.integers(0, 6, size=int(n)).tolist() for n in rng.integers(0, 120, size=40)]
    tok, lens = _flat(seqs)
    bits = oracle.detect_bits(tok, lens, KEY, 0.25, scheme, ctx_width=W)
    counts, T, z = oracle.detect_unique(tok, lens, KEY, 0.25, scheme, ctx_width=W)
    off = 0
    for s, seq in enumerate(seqs):
        seen, G = set(), 0
        for t in range(W, len(seq)):
            tup = tuple(seq[t - W:t + 1])
            if tup not in seen:
                seen.add(tup)
                G += int(bits[off + t])
        assert (counts[s], T[s]) == (G, len(seen))
        assert z[s] == oracle.zscore(G, len(seen), 0.25)
        off += len(seq)


def test_unique_closed_forms():
    W = 1
    # no repeated tuple: the plain detector
    tok = np.arange(1000, 1300, dtype=np.int32)
    lens = np.array([300], dtype=np.int32)
    for scheme in (0, 1):
        assert [a.tolist() for a in oracle.detect_unique(tok, lens, KEY, 0.5, scheme)] == \
               [a.tolist() for a in oracle.detect(tok, lens, KEY, 0.5, scheme)]
    # one token repeated: a single distinct tuple
    c, T, z = oracle.detect_unique(np.full(50, 7, np.int32), [50], KEY, 0.5, 0, ctx_width=3)
    assert T[0] == 1 and c[0] in (0, 1)
    # a cycle of p distinct tokens has p distinct (previous, token) pairs, however long it runs
    p = 9
    cyc = np.tile(np.arange(p, dtype=np.int32) + 100, 30)
    c1, T1, _ = oracle.detect_unique(cyc, [len(cyc)], KEY, 0.5, 1, ctx_width=W)
    c2, T2, _ = oracle.detect_unique(cyc[:p + W], [p + W], KEY, 0.5, 1, ctx_width=W)
    assert T1[0] == p and (c1[0], T1[0]) == (c2[0], T2[0])
    # shorter than the context, and empty
    c, T, z = oracle.detect_unique(np.array([1, 2, 3], np.int32), [0, 3, 0], KEY, 0.5, 0, ctx_width=4)
    assert c.tolist() == [0, 0, 0] and T.tolist() == [0, 0, 0] and z.tolist() == [0.0, 0.0, 0.0]


def test_unique_never_scores_more_than_the_plain_detector():
    tok = inputs.uniform_tokens((20000,), 50, seed=3).numpy().astype(np.int32)
    lens = np.full(100, 200, np.int32)
    c, T, _ = oracle.detect(tok, lens, KEY, 0.25, 0, ctx_width=2)
    cu, Tu, _ = oracle.detect_unique(tok, lens, KEY, 0.25, 0, ctx_width=2)
    assert (cu <= c).all() and (Tu <= T).all() and (Tu - cu <= T - c).all() and (Tu < T).any()


# ---------------------------------------------------------------- truncated text ----
@pytest.mark.parametrize("W", [1, 4])
def test_prefix_z_is_the_detector_on_the_cut_text(W):
    rng = np.random.default_rng(11)
    lens = rng.integers(0, 90, size=64).astype(np.int32)
    tok = rng.integers(0, 32000, size=int(lens.sum())).astype(np.int32)
    keep = rng.integers(-3, 100, size=64).astype(np.int32)
    bits = oracle.detect_bits(tok, lens, KEY, 0.25, 1, ctx_width=W)
    c, T, z = oracle.prefix_z(bits, lens, keep, 0.25, ctx_width=W)
    off, cut, cut_lens = 0, [], []
    for L, k in zip(lens, keep):
        k = int(min(max(k, 0), L))
        cut.append(tok[off:off + k])
        cut_lens.append(k)
        off += int(L)
    cc, TT, zz = oracle.detect(np.concatenate(cut), np.array(cut_lens, np.int32), KEY, 0.25, 1, ctx_width=W)
    assert c.tolist() == cc.tolist() and T.tolist() == TT.tolist() and z.tolist() == zz.tolist()


# ---------------------------------------------------------------- ROC-AUC ----
def _sweep_auc(z, y):
    """Trapezoid area under the (FPR, TPR) curve swept over every threshold, in exact rationals."""
    pos = sorted(v for v, l in zip(z, y) if l)
    neg = sorted(v for v, l in zip(z, y) if not l)
    pts = [(Fraction(0), Fraction(0))]
    for thr in sorted(set(z), reverse=True):
        tpr = Fraction(sum(v >= thr for v in pos), len(pos))
        fpr = Fraction(sum(v >= thr for v in neg), len(neg))
        pts.append((fpr, tpr))
    return sum((x1 - x0) * (y0 + y1) / 2 for (x0, y0), (x1, y1) in zip(pts, pts[1:]))


def test_auc_equals_the_swept_curve_exactly():
    rng = np.random.default_rng(2)
    for n in (2, 7, 60):
        z = rng.integers(-4, 5, size=n).astype(np.float64) / 2     # many ties
        y = rng.integers(0, 2, size=n).astype(np.uint8)
        y[0], y[1] = 0, 1
        auc, st = oracle.roc_auc(z, y)
        exact = _sweep_auc(z.tolist(), y.tolist())
        assert Fraction(2 * int(st[0]) + int(st[1]), 2 * int(st[2]) * int(st[3])) == exact
        assert auc == float(exact)


def test_auc_matches_scikit_learn():
    from sklearn.metrics import roc_auc_score
    rng = np.random.default_rng(4)
    y = (rng.random(3000) < 0.4).astype(np.uint8)
    z = rng.normal(size=3000) + 1.3 * y
    z[::7] = np.round(z[::7])                                       # some ties
    auc, _ = oracle.roc_auc(z, y, threads=4)
    assert abs(auc - roc_auc_score(y, z)) < 1e-12


def test_auc_special_cases():
    assert oracle.roc_auc([3, 4, 1, 2], [1, 1, 0, 0])[0] == 1.0
    assert oracle.roc_auc([1, 2, 3, 4], [1, 1, 0, 0])[0] == 0.0
    assert oracle.roc_auc([5, 5, 5], [1, 0, 0])[0] == 0.5
    assert oracle.roc_auc([0.0, -0.0], [1, 0])[0] == 0.5           # the two zeros tie
    assert np.isnan(oracle.roc_auc([1.0, 2.0], [1, 1])[0])
    assert np.isnan(oracle.roc_auc([], [])[0])
    auc, st = oracle.roc_auc([np.nan, 2.0, 1.0, np.nan], [1, 1, 0, 0])
    assert auc == 1.0 and st.tolist() == [1, 0, 1, 1]
    # relabelling mirrors the curve; an increasing map of the scores leaves it alone
    rng = np.random.default_rng(9)
    z, y = rng.normal(size=500), rng.integers(0, 2, size=500)
    a = oracle.roc_auc(z, y)[0]
    assert abs(a + oracle.roc_auc(z, 1 - y)[0] - 1.0) < 1e-15
    assert oracle.roc_auc(np.exp(z), y)[0] == a


def test_auc_of_two_shifted_normals():
    rng = np.random.default_rng(13)
    n, d = 4000, 1.0
    z = np.concatenate([rng.normal(d, 1, n), rng.normal(0, 1, n)])
    y = np.concatenate([np.ones(n), np.zeros(n)])
    a = oracle.roc_auc(z, y, threads=4)[0]
    want = norm.cdf(d / np.sqrt(2))
    assert abs(a - want) < 4 * np.sqrt(want * (1 - want) / n)


def test_auc_of_detector_scores_separates_watermarked_from_null_text():
    # null streams against streams made only of green tokens: the curve is the unit square
    V, L, N = 5000, 60, 40
    null = inputs.uniform_tokens((N, L), V, seed=21).numpy().astype(np.int32)
    marked = null.copy()
    thr = oracle.threshold(0.25)
    for s in range(N):
        for t in range(1, L):
            v = int(marked[s, t])
            while not oracle.green(oracle.seed_context(KEY, [int(marked[s, t - 1])]), v, thr):
                v = (v + 1) % V
            marked[s, t] = v
    tok = np.concatenate([null.ravel(), marked.ravel()])
    _, _, z = oracle.detect(tok, np.full(2 * N, L, np.int32), KEY, 0.25, 0)
    assert oracle.roc_auc(z, np.r_[np.zeros(N), np.ones(N)])[0] == 1.0
