"""Pins for the oracle's detector (Section 2.2 "Detection", Eq. 5)."""
import math

import mpmath
import numpy as np
import pytest
from scipy import stats

from oracle import py_ref
from paper_2609_03844_b200 import inputs

KEY = 0x5EED


@pytest.mark.parametrize("scheme_name", ["context", "selfsalt"])
def test_counts_equal_brute_force_on_tiny_sequences(oracle, scheme_name):
    """Every sequence over a tiny vocabulary up to length 4, plus random short ones: G and T by
    direct enumeration of Y_t with the big-integer restatement."""
    scheme = oracle.SCHEME_SELFSALT if scheme_name == "selfsalt" else oracle.SCHEME_CONTEXT
    seqs = [[]]
    for L in range(1, 5):
        grids = np.stack(np.meshgrid(*[np.arange(3)] * L, indexing="ij"), -1).reshape(-1, L)
        seqs += [list(map(int, g)) for g in grids]
    rng = np.random.default_rng(30)
    seqs += [list(map(int, rng.integers(0, 8, size=int(rng.integers(0, 7))))) for _ in range(200)]
    seqs += [list(map(int, rng.integers(0, 1 << 31, size=6))) for _ in range(50)]
    lengths = np.array([len(s) for s in seqs], dtype=np.int32)
    flat = np.array([t for s in seqs for t in s], dtype=np.int32)
    for gamma in (0.25, 0.5):
        counts, T, z = oracle.detect(flat, lengths, KEY, gamma, scheme)
        for i, s in enumerate(seqs):
            G, Ts = py_ref.detect_counts(s, KEY, gamma, scheme_name)
            assert (counts[i], T[i]) == (G, Ts)
            if Ts == 0:
                assert z[i] == 0.0
            else:
                assert z[i] == pytest.approx((G - gamma * Ts) / math.sqrt(Ts * gamma * (1 - gamma)),
                                             abs=1e-12)


def test_wider_context_counts_equal_brute_force(oracle):
    rng = np.random.default_rng(31)
    for W in (2, 4):
        for name, scheme in (("context", oracle.SCHEME_CONTEXT), ("selfsalt", oracle.SCHEME_SELFSALT)):
            seqs = [list(map(int, rng.integers(0, 50000, size=int(rng.integers(0, 12)))))
                    for _ in range(60)]
            lengths = np.array([len(s) for s in seqs], dtype=np.int32)
            flat = np.array([t for s in seqs for t in s], dtype=np.int32)
            counts, T, _ = oracle.detect(flat, lengths, KEY, 0.25, scheme, ctx_width=W)
            for i, s in enumerate(seqs):
                assert (counts[i], T[i]) == py_ref.detect_counts(s, KEY, 0.25, name, W)


def test_z_closed_forms(oracle):
    """Eq. 5: G = gamma T gives 0; all green gives sqrt(T(1-gamma)/gamma); none green gives
    -sqrt(T gamma/(1-gamma)).  T = 199, gamma = 1/4, all green: 24.4336..."""
    assert oracle.zscore(50, 200, 0.25) == 0.0
    assert oracle.zscore(199, 199, 0.25) == pytest.approx(math.sqrt(199 * 3.0), abs=1e-12)
    assert round(oracle.zscore(199, 199, 0.25), 4) == 24.4336
    assert oracle.zscore(0, 199, 0.25) == pytest.approx(-math.sqrt(199 / 3.0), abs=1e-12)
    assert oracle.zscore(0, 0, 0.25) == 0.0
    mpmath.mp.dps = 40
    rng = np.random.default_rng(32)
    for _ in range(300):
        T = int(rng.integers(1, 5000))
        G = int(rng.integers(0, T + 1))
        g = float(rng.choice([0.25, 0.5, 0.1, 0.37]))
        gm = mpmath.mpf(g)
        want = (G - gm * T) / mpmath.sqrt(T * gm * (1 - gm))
        assert abs(mpmath.mpf(oracle.zscore(G, T, g)) - want) < mpmath.mpf(10) ** -12


@pytest.mark.parametrize("scheme_name", ["context", "selfsalt"])
@pytest.mark.parametrize("gamma", [0.25, 0.5])
def test_null_law_on_uniform_token_streams(oracle, scheme_name, gamma):
    """Section 3: under H0 the Y_t are i.i.d. Bernoulli(gamma), so for fixed T the green count is
    Binomial(T, gamma) exactly and z has mean 0 and variance 1."""
    scheme = oracle.SCHEME_SELFSALT if scheme_name == "selfsalt" else oracle.SCHEME_CONTEXT
    V, N, L = 128256, 20000, 65
    tokens = inputs.uniform_tokens((N * L,), V, seed=33).numpy()
    lengths = np.full(N, L, dtype=np.int32)
    counts, T, z = oracle.detect(tokens, lengths, KEY, gamma, scheme, threads=4)
    assert np.all(T == L - 1)
    assert abs(z.mean()) < 4 / math.sqrt(N)
    assert abs(z.var() - 1.0) < 0.05
    # chi-square of the count histogram against the Binomial(64, gamma) pmf
    Tn = L - 1
    pmf = stats.binom.pmf(np.arange(Tn + 1), Tn, gamma)
    exp = pmf * N
    keep = exp >= 5
    obs = np.bincount(counts, minlength=Tn + 1).astype(float)
    obs_k = np.append(obs[keep], obs[~keep].sum())
    exp_k = np.append(exp[keep], exp[~keep].sum())
    chi2 = ((obs_k - exp_k) ** 2 / exp_k).sum()
    assert chi2 < stats.chi2.ppf(1 - 1e-6, len(obs_k) - 1)
    # loose KS check against N(0,1): Binomial(64, .) is a lattice whose largest step is the
    # largest pmf value, so D sits near half of that
    assert stats.kstest(z, "norm").statistic < pmf.max() / 2 + 0.03


def test_ragged_batch_and_threads(oracle):
    tokens, lengths = inputs.null_token_streams(300, 0, 90, 32000, seed=34)
    tok, lens = tokens.numpy(), lengths.numpy()
    for scheme in (oracle.SCHEME_CONTEXT, oracle.SCHEME_SELFSALT):
        c1, T1, z1 = oracle.detect(tok, lens, KEY, 0.25, scheme, threads=1)
        c4, T4, z4 = oracle.detect(tok, lens, KEY, 0.25, scheme, threads=4)
        assert np.array_equal(c1, c4) and np.array_equal(T1, T4) and np.array_equal(z1, z4)
        assert np.array_equal(T1, np.maximum(lens - 1, 0))
        # each sequence scored alone gives the same numbers (no leakage across boundaries)
        off = np.concatenate([[0], np.cumsum(lens)])
        for i in (0, 1, 17, 150, 299):
            ci, Ti, zi = oracle.detect(tok[off[i]:off[i + 1]], lens[i:i + 1], KEY, 0.25, scheme)
            assert (ci[0], Ti[0], zi[0]) == (c1[i], T1[i], z1[i])
