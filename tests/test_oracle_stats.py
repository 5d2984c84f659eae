"""Statistical pins from the paper's Section 3 and Appendix H: the Bernoulli green list has
|G_t| ~ Binomial(|V|, gamma), membership is independent across candidates and across contexts,
and the arithmetic of these checks reproduces the numbers the paper prints."""
import math
from pathlib import Path

import numpy as np
import pytest

GOLDEN = Path(__file__).resolve().parent / "golden" / "paper_appendix_h_green_list_size.txt"
KEY = 0x5EED


def _paper():
    vals = {}
    for ln in GOLDEN.read_text().splitlines():
        if ln and not ln.startswith("#"):
            k, v = ln.split()
            vals[k] = float(v)
    return vals


def test_paper_worked_example_arithmetic():
    """Appendix H: gamma = 0.5, |V| = 151936 gives sigma ~ 1.28 per mille ~ 195 tokens of
    ~75968; Hoeffding at 1% is below 2e-13.  Checks the formulas used by the tests below."""
    p = _paper()
    g, V = p["gamma"], p["V"]
    sigma = math.sqrt(g * (1 - g) / V)
    assert round(sigma * 1000, 2) == p["sigma_permille"]
    assert round(sigma * V) == p["sigma_tokens"]
    assert g * V == p["expected_green"]
    bound = 2 * math.exp(-2 * V * p["hoeffding_eps"] ** 2)
    assert bound < p["hoeffding_upper"] and bound > p["hoeffding_upper"] / 2


def _masks_over_keys(oracle, n, V, gamma, scheme, rng):
    """n green lists under n different secret keys (and contexts).  Different keys re-seed every
    candidate, so the lists are independent under both schemes.  (Under the anchored-minhash PRF
    two contexts with the SAME key share the seed of every candidate whose hash is below both
    context hashes, so lists that differ only in context are correlated by construction.)"""
    rows = []
    for _ in range(n):
        key = int(rng.integers(0, 1 << 63, dtype=np.uint64)) * 2 + 1
        ctx = rng.integers(1, V, size=(1, 1)).astype(np.int32)
        rows.append(oracle.green_mask(1, V, ctx, key, gamma, scheme)[0])
    return np.stack(rows)


@pytest.mark.parametrize("scheme_name", ["context", "selfsalt"])
@pytest.mark.parametrize("V,gamma", [(32000, 0.25), (128256, 0.5), (151936, 0.25), (151936, 0.5)])
def test_green_fraction_is_binomial(oracle, scheme_name, V, gamma):
    scheme = oracle.SCHEME_SELFSALT if scheme_name == "selfsalt" else oracle.SCHEME_CONTEXT
    rng = np.random.default_rng(V + int(gamma * 100))
    n = 24
    mask = _masks_over_keys(oracle, n, V, gamma, scheme, rng)
    frac = mask.mean(axis=1)
    sigma = math.sqrt(gamma * (1 - gamma) / V)
    zs = (frac - gamma) / sigma
    assert np.all(np.abs(frac - gamma) < 0.01)          # Hoeffding, < 2e-13 per list
    assert np.all(np.abs(zs) < 5.0)
    assert abs(zs.mean()) < 5.0 / math.sqrt(n)
    assert 0.35 < zs.var(ddof=1) < 2.1                  # chi-square(23)/23 lies there w.p. > 0.9995


def test_green_fraction_pooled_over_many_lists(oracle):
    """Standardised green-list sizes over 600 independent lists look N(0,1): mean 0, variance 1."""
    V, gamma = 32000, 0.25
    rng = np.random.default_rng(11)
    for scheme in (oracle.SCHEME_CONTEXT, oracle.SCHEME_SELFSALT):
        mask = _masks_over_keys(oracle, 600, V, gamma, scheme, rng)
        zs = (mask.sum(axis=1) - gamma * V) / math.sqrt(V * gamma * (1 - gamma))
        assert abs(zs.mean()) < 0.2                    # 4.9 sigma of the mean
        assert abs(zs.var(ddof=1) - 1.0) < 0.3          # 5 sigma of the sample variance


def test_context_scheme_lists_independent_across_contexts_same_key(oracle):
    """Context scheme, one key, many contexts: distinct seeds, so the sizes are i.i.d. too."""
    V, gamma = 32000, 0.5
    rng = np.random.default_rng(13)
    ctx = rng.choice(np.arange(1, V), size=(600, 1), replace=False).astype(np.int32)
    mask = oracle.green_mask(600, V, ctx, KEY, gamma, oracle.SCHEME_CONTEXT)
    zs = (mask.sum(axis=1) - gamma * V) / math.sqrt(V * gamma * (1 - gamma))
    assert abs(zs.mean()) < 0.2
    assert abs(zs.var(ddof=1) - 1.0) < 0.3


def test_membership_independent_across_candidates_and_contexts(oracle):
    """Appendix H: distinct seeds give independent lists, candidates are i.i.d. within a list:
    joint green frequencies equal gamma^2 within binomial bounds."""
    V, gamma = 128256, 0.25
    rng = np.random.default_rng(12)
    for scheme in (oracle.SCHEME_CONTEXT, oracle.SCHEME_SELFSALT):
        ctx = rng.choice(np.arange(1, V), size=(8, 1), replace=False).astype(np.int32)
        m = oracle.green_mask(8, V, ctx, KEY, gamma, scheme).astype(np.int64)
        s2 = math.sqrt(gamma ** 2 * (1 - gamma ** 2))
        if scheme == oracle.SCHEME_CONTEXT:
            for a in range(0, 8, 2):                               # across contexts
                joint = (m[a] & m[a + 1]).mean()
                assert abs(joint - gamma ** 2) < 5 * s2 / math.sqrt(V)
        for lag in (1, 2, 3, 4, 64):                               # across candidates
            joint = (m[0, :-lag] & m[0, lag:]).mean()
            assert abs(joint - gamma ** 2) < 5 * s2 / math.sqrt(V - lag)


def test_context_zero_is_the_additive_prf_fixed_point(oracle):
    """With the additive PRF a zero context gives seed 0 whatever the key (kept, documented)."""
    a = oracle.green_mask(1, 4096, [[0]], 0x1111, 0.5, oracle.SCHEME_CONTEXT)
    b = oracle.green_mask(1, 4096, [[0]], 0x9999, 0.5, oracle.SCHEME_CONTEXT)
    assert np.array_equal(a, b)
    c = oracle.green_mask(1, 4096, [[5]], 0x1111, 0.5, oracle.SCHEME_CONTEXT)
    d = oracle.green_mask(1, 4096, [[5]], 0x9999, 0.5, oracle.SCHEME_CONTEXT)
    assert not np.array_equal(c, d)
