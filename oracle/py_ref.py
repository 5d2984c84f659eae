"""Second, independent restatement of SBW's integer hashes with Python big integers.

TEST INFRASTRUCTURE, NOT PRODUCT.  Nothing here is fast and nothing here is shared with the
C oracle or with the CUDA library: every function works on unbounded Python ints and reduces
explicitly, so a mistake in C's implicit wrap-around (a missing cast, a 32-bit product where a
64-bit one was meant) shows up as a disagreement.  Used by the tests to pin ``sbw_oracle.c`` and
by ``tests/golden/make_spec_vectors.py`` to write the known-answer file.

Passages followed: Section 2.2 (Eq. 1, Philox 4x32-10 as the counter-based RNG), Section 2.3
(Jenkins integer hash), Table 12 (additive and anchored-minhash PRFs), Eq. 5 (z-score).
"""
from __future__ import annotations

import math
from fractions import Fraction

M32 = (1 << 32) - 1
M64 = (1 << 64) - 1


def jenkins(a: int) -> int:
    """Section 2.3: six-step 32-bit integer mix."""
    a &= M32
    a = ((a + 0x7ED55D16) + (a << 12)) & M32
    a = ((a ^ 0xC761C23C) ^ (a >> 19)) & M32
    a = ((a + 0x165667B1) + (a << 5)) & M32
    a = ((a + 0xD3A2646C) ^ (a << 9)) & M32
    a = ((a + 0xFD7046C5) + (a << 3)) & M32
    a = ((a ^ 0xB55A4F09) ^ (a >> 16)) & M32
    return a


def philox4x32_10(ctr, key):
    """Section 2.2: Philox 4x32, ten rounds, on four counter words and two key words."""
    c = [x & M32 for x in ctr]
    k = [x & M32 for x in key]
    for i in range(10):
        k0 = (k[0] + i * 0x9E3779B9) & M32
        k1 = (k[1] + i * 0xBB67AE85) & M32
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        c = [((p1 >> 32) ^ c[1] ^ k0) & M32, p1 & M32, ((p0 >> 32) ^ c[3] ^ k1) & M32, p0 & M32]
    return tuple(c)


def seed_context(key: int, ctx) -> int:
    """Additive PRF: key times the sum of the context ids, modulo 2^64."""
    return (key * sum(t & M32 for t in ctx)) & M64


def seed_selfsalt(key: int, ctx, v: int) -> int:
    """Anchored minhash PRF: window = context ids + candidate, anchored on the candidate."""
    jv = jenkins(v)
    window = [t & M32 for t in ctx] + [v & M32]
    return (key * min(jenkins(x) * jv for x in window)) & M64


def threshold(gamma) -> int:
    """ceil(gamma * 2^32) evaluated exactly on the binary value of gamma."""
    return math.ceil(Fraction(gamma) * (1 << 32))


def green(r: int, v: int, thr: int) -> int:
    """Eq. 1: word 0 of Philox(counter (v,0,0,0), key (lo r, hi r)) below the threshold."""
    x = philox4x32_10((v & M32, 0, 0, 0), (r & M32, (r >> 32) & M32))[0]
    return int(x < thr)


def green_bits(key: int, ctx, gamma, scheme: str, vs) -> str:
    thr = threshold(gamma)
    out = []
    for v in vs:
        r = seed_selfsalt(key, ctx, v) if scheme == "selfsalt" else seed_context(key, ctx)
        out.append(str(green(r, v, thr)))
    return "".join(out)


def detect_counts(tokens, key: int, gamma, scheme: str, W: int = 1):
    """Section 2.2 detection: G and T of one sequence by direct enumeration."""
    thr = threshold(gamma)
    G = 0
    for t in range(W, len(tokens)):
        ctx = tokens[t - W:t]
        v = tokens[t]
        r = seed_selfsalt(key, ctx, v) if scheme == "selfsalt" else seed_context(key, ctx)
        G += green(r, v, thr)
    return G, max(len(tokens) - W, 0)
