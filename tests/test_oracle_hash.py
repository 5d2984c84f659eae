"""Pins for the oracle's integer hashes (Sections 2.2 and 2.3, Table 12 of the paper).

The C oracle is checked against things other than itself: a big-integer restatement, the
frozen known answers under tests/golden/, hand arithmetic, structural invariants, and -- for
Philox -- NVIDIA's cuRAND host generator, which runs on the CPU.
"""
import ctypes
from pathlib import Path

import numpy as np
import pytest

from oracle import py_ref

GOLDEN = Path(__file__).resolve().parent / "golden" / "sbw_spec_v1_vectors.txt"
KEY = 0x5EED


def _golden():
    rows = [ln.split() for ln in GOLDEN.read_text().splitlines() if ln and not ln.startswith("#")]
    return rows


# ---------------------------------------------------------------- Jenkins (Section 2.3)
# Known answers of the frozen reading, typed here by hand from an arbitrary-precision
# expansion of the six steps; the golden file must agree with them and so must both oracles.
JENKINS_KAT = {0: 0x6B4ED927, 1: 0xB48681B6, 2: 0xE267B84C, 0x5EED: 0xE3B64A6C,
               128255: 0xF22AFDC6, 151935: 0x223D4FD0, 0xFFFFFFFF: 0xFE64C182}


def test_jenkins_known_answers(oracle):
    file_vals = {int(r[1], 16): int(r[2], 16) for r in _golden() if r[0] == "jenkins"}
    assert file_vals == JENKINS_KAT
    for a, want in JENKINS_KAT.items():
        assert oracle.jenkins(a) == want
        assert py_ref.jenkins(a) == want


def test_jenkins_matches_bigint_on_random_inputs(oracle):
    rng = np.random.default_rng(1)
    xs = rng.integers(0, 1 << 32, size=20000, dtype=np.uint64)
    edge = [0, 1, 0x7FFFFFFF, 0x80000000, 0xFFFFFFFE, 0xFFFFFFFF, 1 << 12, 1 << 19, 1 << 31]
    for a in list(map(int, xs)) + edge:
        assert oracle.jenkins(a) == py_ref.jenkins(a)


def test_jenkins_steps_are_invertible_hence_bijection_on_samples():
    """Undo the six steps one by one (modular inverses / xor-shift unrolling)."""
    M = (1 << 32) - 1

    def unxorshift_right(y, s):
        x = y
        for _ in range(32 // s + 1):
            x = y ^ (x >> s)
        return x & M

    def inv(a):
        a = unxorshift_right(a ^ 0xB55A4F09, 16)                          # step 6
        a = ((a - 0xFD7046C5) * pow(9, -1, 1 << 32)) & M                   # step 5: a*9 + c
        # step 4: y = (a + c) ^ (a << 9): solve low bits upward, 9 at a time
        # (x << 9) built from k known low bits of x is right in its k+9 low bits
        y, x = a, 0
        for known in (9, 18, 27, 32):
            x = ((y ^ ((x << 9) & M)) - 0xD3A2646C) & M & ((1 << known) - 1)
        a = x
        a = ((a - 0x165667B1) * pow(33, -1, 1 << 32)) & M                  # step 3: a*33 + c
        a = unxorshift_right(a ^ 0xC761C23C, 19)                           # step 2
        a = ((a - 0x7ED55D16) * pow(4097, -1, 1 << 32)) & M                # step 1: a*4097 + c
        return a

    rng = np.random.default_rng(2)
    for a in map(int, rng.integers(0, 1 << 32, size=3000, dtype=np.uint64)):
        assert inv(py_ref.jenkins(a)) == a


def test_jenkins_is_a_bijection_exhaustively(oracle):
    """All 2^32 inputs give 2^32 distinct outputs (512 MiB bitmap inside the C helper)."""
    got = oracle.jenkins_collisions()
    if got < 0:
        pytest.skip("not enough memory for the 2^32-bit bitmap")
    assert got == 0


def test_jenkins_avalanche(oracle):
    """Flipping any input bit flips every output bit roughly half the time (every pair within
    [0.2, 0.8]; the average over all 1024 pairs within 0.5 +- 0.01)."""
    rng = np.random.default_rng(3)
    n = 20000
    xs = rng.integers(0, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32)

    def J(arr):  # vectorised restatement used only to gather statistics quickly
        a = arr.astype(np.uint64)
        m = np.uint64(0xFFFFFFFF)
        a = ((a + np.uint64(0x7ED55D16)) + (a << np.uint64(12))) & m
        a = ((a ^ np.uint64(0xC761C23C)) ^ (a >> np.uint64(19))) & m
        a = ((a + np.uint64(0x165667B1)) + (a << np.uint64(5))) & m
        a = ((a + np.uint64(0xD3A2646C)) ^ (a << np.uint64(9))) & m
        a = ((a + np.uint64(0xFD7046C5)) + (a << np.uint64(3))) & m
        a = ((a ^ np.uint64(0xB55A4F09)) ^ (a >> np.uint64(16))) & m
        return a.astype(np.uint32)

    for a in map(int, xs[:200]):
        assert int(J(np.array([a], dtype=np.uint32))[0]) == oracle.jenkins(a)
    base = J(xs)
    fracs = np.zeros((32, 32))
    for ib in range(32):
        diff = base ^ J(xs ^ np.uint32(1 << ib))
        for ob in range(32):
            fracs[ib, ob] = float(((diff >> np.uint32(ob)) & np.uint32(1)).mean())
    assert fracs.min() > 0.2 and fracs.max() < 0.8, (fracs.min(), fracs.max())
    assert abs(fracs.mean() - 0.5) < 0.01


# ---------------------------------------------------------------- Philox (Section 2.2)
def test_philox_known_answers(oracle):
    rows = [r for r in _golden() if r[0] == "philox"]
    assert len(rows) >= 6
    for r in rows:
        ctr = [int(x, 16) for x in r[1:5]]
        key = [int(x, 16) for x in r[6:8]]
        want = tuple(int(x, 16) for x in r[9:13])
        assert oracle.philox(ctr, key) == want
        assert py_ref.philox4x32_10(ctr, key) == want
    # hand-typed from the arbitrary-precision expansion
    assert oracle.philox((0, 0, 0, 0), (0, 0)) == (0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8)
    assert oracle.philox((0xFFFFFFFF,) * 4, (0xFFFFFFFF,) * 2) == (0x408F276D, 0x41C83B0E,
                                                                0xA20BC7C6, 0x6D5451FD)
    assert oracle.philox((1, 0, 0, 0), (KEY, 0))[0] == 0xE79E8EE4
    assert oracle.philox((0, 0, 0, 0), (KEY, 0))[0] == 0xEE1C2FCC
    assert oracle.philox((12345, 0, 0, 0), (KEY, 0))[0] == 0xF4B068D1


def test_philox_matches_bigint_on_random_inputs(oracle):
    rng = np.random.default_rng(4)
    for _ in range(3000):
        ctr = [int(x) for x in rng.integers(0, 1 << 32, size=4, dtype=np.uint64)]
        key = [int(x) for x in rng.integers(0, 1 << 32, size=2, dtype=np.uint64)]
        assert oracle.philox(ctr, key) == py_ref.philox4x32_10(ctr, key)


def _curand_host():
    for name in ("libcurand.so", "libcurand.so.10", "/usr/local/cuda/lib64/libcurand.so.10"):
        try:
            return ctypes.CDLL(name)
        except OSError:
            continue
    return None


def test_philox_equals_curand_host_generator(oracle):
    """Library special case: NVIDIA's cuRAND *host* Philox4_32_10 generator runs on the CPU.
    It interleaves 65536 streams: with seed s, the group of four outputs number g (from zero)
    holds the four words of Philox(counter (n lo, n hi, j, 0), key (lo s, hi s)) with
    j = g mod 65536 and n = g div 65536, and the generator offset counts single outputs.
    This pins rounds, multipliers, Weyl constants, word order and the seed-to-key split
    independently of any code in this repository."""
    cr = _curand_host()
    if cr is None:
        pytest.skip("libcurand not loadable")
    gen = ctypes.c_void_p()
    CURAND_RNG_PSEUDO_PHILOX4_32_10 = 161
    if cr.curandCreateGeneratorHost(ctypes.byref(gen), CURAND_RNG_PSEUDO_PHILOX4_32_10) != 0:
        pytest.skip("cuRAND host generator unavailable")
    cr.curandSetPseudoRandomGeneratorSeed.argtypes = [ctypes.c_void_p, ctypes.c_ulonglong]
    cr.curandSetGeneratorOffset.argtypes = [ctypes.c_void_p, ctypes.c_ulonglong]
    cr.curandGenerate.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t]
    rng = np.random.default_rng(5)
    seeds = [0, 1, KEY, 0x2987B, 0xFFFFFFFFFFFFFFFF, 0xCF0AEC2D64FEC41D] + \
        [int(x) for x in rng.integers(0, 1 << 63, size=20, dtype=np.uint64)]
    for s in seeds:
        ns = [0, 1, 2, 12345, 128255, 151935, 0xFFFFFFFF, (1 << 32) + 5, (7 << 32) | 0x89ABCDEF] + \
            [int(x) for x in rng.integers(0, 1 << 40, size=10, dtype=np.uint64)]
        for n in ns:
            j = int(rng.integers(0, 65535))
            assert cr.curandSetPseudoRandomGeneratorSeed(gen, s) == 0
            assert cr.curandSetGeneratorOffset(gen, 4 * (n * 65536 + j)) == 0
            out = np.zeros(8, dtype=np.uint32)
            assert cr.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), 8) == 0
            key = (s & 0xFFFFFFFF, s >> 32)
            for grp in range(2):
                ctr = (n & 0xFFFFFFFF, n >> 32, j + grp, 0)
                assert oracle.philox(ctr, key) == tuple(int(x) for x in out[4 * grp:4 * grp + 4]), \
                    (s, n, j, grp)
    cr.curandDestroyGenerator(gen)


# ---------------------------------------------------------------- seeds (Table 12)
def test_context_seed_hand_values(oracle):
    # 0x5EED = 24301; 24301 * 7 = 170107 = 0x2987B
    assert oracle.seed_context(KEY, [7]) == 170107 == 0x2987B
    assert oracle.seed_context(KEY, [0]) == 0                      # additive PRF: ctx 0 -> seed 0
    assert oracle.seed_context(KEY, [1, 2, 4]) == 24301 * 7
    # wrap-around modulo 2^64 and ids taken as unsigned 32-bit
    big = 0xFFFFFFFFFFFFFFC5
    assert oracle.seed_context(big, [0xFFFFFFFF, 0xFFFFFFFF]) == (big * (2 * 0xFFFFFFFF)) % (1 << 64)
    assert oracle.seed_context(KEY, [-1]) == KEY * 0xFFFFFFFF


def test_selfsalt_seed_golden_and_identity(oracle):
    rows = [r for r in _golden() if r[0] == "seed_selfsalt"]
    want_typed = [0xCF0AEC2D64FEC41D, 0x48BB52205F467D94, 0x24967BAA084A0350, 0x71426173312FB1D0]
    assert [int(r[4], 16) for r in rows] == want_typed
    for v, want in enumerate(want_typed):
        assert oracle.seed_selfsalt(KEY, [7], v) == want
    # width-1 closed form: r = key * J(v) * min(J(c), J(v))  (mod 2^64)
    rng = np.random.default_rng(6)
    for _ in range(2000):
        key = int(rng.integers(0, 1 << 63, dtype=np.uint64)) * 2 + 1
        c, v = (int(x) for x in rng.integers(0, 200000, size=2))
        jc, jv = py_ref.jenkins(c), py_ref.jenkins(v)
        assert oracle.seed_selfsalt(key, [c], v) == (key * jv * min(jc, jv)) % (1 << 64)
    # general window against the big-integer restatement
    for _ in range(500):
        key = int(rng.integers(0, 1 << 63, dtype=np.uint64))
        W = int(rng.integers(1, 6))
        ctx = [int(x) for x in rng.integers(0, 1 << 32, size=W, dtype=np.uint64)]
        v = int(rng.integers(0, 1 << 32, dtype=np.uint64))
        assert oracle.seed_selfsalt(key, ctx, v) == py_ref.seed_selfsalt(key, ctx, v)
        assert oracle.seed_context(key, ctx) == py_ref.seed_context(key, ctx)


# ---------------------------------------------------------------- membership (Eq. 1)
def test_threshold_is_ceil_gamma_2_32(oracle):
    assert oracle.threshold(0.25) == 1 << 30
    assert oracle.threshold(0.5) == 1 << 31
    assert oracle.threshold(1e-12) == 1
    assert oracle.threshold(1 - 2.0 ** -40) == 1 << 32
    for g in (0.1, 0.3, 1 / 3, 0.7, 0.999):
        assert oracle.threshold(g) == py_ref.threshold(g)


def test_green_bits_golden(oracle):
    rows = {r[0]: r for r in _golden() if r[0].startswith("green_") and len(r) == 3}
    assert rows["green_context"][2] == "0000001101010110"
    assert rows["green_selfsalt"][2] == "0110011100001100"
    m = oracle.green_mask(1, 16, [[7]], KEY, 0.25, oracle.SCHEME_CONTEXT)
    assert "".join(map(str, m[0])) == rows["green_context"][2]
    m = oracle.green_mask(1, 16, [[7]], KEY, 0.25, oracle.SCHEME_SELFSALT)
    assert "".join(map(str, m[0])) == rows["green_selfsalt"][2]
    words = [int(r[4], 16) for r in _golden() if r[0] == "word0_context"]
    assert words == [0x59884A6C, 0xC6E8E8B5, 0x6108E95A, 0x5EEFE02F]
    for v, x in enumerate(words):
        assert oracle.philox((v, 0, 0, 0), (0x2987B, 0))[0] == x
        assert oracle.green(0x2987B, v, 1 << 30) == int(x < (1 << 30))


def test_green_is_strict_and_uses_word0(oracle):
    r, v = 0x0123456789ABCDEF, 4242
    x = py_ref.philox4x32_10((v, 0, 0, 0), (r & 0xFFFFFFFF, r >> 32))[0]
    assert oracle.green(r, v, x) == 0          # strict "<" of Eq. 1
    assert oracle.green(r, v, x + 1) == 1
    assert oracle.green(r, v, 1 << 32) == 1    # threshold 2^32 accepts every word


def test_green_counts_golden(oracle):
    for r in (r for r in _golden() if r[0] == "green_count"):
        scheme = oracle.SCHEME_SELFSALT if r[1] == "selfsalt" else oracle.SCHEME_CONTEXT
        V, gamma, ctx, want = int(r[2]), float(r[3]), int(r[4]), int(r[5])
        m = oracle.green_mask(1, V, [[ctx]], KEY, gamma, scheme)
        assert int(m.sum()) == want
    typed = {("context", 32000): 7946, ("context", 128256): 64283, ("selfsalt", 32000): 8021}
    got = {(r[1], int(r[2])): int(r[5]) for r in _golden() if r[0] == "green_count"}
    assert got == typed


def test_green_mask_matches_bigint_with_offset_and_width(oracle):
    rng = np.random.default_rng(7)
    for scheme, name in ((oracle.SCHEME_CONTEXT, "context"), (oracle.SCHEME_SELFSALT, "selfsalt")):
        for W in (1, 2, 4):
            B, V, off = 3, 37, int(rng.integers(0, 100000))
            ctx = rng.integers(0, 150000, size=(B, W)).astype(np.int32)
            key = int(rng.integers(0, 1 << 63, dtype=np.uint64))
            gamma = float(rng.choice([0.25, 0.5, 0.37]))
            m = oracle.green_mask(B, V, ctx, key, gamma, scheme, vocab_offset=off)
            for b in range(B):
                want = py_ref.green_bits(key, [int(t) for t in ctx[b]], gamma, name,
                                         range(off, off + V))
                assert "".join(map(str, m[b])) == want
