"""Pins for the oracle's common random generator (CPU only).

The paper asks only for a common generator of fresh N(0, I_d) vectors
(Algorithm 1, first step); the generator itself is Philox4x32-10 + Box-Muller.
The checks here tie the C oracle to things that are not the C oracle: the
published known-answer vectors, an arbitrary-precision integer restatement, hand
evaluated rounds, exact symmetries of the Box-Muller map, and the N(0,1) law.
"""
import math
import os

import numpy as np
import pytest
from scipy import stats

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
MASK = (1 << 32) - 1


# ---- arbitrary-precision restatement of Philox4x32-10 (Python ints) -----------

def bigint_philox(ctr, key, rounds=10):
    c = [int(v) for v in ctr]
    k = [int(v) for v in key]
    for r in range(rounds):
        if r:
            k = [(k[0] + 0x9E3779B9) & MASK, (k[1] + 0xBB67AE85) & MASK]
        pa = 0xD2511F53 * c[0]
        pb = 0xCD9E8D57 * c[2]
        c = [(pb >> 32) ^ c[1] ^ k[0], pb & MASK, (pa >> 32) ^ c[3] ^ k[1], pa & MASK]
    return c


def test_published_known_answer_vectors():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for row in rows:
        v = [int(x, 16) for x in row]
        got = oracle.philox4x32_10(v[0:4], v[4:6])
        assert [int(x) for x in got] == v[6:10]
        assert bigint_philox(v[0:4], v[4:6]) == v[6:10]


def test_single_round_by_hand():
    # counter (1,0,0,0), key (0,0): only the product M_A * 1 = 0x00000000_D2511F53 is non-zero;
    # its low word lands in slot 3, its (zero) high word in slot 2.
    assert [int(x) for x in oracle.philox_round([1, 0, 0, 0], [0, 0])] == [0, 0, 0, 0xD2511F53]
    # counter (0,0,1,0): M_B * 1 -> low word in slot 1.
    assert [int(x) for x in oracle.philox_round([0, 0, 1, 0], [0, 0])] == [0, 0xCD9E8D57, 0, 0]
    # all-ones counter, key (k0,k1): M*(2^32-1) = (M-1)*2^32 + (2^32-M)
    k0, k1 = 0x12345678, 0x9ABCDEF0
    ma, mb = 0xD2511F53, 0xCD9E8D57
    expect = [(mb - 1) ^ MASK ^ k0, (1 << 32) - mb, (ma - 1) ^ MASK ^ k1, (1 << 32) - ma]
    assert [int(x) for x in oracle.philox_round([MASK] * 4, [k0, k1])] == expect


def test_against_bigint_restatement_on_many_counters():
    rng = np.random.default_rng(12345)
    cases = rng.integers(0, 1 << 32, size=(20000, 6), dtype=np.uint64)
    edge = [[0, 0, 0, 0, 0, 0], [MASK] * 6, [MASK, 0, 0, 0, 0, 0], [0, MASK, 0, 0, 0, 0],
            [0, 0, MASK, 0, 0, 0], [0, 0, 0, MASK, 0, 0], [0, 0, 0, 0, MASK, 0], [0, 0, 0, 0, 0, MASK]]
    for row in list(cases) + edge:
        row = [int(v) for v in row]
        got = [int(x) for x in oracle.philox4x32_10(row[:4], row[4:])]
        assert got == bigint_philox(row[:4], row[4:])


def test_keying_of_xi_words():
    # key = (seed lo, seed hi); counter = (q lo, q hi, j, t)
    for seed, t, j, q in [(1, 0, 0, 0), (0xDEADBEEFCAFEF00D, 7, 4095, 3), (5, 2, 1, (1 << 32) + 17),
                          (2**64 - 1, 2**32 - 1, 2**32 - 1, 2**62 - 1)]:
        want = bigint_philox([q & MASK, q >> 32, j, t], [seed & MASK, seed >> 32])
        assert [int(x) for x in oracle.xi_words(seed, t, j, q)] == want
    # distinct (q, j, t) give distinct blocks (the map is a bijection of the counter)
    seen = set()
    for q in range(64):
        for j in range(32):
            for t in range(8):
                seen.add(tuple(int(x) for x in oracle.xi_words(9, t, j, q)))
    assert len(seen) == 64 * 32 * 8


def test_word_stream_bit_balance_and_serial_correlation():
    W = oracle.xi_words_range(3, 0, 5, 0, 1 << 15).astype(np.uint64)   # 2^17 words
    flat = W.reshape(-1)
    n = flat.size
    for bit in range(32):
        ones = int(((flat >> np.uint64(bit)) & np.uint64(1)).sum())
        assert abs(ones - n / 2) < 5 * math.sqrt(n / 4)
    u = flat.astype(np.float64) / 2**32
    r = np.corrcoef(u[:-1], u[1:])[0, 1]
    assert abs(r) < 5 / math.sqrt(n)


# ---- uniforms -------------------------------------------------------------------

def test_uniform_is_exact_and_open():
    assert oracle.uniform(0) == 2.0**-24
    assert oracle.uniform(0x1FF) == 2.0**-24                  # low 9 bits are dropped
    assert oracle.uniform(0x200) == 3 * 2.0**-24
    assert oracle.uniform(MASK) == 1.0 - 2.0**-24
    for w in (0, 0x200, 0x87654321, MASK):
        u = oracle.uniform(w)
        assert float(np.float32(u)) == u and 0.0 < u < 1.0


# ---- Box-Muller -----------------------------------------------------------------

def test_box_muller_symmetries():
    rng = np.random.default_rng(7)
    for _ in range(200):
        w = [int(v) for v in rng.integers(0, 1 << 32, size=4)]
        z = oracle.box_muller(w)
        # adding half a turn to the angle word negates the pair
        w2 = [w[0], w[1] ^ 0x80000000, w[2], w[3] ^ 0x80000000]
        assert np.allclose(oracle.box_muller(w2), -z, rtol=0, atol=1e-14)
        # complementing the angle index maps theta -> 2 pi - theta: cos kept, sin negated
        w3 = [w[0], w[1] ^ MASK, w[2], w[3] ^ MASK]
        z3 = oracle.box_muller(w3)
        assert np.allclose(z3, z * np.array([1, -1, 1, -1]), rtol=0, atol=1e-14)
        # a quarter turn rotates (cos, sin) -> (-sin, cos)
        w4 = [w[0], (w[1] + 0x40000000) & MASK, w[2], (w[3] + 0x40000000) & MASK]
        z4 = oracle.box_muller(w4)
        assert np.allclose(z4, np.array([-z[1], z[0], -z[3], z[2]]), rtol=0, atol=1e-14)
        # the radius inverts to the uniform: u = exp(-(z0^2 + z1^2) / 2)
        assert math.isclose(math.exp(-(z[0] ** 2 + z[1] ** 2) / 2), oracle.uniform(w[0]), rel_tol=1e-12)
        assert math.isclose(math.exp(-(z[2] ** 2 + z[3] ** 2) / 2), oracle.uniform(w[2]), rel_tol=1e-12)
        # the low 9 bits of every word are ignored
        w5 = [v ^ 0x155 for v in w]
        assert np.array_equal(oracle.box_muller(w5), z)


def test_box_muller_extremes():
    # smallest uniform -> largest radius sqrt(2 * 24 * ln 2); angle index 0 -> theta = pi 2^-23
    z = oracle.box_muller([0, 0, MASK, MASK])
    rmax = math.sqrt(48 * math.log(2))
    th = math.pi * 2.0**-23
    assert math.isclose(z[0], rmax * math.cos(th), rel_tol=1e-14)
    assert math.isclose(z[1], rmax * math.sin(th), rel_tol=1e-12)
    rmin = math.sqrt(-2 * math.log1p(-(2.0**-24)))
    assert math.isclose(z[2], rmin * math.cos(th), rel_tol=1e-12)
    assert math.isclose(z[3], -rmin * math.sin(th), rel_tol=1e-9)
    assert abs(z[0]) < 5.78


def test_xi_block_is_box_muller_of_its_words():
    for (seed, t, j, q) in [(1, 0, 0, 0), (11, 3, 7, 123456789012)]:
        assert np.array_equal(oracle.xi_block(seed, t, j, q), oracle.box_muller(oracle.xi_words(seed, t, j, q)))
    # xi_range indexes coordinate k as lane k & 3 of block k >> 2
    r = oracle.xi_range(1, 0, 2, 5, 14)
    for idx, k in enumerate(range(5, 14)):
        assert r[idx] == oracle.xi_block(1, 0, 2, k >> 2)[k & 3]


def test_gaussian_law_of_xi():
    # 2^20 coordinates of one vector: N(0,1) by moments and by Kolmogorov-Smirnov
    z = oracle.xi_range(2024, 1, 3, 0, 1 << 20)
    n = z.size
    assert abs(z.mean()) < 4 / math.sqrt(n)
    assert abs(z.var() - 1) < 4 * math.sqrt(2 / n)
    assert abs((z**4).mean() - 3) < 4 * math.sqrt(96 / n)
    assert abs((z**3).mean()) < 4 * math.sqrt(15 / n)
    assert stats.kstest(z, "norm").pvalue > 1e-3
    # each of the four lanes separately (a sign or a swapped cos/sin would not show in the pool,
    # a wrong angle range would)
    for lane in range(4):
        assert stats.kstest(z[lane::4], "norm").pvalue > 1e-3
    # the two members of a pair are uncorrelated, also in their squares (true for Box-Muller)
    a, b = z[0::4], z[1::4]
    assert abs(np.corrcoef(a, b)[0, 1]) < 5 / math.sqrt(a.size)
    assert abs(np.corrcoef(a * a, b * b)[0, 1]) < 5 / math.sqrt(a.size)
    # polar angle of a pair is uniform on the circle, radius^2 / 2 is Exp(1)
    ang = (np.arctan2(b, a) / (2 * math.pi)) % 1.0
    assert stats.kstest(ang, "uniform").pvalue > 1e-3
    assert stats.kstest((a * a + b * b) / 2, "expon").pvalue > 1e-3


def test_vectors_and_rounds_are_fresh():
    # different j, different t and different seeds give uncorrelated vectors
    base = oracle.xi_range(5, 0, 0, 0, 1 << 16)
    for other in (oracle.xi_range(5, 0, 1, 0, 1 << 16), oracle.xi_range(5, 1, 0, 0, 1 << 16),
                  oracle.xi_range(6, 0, 0, 0, 1 << 16)):
        assert abs(np.corrcoef(base, other)[0, 1]) < 5 / math.sqrt(base.size)
    assert np.array_equal(base, oracle.xi_range(5, 0, 0, 0, 1 << 16))


# ---- the two loop helpers the GPU generator tests take their expected values from ------------

def test_xi_words_range_is_xi_words_block_by_block():
    # a window that starts away from zero and crosses a multiple of 2^32 (the high counter word
    # changes inside it): row r must be the words of block q0 + r, not of block r or q0 + r +- 1
    for seed, t, j, q0, nq in [(0xDEADBEEFCAFEF00D, 7, 4095, (1 << 32) - 37, 80), (5, 2, 1, 12345, 50),
                               (3, 0, 5, 0, 16), (2**64 - 1, 2**32 - 1, 2**32 - 1, (1 << 40) + 3, 9)]:
        W = oracle.xi_words_range(seed, t, j, q0, q0 + nq)
        assert W.shape == (nq, 4) and W.dtype == np.uint32
        for r in range(nq):
            q = q0 + r
            assert [int(x) for x in W[r]] == bigint_philox([q & MASK, q >> 32, j, t], [seed & MASK, seed >> 32])
            assert np.array_equal(W[r], oracle.xi_words(seed, t, j, q))
        # neighbouring windows tile without overlap or gap
        assert np.array_equal(oracle.xi_words_range(seed, t, j, q0 + 3, q0 + nq), W[3:])


def test_box_muller_many_is_box_muller_row_by_row():
    rng = np.random.default_rng(99)
    words = rng.integers(0, 1 << 32, size=(400, 4), dtype=np.uint64).astype(np.uint32)
    words[0] = [0, 0, MASK, MASK]                       # extremes of radius and angle
    words[1] = [MASK, 0x40000000, 0x200, 0x80000000]
    Z = oracle.box_muller_many(words)
    assert Z.shape == (400, 4) and Z.dtype == np.float64
    two_pi = 2 * math.pi
    for r in range(400):
        assert np.array_equal(Z[r], oracle.box_muller(words[r]))
        # and against the closed form itself, written with the math module
        for pair in range(2):
            u1 = ((int(words[r, 2 * pair]) >> 9) + 0.5) / 2**23
            u2 = ((int(words[r, 2 * pair + 1]) >> 9) + 0.5) / 2**23
            rad = math.sqrt(-2.0 * math.log(u1))
            assert math.isclose(Z[r, 2 * pair], rad * math.cos(two_pi * u2), rel_tol=1e-12, abs_tol=1e-13)
            assert math.isclose(Z[r, 2 * pair + 1], rad * math.sin(two_pi * u2), rel_tol=1e-12, abs_tol=1e-13)
    # rows are independent of their neighbours: a permutation of the rows permutes the output
    perm = rng.permutation(400)
    assert np.array_equal(oracle.box_muller_many(words[perm]), Z[perm])
