"""Pins for the oracle's random-number layer (CPU only)."""
import math
import os

import numpy as np
from scipy import stats

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")
M0, M1 = 0xD2511F53, 0xCD9E8D57
W0, W1 = 0x9E3779B9, 0xBB67AE85
MASK = 0xFFFFFFFF


def test_philox_known_answers():
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        out = oracle.philox4x32_10(v[0:4], v[4:6])
        assert [int(x) for x in out] == v[6:10]


def _philox_inverse(out, key):
    """Undo the ten rounds: the multipliers are odd, hence invertible modulo 2^32."""
    inv0, inv1 = pow(M0, -1, 1 << 32), pow(M1, -1, 1 << 32)
    c = list(out)
    keys = [((key[0] + r * W0) & MASK, (key[1] + r * W1) & MASK) for r in range(10)]
    for r in reversed(range(10)):
        k0, k1 = keys[r]
        prev2 = (c[1] * inv1) & MASK          # lo(M1 * c2) = new c1
        prev0 = (c[3] * inv0) & MASK          # lo(M0 * c0) = new c3
        prev1 = c[0] ^ ((M1 * prev2) >> 32) ^ k0
        prev3 = c[2] ^ ((M0 * prev0) >> 32) ^ k1
        c = [prev0, prev1, prev2, prev3]
    return c


def test_philox_is_a_bijection_with_the_stated_round_structure():
    rng = np.random.default_rng(7)
    for _ in range(200):
        ctr = [int(x) for x in rng.integers(0, 1 << 32, 4, dtype=np.uint64)]
        key = [int(x) for x in rng.integers(0, 1 << 32, 2, dtype=np.uint64)]
        out = [int(x) for x in oracle.philox4x32_10(ctr, key)]
        assert _philox_inverse(out, key) == ctr


def test_philox_avalanche():
    rng = np.random.default_rng(11)
    flips = []
    for _ in range(300):
        ctr = [int(x) for x in rng.integers(0, 1 << 32, 4, dtype=np.uint64)]
        key = [int(x) for x in rng.integers(0, 1 << 32, 2, dtype=np.uint64)]
        a = oracle.philox4x32_10(ctr, key)
        w, bit = int(rng.integers(0, 4)), int(rng.integers(0, 32))
        ctr[w] ^= 1 << bit
        b = oracle.philox4x32_10(ctr, key)
        flips.append(sum(bin(int(x) ^ int(y)).count("1") for x, y in zip(a, b)))
    assert abs(np.mean(flips) - 64.0) < 1.5


def test_gumbel_stream_layout():
    """Group uniform (28 bits) and position (4 bits) from one word of the coarse stream, four groups 32 apart per
    call; element uniform from the fine stream, four elements per call."""
    seed, step, seq, node = 0x1234567811223344, 5, 17, 9
    key = [seed & MASK, seed >> 32]
    for e in [0, 1, 3, 4, 15, 16, 17, 511, 512, 1023, 1535, 1536, 2047, 2048, 2049, 31999, 50271]:
        g = e >> 4
        coarse = oracle.philox4x32_10([(g >> 7) * 32 + (g & 31), node | (0 << 28), seq, step], key)
        word = int(coarse[(g >> 5) & 3])
        fine = oracle.philox4x32_10([e >> 2, node | (1 << 28), seq, step], key)
        tg, a, te = oracle.gumbel_parts(seed, step, seq, node, e)
        assert math.isclose(tg, -math.log(((word >> 4) + 0.5) / 2.0 ** 28), rel_tol=1e-14)
        assert a == word & 15
        assert math.isclose(te, -math.log((int(fine[e & 3]) + 0.5) / 2.0 ** 32), rel_tol=1e-14)
        g_noise = oracle.gumbel(seed, step, seq, node, e)
        assert math.isclose(g_noise, -math.log(tg / 16 + (te if (e & 15) != a else 0.0)), rel_tol=1e-13)
    # every group of a row reads its own word: (call, word) pairs are distinct
    pairs = {((g >> 7) * 32 + (g & 31), (g >> 5) & 3) for g in range(4096)}
    assert len(pairs) == 4096


def test_streams_are_keyed_by_every_coordinate():
    base = oracle.gumbel(1, 2, 3, 4, 5)
    assert base != oracle.gumbel(2, 2, 3, 4, 5)
    assert base != oracle.gumbel(1 + (1 << 32), 2, 3, 4, 5)
    assert base != oracle.gumbel(1, 3, 3, 4, 5)
    assert base != oracle.gumbel(1, 2, 4, 4, 5)
    assert base != oracle.gumbel(1, 2, 3, 5, 5)
    assert base != oracle.gumbel(1, 2, 3, 4, 6)
    assert oracle.accept_uniform(1, 2, 3, 4, 0) != oracle.accept_uniform(1, 2, 3, 4, 1)
    assert oracle.accept_uniform(1, 2, 3, 4, 0) != oracle.accept_uniform(1, 2, 3, 4, 5)


def test_group_construction_gives_iid_gumbels():
    # The 16 noises of a group are built from their order statistics (largest first); they must come out i.i.d.
    # standard Gumbel: right marginal at every position, the group maximum distributed as Gumbel + ln 16, the
    # largest at a uniform position, no correlation between positions, and each pair ordered either way equally often.
    n = 20000
    G = np.array([[oracle.gumbel(77, 1, s, 3, 32 + j) for j in range(16)] for s in range(n)])
    cdf = lambda x: np.exp(-np.exp(-x))
    for j in (0, 5, 15):
        assert stats.kstest(G[:, j], cdf).pvalue > 1e-3
    assert stats.kstest(G.max(axis=1) - math.log(16.0), cdf).pvalue > 1e-3
    assert stats.kstest(np.sort(G, axis=1)[:, -2], lambda x: cdf(x) ** 15 * (16 - 15 * cdf(x))).pvalue > 1e-3
    pos = np.bincount(G.argmax(axis=1), minlength=16)
    assert stats.chisquare(pos).pvalue > 1e-3
    c = np.corrcoef(G.T)
    assert np.abs(c - np.eye(16)).max() < 0.04
    wins = (G[:, 2] > G[:, 9]).mean()
    assert abs(wins - 0.5) < 4 * 0.5 / math.sqrt(n)
    # the position named by the coarse stream really holds the largest noise
    for s in range(50):
        _, a, _ = oracle.gumbel_parts(77, 1, s, 3, 32)
        assert int(G[s].argmax()) == a


def test_gumbel_law():
    n = 200000
    g = np.array([oracle.gumbel(42, 0, i // 50000, 1 + i % 7, i) for i in range(n)])
    assert abs(g.mean() - 0.5772156649) < 4 * math.sqrt(math.pi ** 2 / 6 / n)
    assert abs(g.var() - math.pi ** 2 / 6) < 0.03
    ks = stats.kstest(g, lambda x: np.exp(-np.exp(-x)))
    assert ks.pvalue > 1e-3


def test_uniform_streams():
    n = 100000
    ua = np.array([oracle.accept_uniform(3, 1, i, 2, i % 5) for i in range(n)])
    ur = np.array([oracle.resample_uniform(3, 1, i, 2) for i in range(n)])
    assert ua.min() >= 0.0 and ua.max() < 1.0
    assert np.all(ua * 2 ** 24 == np.floor(ua * 2 ** 24))      # 24-bit grid, exactly representable in fp32
    assert ur.min() > 0.0 and ur.max() < 1.0
    assert stats.kstest(ua, "uniform").pvalue > 1e-3
    assert stats.kstest(ur, "uniform").pvalue > 1e-3
    assert abs(np.corrcoef(ua, ur)[0, 1]) < 0.02
    assert oracle.lib().rsd_oracle_rng_layout() == 3
