"""Pins for the oracle's Stochastic Beam Search step (Algorithm 9, Eqs. 10-12, Theorem 3.2): CPU only."""
import itertools

import mpmath
import numpy as np
from scipy import stats

import oracle


def test_truncation_matches_eq_11_in_high_precision():
    mpmath.mp.dps = 60
    rng = np.random.default_rng(0)
    for _ in range(300):
        u = float(rng.normal(0, 5))
        z = float(rng.normal(0, 5))
        phi = z - float(rng.exponential(3.0))
        ref = -mpmath.log(mpmath.exp(-u) - mpmath.exp(-z) + mpmath.exp(-phi))
        got = oracle.truncated_gumbel(u, phi, z)
        assert abs(got - float(ref)) < 1e-12 * max(1.0, abs(float(ref)))
    # far-apart magnitudes where the printed formula would overflow in double
    for u, z, phi in [(-800.0, -790.0, -795.0), (700.0, 720.0, 100.0), (0.0, 5.0, -900.0)]:
        ref = -mpmath.log(mpmath.exp(-u) - mpmath.exp(-z) + mpmath.exp(-phi))
        assert abs(oracle.truncated_gumbel(u, phi, z) - float(ref)) < 1e-9 * max(1.0, abs(float(ref)))


def test_truncation_is_monotone_and_bounded_by_the_parent_value():
    rng = np.random.default_rng(1)
    for _ in range(100):
        u, z = float(rng.normal(0, 3)), float(rng.normal(0, 3))
        phis = np.sort(z - rng.exponential(2.0, 20))
        psi = np.array([oracle.truncated_gumbel(u, float(p), z) for p in phis])
        assert np.all(np.diff(psi) >= 0) and np.all(psi <= u)
        assert oracle.truncated_gumbel(u, z, z) == u       # the row maximum maps to the parent's value
    assert oracle.truncated_gumbel(0.0, -np.inf, 1.0) == -np.inf


def test_root_level_equals_gumbel_top_w_on_the_same_noise():
    rng = np.random.default_rng(2)
    rows = rng.normal(0, 2, (5, 1, 3000)).astype(np.float32)
    W = 6
    s = oracle.sbs_step(rows, W, 0, None, None, seed=7, step=1)
    g = oracle.gumbel_topk(rows, [W], [0], seed=7, step=1)
    assert np.array_equal(s["token"], g["token"][:, 0, :])
    assert np.all(s["parent"] == 0)
    assert np.allclose(s["sum_logprob"], g["logprob"][:, 0, :], atol=1e-12)
    assert np.allclose(s["trunc_gumbel"][:, 0], 0.0, atol=1e-12)   # psi of the best child = Gamma_root = 0
    assert np.all(np.diff(s["trunc_gumbel"], axis=1) < 0) and np.all(s["count"] == W)


def test_children_of_one_parent_are_a_prefix_of_its_own_order():
    # Theorem 3.2: the selected children of a parent, in stored order, are that parent's top picks by phi~.
    rng = np.random.default_rng(3)
    B, n_par, V, W = 6, 4, 2000, 4
    rows = rng.normal(0, 2, (B, n_par, V)).astype(np.float32)
    sig = -rng.exponential(2.0, (B, n_par))
    gam = np.sort(rng.normal(0, 1, (B, n_par)), axis=1)[:, ::-1].copy()
    first = 1
    s = oracle.sbs_step(rows, W, first, sig, gam, seed=11, step=0)
    g = oracle.gumbel_topk(rows, [W] * n_par, list(range(first, first + n_par)), seed=11, step=0)
    for b in range(B):
        for k in range(n_par):
            mine = [int(t) for t, p in zip(s["token"][b], s["parent"][b]) if p == k]
            assert mine == [int(t) for t in g["token"][b, k, :len(mine)]]
        assert np.all(np.diff(s["trunc_gumbel"][b]) <= 0)
        for i in range(W):
            k = s["parent"][b, i]
            assert s["trunc_gumbel"][b, i] <= gam[b, k] + 1e-12
            x = rows[b, k].astype(np.float64)
            logp = x - (x.max() + np.log(np.exp(x - x.max()).sum()))
            assert abs(s["sum_logprob"][b, i] - (sig[b, k] + logp[s["token"][b, i]])) < 1e-12


def test_beam_is_an_ordered_sample_of_sequences_without_replacement():
    # Section 3.2.1: top-W at a level == sampling W sequences of that length without replacement.
    rng = np.random.default_rng(4)
    V, W, n = 3, 3, 120000
    p1 = rng.dirichlet(np.ones(V))
    p2 = rng.dirichlet(np.ones(V), V)                      # p2[x1] = p(. | x1)
    root = np.broadcast_to(np.log(p1).astype(np.float32)[None, None, :], (n, 1, V))
    s0 = oracle.sbs_step(root, W, 0, None, None, seed=21, step=0, is_logprob=True)
    rows1 = np.log(p2).astype(np.float32)[s0["token"]]    # [n, W, V]: row of parent slot k = p(. | its token)
    s1 = oracle.sbs_step(rows1, W, 1, s0["sum_logprob"], s0["trunc_gumbel"], seed=21, step=0, is_logprob=True)
    first_tok = np.take_along_axis(s0["token"], s1["parent"], axis=1)
    seqs = first_tok * V + s1["token"]                     # leaf index of each selected sequence
    leaf_p = (p1[:, None] * p2).reshape(-1)
    tuples = list(itertools.permutations(range(V * V), W))
    index = {t: i for i, t in enumerate(tuples)}
    counts = np.zeros(len(tuples))
    for t in map(tuple, seqs):
        counts[index[t]] += 1
    expected = np.zeros(len(tuples))
    for i, t in enumerate(tuples):
        prob, rest = 1.0, 1.0
        for x in t:
            prob *= leaf_p[x] / rest
            rest -= leaf_p[x]
        expected[i] = prob * n
    big = expected >= 10
    obs = np.append(counts[big], counts[~big].sum())
    exp = np.append(expected[big], expected[~big].sum())
    assert stats.chisquare(obs, exp).pvalue > 1e-3
    # the sum log-probabilities carried forward are the sequences' log-probabilities
    assert np.allclose(s1["sum_logprob"], np.log(leaf_p)[seqs], atol=1e-5)


def test_minus_infinity_candidates_are_dropped():
    row = np.full((1, 2, 30), -np.inf, np.float32)
    row[0, 0, [2, 9]] = [0.0, 1.0]
    row[0, 1, 5] = 0.3
    s = oracle.sbs_step(row, 4, 1, np.zeros((1, 2)), np.array([[0.0, -0.5]]), seed=3, step=0)
    assert s["count"][0] == 3 and s["token"][0, 3] == -1 and s["status"][0] & oracle.ST_FEWER_THAN_K
    assert sorted(zip(s["parent"][0, :3].tolist(), s["token"][0, :3].tolist())) == [(0, 2), (0, 9), (1, 5)]
