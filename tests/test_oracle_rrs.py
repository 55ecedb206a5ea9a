"""Pins for the oracle's recursive rejection sampling (Algorithm 1, Eqs. 1-4, Theorem 3.1): CPU only."""
import itertools

import numpy as np
import pytest

import oracle


def _rand_dist(rng, V, zeros=0):
    p = rng.gamma(1.0, 1.0, V)
    if zeros:
        p[rng.choice(V, zeros, replace=False)] = 0.0
    return p / p.sum()


def _output_law(p, q, K):
    """Exact law of Z (Eq. 4) when the drafts are an ordered sample without replacement from p."""
    V = len(p)
    support = [x for x in range(V) if p[x] > 0]
    law = np.zeros(V)
    accept_total = 0.0
    for tup in itertools.permutations(support, K):
        w, rest = 1.0, 1.0
        for x in tup:
            w *= p[x] / rest
            rest -= p[x]
        theta, residual, _ = oracle.rrs_chain(p, q, tup)
        alive = 1.0
        for k, x in enumerate(tup):
            law[x] += w * alive * theta[k]
            accept_total += w * alive * theta[k]
            alive *= 1.0 - theta[k]
        law += w * alive * residual
    return law, accept_total


@pytest.mark.parametrize("V,K", [(2, 1), (3, 2), (4, 2), (4, 3), (5, 3), (6, 3), (6, 2)])
def test_theorem_3_1_output_is_target_distributed(V, K):
    rng = np.random.default_rng(100 * V + K)
    for trial in range(4):
        p = _rand_dist(rng, V)
        q = _rand_dist(rng, V, zeros=(trial % 2) * (V > 3))
        law, _ = _output_law(p, q, K)
        assert np.allclose(law, q, atol=1e-12)


def test_theorem_3_1_when_draft_equals_target():
    rng = np.random.default_rng(5)
    p = _rand_dist(rng, 5)
    law, acc = _output_law(p, p.copy(), 2)
    assert np.allclose(law, p, atol=1e-12)
    assert abs(acc - 1.0) < 1e-12                          # theta = 1 at the first draft


def test_k1_is_ordinary_speculative_sampling():
    # Section 2: accept with min(1, q/p), else draw from Norm[(q - p)+]; acceptance probability sum min(p, q)
    rng = np.random.default_rng(6)
    for V in (3, 7, 50):
        p, q = _rand_dist(rng, V), _rand_dist(rng, V)
        acc = 0.0
        for x in range(V):
            theta, residual, _ = oracle.rrs_chain(p, q, [x])
            assert abs(theta[0] - min(1.0, q[x] / p[x])) < 1e-15
            r = np.maximum(q - p, 0.0)
            assert np.allclose(residual, r / r.sum(), atol=1e-15)
            acc += p[x] * theta[0]
        assert abs(acc - np.minimum(p, q).sum()) < 1e-12


def test_bernoulli_toy_k2_always_accepts():
    # Section 3.1, toy example: two drafts without replacement from Ber(p) against Ber(q) are never both rejected
    for a in np.linspace(0.02, 0.98, 13):
        for b in np.linspace(0.02, 0.98, 13):
            p, q = np.array([1 - a, a]), np.array([1 - b, b])
            _, acc = _output_law(p, q, 2)
            assert abs(acc - 1.0) < 1e-12


def test_second_draft_uses_the_draft_that_generated_the_first():
    # Eq. 2 forms the residual with p^(1) (before removal); Eq. 1 then conditions p^(2) on the removed token.
    p = np.array([0.5, 0.3, 0.2])
    q = np.array([0.2, 0.3, 0.5])
    theta, residual, _ = oracle.rrs_chain(p, q, [0, 1])
    assert abs(theta[0] - 0.4) < 1e-15
    q2 = np.array([0.0, 0.0, 1.0])                         # Norm[(q - p)+] = (0, 0, 0.3) / 0.3
    p2 = np.array([0.0, 0.6, 0.4])                         # p without token 0, renormalised
    assert abs(theta[1] - min(1.0, q2[1] / p2[1])) < 1e-15
    r = np.maximum(q2 - p2, 0.0)
    assert np.allclose(residual, r / r.sum())


def test_residual_closed_form_identity():
    # q^(j+1) = Norm[(q - A_j p)+] with A_{j+1} = A_j + Z_j / (1 - P_j), Z_j = sum (q - A_j p)+, P_j = removed mass.
    rng = np.random.default_rng(8)
    for V, K in [(6, 3), (20, 5), (200, 8)]:
        p, q = _rand_dist(rng, V), _rand_dist(rng, V)
        # order the tokens as a sample without replacement would likely do; any order satisfies the identity
        tokens = list(rng.choice(V, K, replace=False, p=p))
        theta, residual, _ = oracle.rrs_chain(p, q, tokens)
        A, P, Z = 0.0, 0.0, 1.0
        for j, x in enumerate(tokens):
            r_x = max(q[x] - A * p[x], 0.0)
            th = min(1.0, r_x * (1.0 - P) / (Z * p[x]))
            assert abs(th - theta[j]) < 1e-12
            if th >= 1.0:
                # an accepted-for-sure token is "rejected" by the chain function anyway; the identity for later
                # residuals needs theta < 1 (a rejected token has zero residual mass), so stop here
                break
            A = A + Z / (1.0 - P)
            P = P + p[x]
            Z = np.maximum(q - A * p, 0.0).sum()
        else:
            r = np.maximum(q - A * p, 0.0)
            assert np.allclose(residual, r / r.sum(), atol=1e-12)


def test_degenerate_inputs_set_status_bits():
    p = np.array([0.5, 0.5, 0.0])
    q = np.array([0.2, 0.3, 0.5])
    theta, _, st = oracle.rrs_chain(p, q, [2])
    assert theta[0] == 1.0 and st & oracle.ST_ZERO_DRAFT_PROB
    theta, residual, st = oracle.rrs_chain(p, p.copy(), [0])
    assert theta[0] == 1.0 and st & oracle.ST_ZERO_RESIDUAL and np.allclose(residual, p)
    theta, _, st = oracle.rrs_chain(np.array([1.0, 0.0]), np.array([0.5, 0.5]), [0, 1])
    assert st & oracle.ST_DRAFT_EXHAUSTED and theta[1] == 0.0
