"""Pins for the oracle's two baseline verifiers (Section 2): multi-round rejection sampling with one draft model
and K-sequential selection (K-SEQ).  Both take K independent drafts from p and must return a token distributed as
q; the acceptance probabilities have closed forms.  CPU only."""
import itertools

import numpy as np
import pytest

import oracle


def _rand_dist(rng, V, zeros=0):
    p = rng.gamma(1.0, 1.0, V)
    if zeros:
        p[rng.choice(V, zeros, replace=False)] = 0.0
    return p / p.sum()


def _output_law(rule, p, q, K, gamma=1.0):
    """Exact law of the emitted token when the K drafts are independent draws from p (all V^K tuples)."""
    V = len(p)
    law = np.zeros(V)
    accept_total = 0.0
    for tup in itertools.product(range(V), repeat=K):
        w = float(np.prod([p[x] for x in tup]))
        if w == 0.0:
            continue
        theta, residual, _ = oracle.baseline_chain(rule, p, q, tup, gamma)
        alive = 1.0
        for k, x in enumerate(tup):
            law[x] += w * alive * theta[k]
            accept_total += w * alive * theta[k]
            alive *= 1.0 - theta[k]
        law += w * alive * residual
    return law, accept_total


@pytest.mark.parametrize("V,K", [(2, 1), (3, 2), (4, 3), (5, 3), (6, 2)])
def test_multiround_output_is_target_distributed(V, K):
    rng = np.random.default_rng(7 * V + K)
    for trial in range(3):
        p = _rand_dist(rng, V)
        q = _rand_dist(rng, V, zeros=(trial % 2) * (V > 3))
        law, _ = _output_law(oracle.RULE_MULTIROUND, p, q, K)
        assert np.allclose(law, q, atol=1e-12)


def test_multiround_first_round_is_speculative_sampling_and_draft_is_kept():
    rng = np.random.default_rng(3)
    p, q = _rand_dist(rng, 6), _rand_dist(rng, 6)
    theta, residual, _ = oracle.baseline_chain(oracle.RULE_MULTIROUND, p, q, [2, 2])
    assert abs(theta[0] - min(1.0, q[2] / p[2])) < 1e-15
    q2 = np.maximum(q - p, 0.0)
    q2 /= q2.sum()
    # the same token may be drawn again: its second threshold uses the residual and the unchanged draft
    assert abs(theta[1] - min(1.0, q2[2] / p[2])) < 1e-15
    q3 = np.maximum(q2 - p, 0.0)
    assert np.allclose(residual, q3 / q3.sum(), atol=1e-15)
    # recursive rejection sampling differs here: it removes token 2 from the draft after the first rejection
    theta_rrs, _, _ = oracle.rrs_chain(p, q, [2, 3])
    theta_mr, _, _ = oracle.baseline_chain(oracle.RULE_MULTIROUND, p, q, [2, 3])
    assert theta_rrs[0] == theta_mr[0]
    if q2[3] > 0 and theta_mr[1] < 1.0:
        assert theta_rrs[1] < theta_mr[1]                  # p(3) / (1 - p(2)) > p(3) lowers the ratio


@pytest.mark.parametrize("V,K", [(3, 2), (4, 3), (5, 2), (5, 3)])
def test_kseq_output_is_target_distributed_and_acceptance_closed_form(V, K):
    rng = np.random.default_rng(11 * V + K)
    for trial in range(3):
        p, q = _rand_dist(rng, V), _rand_dist(rng, V, zeros=(trial % 2) * (V > 3))
        # gamma = K is always admissible; smaller values are admissible when (1 - (1 - beta)^K) / beta <= gamma
        gammas = [float(K)]
        for g in (1.0, 1.5, 2.0):
            beta = np.minimum(p, q / g).sum()
            if g <= K and (1 - (1 - beta) ** K) / beta <= g + 1e-12:
                gammas.append(g)
        for g in gammas:
            law, acc = _output_law(oracle.RULE_KSEQ, p, q, K, g)
            assert np.allclose(law, q, atol=1e-12), (g, law, q)
            beta = np.minimum(p, q / g).sum()
            assert abs(acc - (1 - (1 - beta) ** K)) < 1e-12    # each draft is accepted with probability beta


def test_kseq_with_one_draft_and_gamma_one_is_speculative_sampling():
    rng = np.random.default_rng(13)
    p, q = _rand_dist(rng, 7), _rand_dist(rng, 7)
    for x in range(7):
        theta, residual, _ = oracle.baseline_chain(oracle.RULE_KSEQ, p, q, [x], 1.0)
        assert abs(theta[0] - min(1.0, q[x] / p[x])) < 1e-15
        r = np.maximum(q - p, 0.0)
        assert np.allclose(residual, r / r.sum(), atol=1e-15)


def test_verify_tree_rules_on_a_star_tree():
    # root with K children drawn independently from the draft (a repeat included): the walk's thresholds equal the
    # chain's, and the three rules agree on the first child and differ afterwards
    rng = np.random.default_rng(17)
    V, K = 40, 3
    draft = rng.normal(0, 1.5, (1, 1, V)).astype(np.float32)
    target = (draft[:, :1] + rng.normal(0, 1.0, (1, 1 + K, V))).astype(np.float32)
    parent = np.array([-1, 0, 0, 0], np.int32)
    p = np.exp(draft[0, 0].astype(np.float64)); p /= p.sum()
    q = np.exp(target[0, 0].astype(np.float64)); q /= q.sum()
    toks = [int(np.argmax(p)), int(np.argmax(p)), int(np.argsort(p)[-2])]
    token = np.array([[-1] + toks], np.int32)
    seen = {}
    for rule, gamma in ((oracle.RULE_RRS, 1.0), (oracle.RULE_MULTIROUND, 1.0), (oracle.RULE_KSEQ, 2.0)):
        # find a seed whose walk rejects all three children, so that every threshold is exercised
        for seed in range(200):
            out = oracle.verify_tree(draft, target, parent, token, 1, seed=seed, step=0, rule=rule, gamma=gamma,
                                     want_weights=True)
            if out["stop_reason"][0] == 0:
                break
        assert out["stop_reason"][0] == 0
        th = out["theta"][0, 1:]
        if rule == oracle.RULE_RRS:
            # the repeat of a removed token has draft probability 0 and no residual mass: threshold 0
            ref, res, _ = oracle.rrs_chain(p, q, toks)
        else:
            ref, res, _ = oracle.baseline_chain(rule, p, q, toks, gamma)
        assert np.allclose(th, ref, atol=1e-12)
        assert np.allclose(out["final_weights"][0], res, atol=1e-12)
        seen[rule] = th
    assert seen[oracle.RULE_RRS][0] == seen[oracle.RULE_MULTIROUND][0]
    assert seen[oracle.RULE_KSEQ][0] <= seen[oracle.RULE_MULTIROUND][0]
