"""Pins for the oracle's sampling temperature (Section 4 samples at temperature 0.3 or 1.0): CPU only.

Temperature T divides a row before anything else: drafting and verification then see softmax(row / T)."""
import numpy as np
from scipy import stats

import oracle
import workloads


def _softmax(x):
    x = np.asarray(x, np.float64)
    e = np.exp(x - x.max())
    return e / e.sum()


def test_half_temperature_equals_doubled_rows_exactly():
    # dividing by 0.5 and multiplying by 2 are both exact, so every output must agree to the last bit
    rng = np.random.default_rng(0)
    rows = rng.normal(0, 1.5, (3, 4, 300)).astype(np.float32)
    a = oracle.gumbel_topk(rows, [3, 2, 1, 4], [0, 1, 2, 3], seed=5, step=1, max_k=4, temperature=0.5)
    b = oracle.gumbel_topk(rows * np.float32(2), [3, 2, 1, 4], [0, 1, 2, 3], seed=5, step=1, max_k=4)
    for key in ("token", "perturbed", "logprob"):
        assert np.array_equal(a[key], b[key])
    sig = rng.normal(-3, 1, (3, 4))
    gam = rng.normal(0, 1, (3, 4))
    a = oracle.sbs_step(rows, 4, 1, sig, gam, seed=5, step=1, temperature=0.5)
    b = oracle.sbs_step(rows * np.float32(2), 4, 1, sig, gam, seed=5, step=1)
    for key in ("token", "parent", "sum_logprob", "trunc_gumbel"):
        assert np.array_equal(a[key], b[key])
    branching = (2, 2)
    parent = workloads.rsdc_parent_array(branching)
    draft = rng.normal(0, 1.5, (5, 3, 64)).astype(np.float32)
    target = (np.concatenate([draft, rng.normal(0, 1.5, (5, 4, 64)).astype(np.float32)], 1)
              + rng.normal(0, 0.7, (5, 7, 64)).astype(np.float32))
    k, nodes = workloads.rsdc_rows(branching)
    d = oracle.gumbel_topk(draft, k, nodes, seed=2, step=0, temperature=0.5)
    token = workloads.rsdc_tokens_from_rows(branching, d["token"])
    a = oracle.verify_tree(draft, target, parent, token, 2, seed=2, step=0, draft_temperature=0.5,
                           target_temperature=0.5)
    b = oracle.verify_tree(draft * np.float32(2), target * np.float32(2), parent, token, 2, seed=2, step=0)
    for key in ("accepted_len", "accepted_node", "last_token", "stop_reason"):
        assert np.array_equal(a[key], b[key])
    assert np.array_equal(np.nan_to_num(a["theta"], nan=-1.0), np.nan_to_num(b["theta"], nan=-1.0))


def test_first_pick_follows_the_tempered_softmax():
    rng = np.random.default_rng(1)
    V, n, T = 40, 60000, 0.3
    logits = rng.normal(0, 1.0, V).astype(np.float32)
    p = _softmax(logits.astype(np.float64) / T)
    rows = np.broadcast_to(logits[None, None, :], (n, 1, V))
    out = oracle.gumbel_topk(rows, [1], [0], seed=11, step=0, temperature=T)
    counts = np.bincount(out["token"][:, 0, 0], minlength=V).astype(float)
    keep = p * n > 5
    obs = np.append(counts[keep], counts[~keep].sum())
    exp = np.append(p[keep] * n, p[~keep].sum() * n)
    assert stats.chisquare(obs, exp).pvalue > 1e-3
    # the returned log-probability is that of the tempered distribution
    x = int(out["token"][0, 0, 0])
    assert abs(out["logprob"][0, 0, 0] - np.log(p[x])) < 1e-9
    # it is much more peaked than at temperature 1
    assert p.max() > 2 * _softmax(logits).max()


def test_log_probability_rows_are_rescored_under_a_temperature():
    # log-softmax rows divided by T differ from logits / T by a per-row constant only: same picks, same log-probs
    rng = np.random.default_rng(2)
    x = rng.normal(0, 2, (2, 2, 500)).astype(np.float32)
    lp = (x - np.log(np.exp(x.astype(np.float64)).sum(-1, keepdims=True))).astype(np.float32)
    a = oracle.gumbel_topk(lp, [3, 3], [0, 1], seed=3, step=0, is_logprob=True, temperature=0.3)
    b = oracle.gumbel_topk(x, [3, 3], [0, 1], seed=3, step=0, temperature=0.3)
    assert np.array_equal(a["token"], b["token"])
    assert np.allclose(a["logprob"], b["logprob"], atol=2e-5)      # fp32 rounding of the stored log-probs, / 0.3
    # and temperature 1 (or 0, meaning none) leaves log-probability rows untouched
    c = oracle.gumbel_topk(lp, [3, 3], [0, 1], seed=3, step=0, is_logprob=True, temperature=1.0)
    d = oracle.gumbel_topk(lp, [3, 3], [0, 1], seed=3, step=0, is_logprob=True, temperature=0.0)
    assert np.array_equal(c["token"], d["token"]) and np.array_equal(c["logprob"], d["logprob"])


def test_acceptance_threshold_uses_both_temperatures():
    # chain tree, first child: theta = min(1, q_T(x) / p_T(x)) with each row tempered by its own temperature
    rng = np.random.default_rng(3)
    B, V = 50, 30
    draft = rng.normal(0, 1.5, (B, 1, V)).astype(np.float32)
    target = rng.normal(0, 1.5, (B, 2, V)).astype(np.float32)
    parent = np.array([-1, 0], np.int32)
    token = np.stack([np.full(B, -1), rng.integers(0, V, B)], 1).astype(np.int32)
    out = oracle.verify_tree(draft, target, parent, token, 1, seed=4, step=0, draft_temperature=0.3,
                             target_temperature=0.7)
    for b in range(B):
        p = _softmax(draft[b, 0].astype(np.float64) / 0.3)
        q = _softmax(target[b, 0].astype(np.float64) / 0.7)
        x = token[b, 1]
        assert abs(out["theta"][b, 1] - min(1.0, q[x] / p[x])) < 1e-12
    res = oracle.resample_residual(None, target[:, 0], None, np.zeros(B, np.int32), seed=4, step=0,
                                   target_temperature=0.7)
    for b in range(B):
        assert np.allclose(res["residual"][b], _softmax(target[b, 0].astype(np.float64) / 0.7), atol=1e-15)
