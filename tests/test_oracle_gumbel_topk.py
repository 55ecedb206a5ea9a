"""Pins for the oracle's Gumbel-Top-k drafting (Algorithm 4, Eqs. 5-7): CPU only."""
import itertools

import numpy as np
from scipy import stats

import oracle


def _plackett_luce(p, tup):
    """Probability of drawing `tup` in order, without replacement, from p."""
    prob, rest = 1.0, 1.0
    for x in tup:
        prob *= p[x] / rest
        rest -= p[x]
    return prob


def _broadcast_rows(row, B):
    return np.broadcast_to(row.astype(np.float32)[None, None, :], (B, 1, row.shape[0]))


def test_ordered_picks_follow_sampling_without_replacement_small_vocab():
    # Section 3.2.1: the b_l picks, in decreasing perturbed order, are an ordered sample without replacement.
    rng = np.random.default_rng(0)
    V, k, n = 5, 3, 60000
    logits = rng.normal(0, 1.5, V)
    p = np.exp(logits) / np.exp(logits).sum()
    out = oracle.gumbel_topk(_broadcast_rows(logits, n), [k], [3], seed=99, step=0)
    tuples = list(itertools.permutations(range(V), k))
    index = {t: i for i, t in enumerate(tuples)}
    counts = np.zeros(len(tuples))
    for t in map(tuple, out["token"][:, 0, :]):
        counts[index[t]] += 1
    expected = np.array([_plackett_luce(p, t) for t in tuples]) * n
    assert expected.min() > 5
    assert stats.chisquare(counts, expected).pvalue > 1e-3


def test_first_and_second_pick_law_vocab_50():
    rng = np.random.default_rng(1)
    V, n = 50, 80000
    logits = rng.normal(0, 2.0, V)
    p = np.exp(logits) / np.exp(logits).sum()
    out = oracle.gumbel_topk(_broadcast_rows(logits, n), [2], [0], seed=5, step=3)
    first = np.bincount(out["token"][:, 0, 0], minlength=V).astype(float)
    keep = p * n > 5
    obs = np.append(first[keep], first[~keep].sum())
    exp = np.append(p[keep] * n, p[~keep].sum() * n)
    assert stats.chisquare(obs, exp).pvalue > 1e-3
    # second pick given the first: p(y) / (1 - p(x)); marginal over x
    second = np.bincount(out["token"][:, 0, 1], minlength=V).astype(float)
    marg = np.array([sum(p[x] * p[y] / (1 - p[x]) for x in range(V) if x != y) for y in range(V)])
    obs2 = np.append(second[keep], second[~keep].sum())
    exp2 = np.append(marg[keep] * n, marg[~keep].sum() * n)
    assert stats.chisquare(obs2, exp2).pvalue > 1e-3
    assert np.all(out["token"][:, 0, 0] != out["token"][:, 0, 1])


def test_top1_is_argmax_of_logprob_plus_gumbel():
    rng = np.random.default_rng(2)
    B, R, V = 3, 2, 257
    rows = rng.normal(0, 2, (B, R, V)).astype(np.float32)
    nodes = [4, 11]
    out = oracle.gumbel_topk(rows, [1, 1], nodes, seed=8, step=2, seq_base=10)
    for b in range(B):
        for r in range(R):
            x = rows[b, r].astype(np.float64)
            logp = x - (x.max() + np.log(np.exp(x - x.max()).sum()))
            pert = np.array([logp[e] + oracle.gumbel(8, 2, 10 + b, nodes[r], e) for e in range(V)])
            assert out["token"][b, r, 0] == int(np.argmax(pert))
            assert abs(out["perturbed"][b, r, 0] - pert.max()) < 1e-12
            assert abs(out["logprob"][b, r, 0] - logp[np.argmax(pert)]) < 1e-12


def test_sorted_decreasing_and_shift_invariant():
    rng = np.random.default_rng(3)
    rows = rng.normal(0, 2, (4, 3, 1000)).astype(np.float32)
    a = oracle.gumbel_topk(rows, [4, 2, 3], [0, 1, 2], seed=1, step=0, max_k=4)
    b = oracle.gumbel_topk(rows + np.float32(2.0), [4, 2, 3], [0, 1, 2], seed=1, step=0, max_k=4)
    assert np.array_equal(a["token"], b["token"])          # argtop is invariant to the row constant
    assert np.all(np.diff(a["perturbed"][:, 0, :], axis=-1) < 0)
    assert np.all(a["token"][:, 1, 2:] == -1) and np.all(a["token"][:, 2, 3:] == -1)
    assert np.all(a["margin"] > 0)
    # log-probabilities given as such are used as they are
    x = rows.astype(np.float64)
    lse = np.log(np.exp(x - x.max(-1, keepdims=True)).sum(-1, keepdims=True)) + x.max(-1, keepdims=True)
    c = oracle.gumbel_topk((x - lse).astype(np.float32), [4, 2, 3], [0, 1, 2], seed=1, step=0, max_k=4,
                           is_logprob=True)
    assert np.mean(a["token"] == c["token"]) > 0.95        # equal up to the fp32 rounding of the log-probs


def test_noise_is_per_node_and_per_sequence():
    row = np.zeros(4000, np.float32)
    rows = np.broadcast_to(row[None, None, :], (2, 2, 4000))
    out = oracle.gumbel_topk(rows, [3, 3], [1, 2], seed=4, step=0)
    picks = {tuple(out["token"][b, r]) for b in range(2) for r in range(2)}
    assert len(picks) == 4


def test_minus_infinity_and_nan_are_never_selected():
    row = np.full(40, -np.inf, np.float32)
    row[[3, 17]] = [0.5, 1.5]
    row[20] = np.nan
    out = oracle.gumbel_topk(row[None, None, :], [4], [0], seed=0, step=0)
    assert set(out["token"][0, 0, :2]) == {3, 17} and np.all(out["token"][0, 0, 2:] == -1)
    assert out["status"][0] & oracle.ST_FEWER_THAN_K and out["status"][0] & oracle.ST_NAN_INPUT


def test_bf16_rows_widen_exactly():
    rng = np.random.default_rng(4)
    x = rng.normal(0, 2, (2, 2, 500)).astype(np.float32)
    bits = (x.view(np.uint32) >> 16).astype(np.uint16)                  # truncate to a bf16 pattern
    widened = (bits.astype(np.uint32) << 16).view(np.float32)
    a = oracle.gumbel_topk(bits, [3, 3], [0, 1], seed=2, step=1)
    b = oracle.gumbel_topk(widened, [3, 3], [0, 1], seed=2, step=1)
    assert np.array_equal(a["token"], b["token"]) and np.array_equal(a["perturbed"], b["perturbed"])
