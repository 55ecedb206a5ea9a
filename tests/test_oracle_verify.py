"""Pins for the oracle's tree verification walk (Section 3.2.2, Algorithm 6) and final-token draw: CPU only."""
import numpy as np
from scipy import stats

import oracle
import workloads


def _softmax(x):
    x = x.astype(np.float64)
    e = np.exp(x - x.max())
    return e / e.sum()


def test_inverse_cdf_edges():
    w = np.array([0.0, 0.25, 0.0, 0.5, 0.25, 0.0])
    assert oracle.inverse_cdf(w, 1e-9)[0] == 1
    assert oracle.inverse_cdf(w, 0.25)[0] == 3            # a running sum equal to u*total is not "greater"
    assert oracle.inverse_cdf(w, 0.2499999)[0] == 1
    assert oracle.inverse_cdf(w, 0.75)[0] == 4
    assert oracle.inverse_cdf(w, 0.999999)[0] == 4        # never a zero-weight token
    y, m = oracle.inverse_cdf(w * 7.0, 0.5)               # unnormalised weights; margin relative to the total
    assert y == 3 and abs(m - 0.25) < 1e-12
    rng = np.random.default_rng(0)
    p = rng.dirichlet(np.ones(40))
    us = (np.arange(200000) + 0.5) / 200000
    draws = np.array([oracle.inverse_cdf(p, u)[0] for u in us])
    assert np.allclose(np.bincount(draws, minlength=40) / len(us), p, atol=2e-5)


def test_chain_tree_is_single_sequence_speculative_decoding():
    # Section 2: with one draft per level the walk accepts each token with min(1, q/p), stops at the first
    # rejection with a draw from Norm[(q - p)+], and draws a bonus token from q after L acceptances.
    rng = np.random.default_rng(1)
    B, V, L = 200, 30, 3
    draft = rng.normal(0, 1.5, (B, L, V)).astype(np.float32)
    target = (np.concatenate([draft, rng.normal(0, 1.5, (B, 1, V)).astype(np.float32)], 1)
              + rng.normal(0, 1.0, (B, L + 1, V)).astype(np.float32))
    parent = np.array([-1, 0, 1, 2], np.int32)
    token = np.concatenate([np.full((B, 1), -1), rng.integers(0, V, (B, L))], 1).astype(np.int32)
    out = oracle.verify_tree(draft, target, parent, token, L, seed=77, step=4, seq_base=1000)
    n_full = 0
    for b in range(B):
        cur, acc = 0, []
        weights = None
        for l in range(L):
            p, q = _softmax(draft[b, cur]), _softmax(target[b, cur])
            x = token[b, l + 1]
            u = oracle.accept_uniform(77, 4, 1000 + b, cur, 0)
            if u < min(1.0, q[x] / p[x]):
                acc.append(l + 1)
                cur = l + 1
            else:
                r = np.maximum(q - p, 0.0)
                weights = r / r.sum()
                break
        if weights is None:
            weights = _softmax(target[b, cur])
            n_full += 1
            assert out["stop_reason"][b] == oracle.STOP_LEAF
        else:
            assert out["stop_reason"][b] == oracle.STOP_ALL_REJECTED
        assert out["accepted_len"][b] == len(acc)
        assert list(out["accepted_node"][b, :len(acc)]) == acc
        assert list(out["accepted_token"][b, :len(acc)]) == [token[b, n] for n in acc]
        assert np.all(out["accepted_node"][b, len(acc):] == -1)
        last, _ = oracle.inverse_cdf(weights, oracle.resample_uniform(77, 4, 1000 + b, cur))
        assert out["last_token"][b] == last
    assert 0 < n_full < B


def test_identical_draft_and_target_accepts_everything():
    rng = np.random.default_rng(2)
    b = (2, 2)
    parent = workloads.rsdc_parent_array(b)
    B, V = 5, 64
    rows = rng.normal(0, 2, (B, 7, V)).astype(np.float32)
    k, nodes = workloads.rsdc_rows(b)
    d = oracle.gumbel_topk(rows[:, :3], k, nodes, seed=3, step=0)
    token = workloads.rsdc_tokens_from_rows(b, d["token"])
    out = oracle.verify_tree(rows[:, :3], rows, parent, token, 2, seed=3, step=0, want_weights=True)
    assert np.all(out["accepted_len"] == 2) and np.all(out["stop_reason"] == oracle.STOP_LEAF)
    assert np.all(out["accepted_node"][:, 0] == 1) and np.all(out["accepted_node"][:, 1] == 3)  # always the first child
    for s in range(B):
        leaf = out["accepted_node"][s, 1]
        assert np.allclose(out["final_weights"][s], _softmax(rows[s, leaf]), atol=1e-15)
        assert out["last_token"][s] == oracle.inverse_cdf(_softmax(rows[s, leaf]),
                                                          oracle.resample_uniform(3, 0, s, int(leaf)))[0]


def test_node_without_children_draws_from_its_target_row():
    rng = np.random.default_rng(3)
    V = 20
    parent = np.array([[-1, 0, 0, 1, 1]], np.int32)        # per-sequence topology; node 2 has no children
    token = np.array([[-1, 4, 7, 1, -1]], np.int32)        # node 4 is absent
    draft = rng.normal(0, 1, (1, 3, V)).astype(np.float32)
    target = rng.normal(0, 1, (1, 5, V)).astype(np.float32)
    # force: child 1 (token 4) rejected, child 2 (token 7) accepted -> lands on node 2, which is childless
    target[0, 0, 4] = -30.0
    target[0, 0, 7] = 30.0
    out = oracle.verify_tree(draft, target, parent, token, 2, seed=1, step=0, want_weights=True)
    assert out["accepted_len"][0] == 1 and out["accepted_node"][0, 0] == 2 and out["accepted_token"][0, 0] == 7
    assert out["stop_reason"][0] == oracle.STOP_NO_CHILDREN
    assert np.allclose(out["final_weights"][0], _softmax(target[0, 2]), atol=1e-15)
    assert not np.isnan(out["theta"][0, 1]) and not np.isnan(out["theta"][0, 2]) and np.isnan(out["theta"][0, 3])
    # absent children are skipped: making node 3 absent as well leaves node 1 childless too
    token2 = token.copy()
    token2[0, 2] = -1
    target2 = target.copy()
    target2[0, 0, 4] = 30.0
    out2 = oracle.verify_tree(draft, target2, parent, token2, 2, seed=1, step=0)
    assert out2["accepted_node"][0, 0] == 1 and out2["accepted_len"][0] == 2 and out2["accepted_node"][0, 1] == 3


def test_first_emitted_token_is_target_distributed_vocab_50():
    # Theorem 3.1 through the whole pipeline: drafts by Gumbel-Top-k (3 children of the root), verification by the
    # walk, randomness from the counter streams.  The first new token must follow q(. | root).
    rng = np.random.default_rng(4)
    V, n, K = 50, 60000, 3
    ld = rng.normal(0, 1.5, V).astype(np.float32)
    lt = (ld + rng.normal(0, 1.0, V)).astype(np.float32)
    q = _softmax(lt)
    draft = np.broadcast_to(ld[None, None, :], (n, 1, V))
    target = np.broadcast_to(lt[None, None, :], (n, 1 + K, V))
    parent = np.array([-1, 0, 0, 0], np.int32)
    d = oracle.gumbel_topk(draft, [K], [0], seed=9, step=2)
    token = np.concatenate([np.full((n, 1), -1, np.int32), d["token"][:, 0, :]], 1)
    out = oracle.verify_tree(draft, target, parent, token, 1, seed=9, step=2)
    first = np.where(out["accepted_len"] > 0, out["accepted_token"][:, 0], out["last_token"])
    counts = np.bincount(first, minlength=V).astype(float)
    keep = q * n > 5
    obs = np.append(counts[keep], counts[~keep].sum())
    exp = np.append(q[keep] * n, q[~keep].sum() * n)
    assert stats.chisquare(obs, exp).pvalue > 1e-3
    # acceptance is far more likely than with one draft (K = 1 accepts with sum min(p, q))
    assert (out["accepted_len"] > 0).mean() > np.minimum(_softmax(ld), q).sum() + 0.05


def test_two_level_joint_law_small_vocab():
    # Two levels, V = 4: the pair (first token, second token) must follow q(x1 | root) q(x2 | x1's node row).
    # Rows are attached to node slots, so condition on the slot: check the first token's law and that, given
    # the walk reached slot s, the next emitted token follows slot s's target row.
    rng = np.random.default_rng(5)
    V, n = 4, 80000
    b = (2, 2)
    parent = workloads.rsdc_parent_array(b)
    drow = rng.normal(0, 1, (3, V)).astype(np.float32)
    trow = (np.concatenate([drow, rng.normal(0, 1, (4, V)).astype(np.float32)], 0)
            + rng.normal(0, 0.8, (7, V)).astype(np.float32))
    draft = np.broadcast_to(drow[None], (n, 3, V))
    target = np.broadcast_to(trow[None], (n, 7, V))
    k, nodes = workloads.rsdc_rows(b)
    d = oracle.gumbel_topk(draft, k, nodes, seed=31, step=0)
    token = workloads.rsdc_tokens_from_rows(b, d["token"])
    out = oracle.verify_tree(draft, target, parent, token, 2, seed=31, step=0)
    first = np.where(out["accepted_len"] > 0, out["accepted_token"][:, 0], out["last_token"])
    assert stats.chisquare(np.bincount(first, minlength=V), _softmax(trow[0]) * n).pvalue > 1e-3
    for slot in (1, 2):
        sel = (out["accepted_len"] >= 1) & (out["accepted_node"][:, 0] == slot)
        second = np.where(out["accepted_len"][sel] > 1, out["accepted_token"][sel, 1], out["last_token"][sel])
        assert sel.sum() > 5000
        assert stats.chisquare(np.bincount(second, minlength=V), _softmax(trow[slot]) * sel.sum()).pvalue > 1e-3


def test_resample_residual_entry():
    rng = np.random.default_rng(6)
    B, V = 6, 40
    d = rng.normal(0, 1, (B, V)).astype(np.float32)
    t = (d + rng.normal(0, 1, (B, V))).astype(np.float32)
    nodes = np.arange(B, dtype=np.int32) + 2
    plain = oracle.resample_residual(None, t, None, nodes, seed=5, step=1)
    for b in range(B):
        assert np.allclose(plain["residual"][b], _softmax(t[b]), atol=1e-15)
        assert plain["token"][b] == oracle.inverse_cdf(_softmax(t[b]), oracle.resample_uniform(5, 1, b, int(nodes[b])))[0]
    rej = np.array([[3, 8, -1]] * B, np.int32)
    res = oracle.resample_residual(d, t, rej, nodes, seed=5, step=1)
    for b in range(B):
        _, expect, _ = oracle.rrs_chain(_softmax(d[b]), _softmax(t[b]), [3, 8])
        assert np.allclose(res["residual"][b], expect, atol=1e-15)


def test_gumbel_top1_final_token_follows_the_residual():
    # Algorithm 6 draws the last token by Gumbel-Top-1: over many independent sequences its law must be the
    # distribution it is drawn from (here: the target row of a root without children), like the inverse-CDF draw
    rng = np.random.default_rng(41)
    V, B = 50, 40000
    row = rng.normal(0, 1.5, V).astype(np.float32)
    row[7] = -np.inf                                           # a token without mass is never drawn
    target = np.broadcast_to(row, (B, 1, V)).copy()
    draft = np.zeros((B, 1, V), np.float32)
    parent = np.array([-1], np.int32)
    token = np.full((B, 1), -1, np.int32)
    q = np.exp(row.astype(np.float64) - row[np.isfinite(row)].max())
    q /= q.sum()
    laws = {}
    for sampler in (0, 1):
        out = oracle.verify_tree(draft, target, parent, token, 0, seed=5, step=1, final_sampler=sampler)
        counts = np.bincount(out["last_token"], minlength=V).astype(np.float64)
        assert counts[7] == 0
        keep = q > 0
        chi2 = (((counts - B * q) ** 2)[keep] / (B * q[keep])).sum()
        assert chi2 < 100.0, (sampler, chi2)                  # 48 degrees of freedom: 100 is far in the tail
        laws[sampler] = out["last_token"]
    assert (laws[0] != laws[1]).mean() > 0.5                    # two different samplers, one law


def test_first_emitted_token_is_target_distributed_with_gumbel_top1_last_draw():
    # Theorem 3.1 with Algorithm 6's own last step: three children of the root drawn by Gumbel-Top-k, the walk, and
    # the last token by Gumbel-Top-1 on the residual.  The noise of that last draw must be independent of the noise
    # that drafted the children (it has streams of its own): were it the node's drafting noise again, the residual
    # draw after three rejections would lean towards the fourth-best perturbed draft value and the first emitted
    # token would no longer follow q(. | root).
    rng = np.random.default_rng(44)
    V, n, K = 50, 60000, 3
    ld = rng.normal(0, 1.5, V).astype(np.float32)
    lt = (ld + rng.normal(0, 1.5, V)).astype(np.float32)      # far apart: all three rejected fairly often
    q = _softmax(lt)
    draft = np.broadcast_to(ld[None, None, :], (n, 1, V))
    target = np.broadcast_to(lt[None, None, :], (n, 1 + K, V))
    parent = np.array([-1, 0, 0, 0], np.int32)
    d = oracle.gumbel_topk(draft, [K], [0], seed=13, step=5)
    token = np.concatenate([np.full((n, 1), -1, np.int32), d["token"][:, 0, :]], 1)
    out = oracle.verify_tree(draft, target, parent, token, 1, seed=13, step=5, final_sampler=1)
    rejected_all = out["accepted_len"] == 0
    assert 0.1 < rejected_all.mean() < 0.9                    # both branches carry weight
    first = np.where(out["accepted_len"] > 0, out["accepted_token"][:, 0], out["last_token"])
    counts = np.bincount(first, minlength=V).astype(float)
    keep = q * n > 5
    obs = np.append(counts[keep], counts[~keep].sum())
    exp = np.append(q[keep] * n, q[~keep].sum() * n)
    assert stats.chisquare(obs, exp).pvalue > 1e-3
    # the same law as with the inverse-CDF draw, from different random numbers
    out0 = oracle.verify_tree(draft, target, parent, token, 1, seed=13, step=5, final_sampler=0)
    assert np.array_equal(out0["accepted_len"], out["accepted_len"])
    assert (out0["last_token"][rejected_all] != out["last_token"][rejected_all]).mean() > 0.3
