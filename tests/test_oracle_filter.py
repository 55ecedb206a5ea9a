"""Pins for the oracle's top-k / nucleus filtering of a row (Section 4's sampling settings): CPU only."""
import numpy as np
from scipy import stats

import oracle


def _softmax(x):
    x = np.asarray(x, np.float64)
    e = np.exp(x - x[np.isfinite(x)].max())
    e[~np.isfinite(x)] = 0.0
    return e / e.sum()


def test_worked_example_and_identities():
    # probabilities 0.5, 0.3, 0.15, 0.05: a nucleus of 0.9 needs the first three (0.8 < 0.9 <= 0.95)
    p = np.array([0.15, 0.5, 0.05, 0.3])
    rows = np.log(p).astype(np.float32)[None, None, :]
    f = oracle.filter_rows(rows, top_p=0.9)
    assert f["keep"][0, 0].tolist() == [True, True, False, True] and f["kept"][0, 0] == 3
    assert abs(f["margin"][0, 0] - 0.05) < 1e-6               # 0.95 - 0.9 (the float32 logs move it a little)
    assert oracle.filter_rows(rows, top_p=0.8 - 1e-9)["kept"][0, 0] == 2
    assert oracle.filter_rows(rows, top_p=0.5 - 1e-9)["kept"][0, 0] == 1
    assert oracle.filter_rows(rows, top_p=1e-12)["kept"][0, 0] == 1          # never empty
    assert oracle.filter_rows(rows, top_k=2)["keep"][0, 0].tolist() == [False, True, False, True]
    # top-k first, then the nucleus of what is left: {0.5, 0.3} renormalised to {0.625, 0.375}
    assert oracle.filter_rows(rows, top_k=2, top_p=0.7)["kept"][0, 0] == 2
    assert oracle.filter_rows(rows, top_k=2, top_p=0.6)["kept"][0, 0] == 1
    # no filter: every finite entry stays, bit for bit
    rng = np.random.default_rng(0)
    big = rng.normal(0, 2, (3, 2, 300)).astype(np.float32)
    big[1, 0, 7] = -np.inf
    for kw in (dict(), dict(top_k=0, top_p=1.0), dict(top_k=300), dict(top_k=10 ** 6, top_p=2.0)):
        f = oracle.filter_rows(big, **kw)
        assert np.array_equal(f["keep"], np.isfinite(big))
        assert np.array_equal(oracle.apply_filter(big, f["keep"]), big)


def test_equal_values_go_to_the_smaller_token():
    rows = np.zeros((1, 1, 8), np.float32)                      # eight equal tokens
    assert oracle.filter_rows(rows, top_k=3)["keep"][0, 0].tolist() == [True] * 3 + [False] * 5
    assert oracle.filter_rows(rows, top_p=0.5)["keep"][0, 0].tolist() == [True] * 4 + [False] * 4
    assert oracle.filter_rows(rows, top_p=0.51)["keep"][0, 0].tolist() == [True] * 5 + [False] * 3
    rows[0, 0, 5] = 1.0
    assert oracle.filter_rows(rows, top_k=2)["keep"][0, 0].tolist() == [True, False, False, False, False, True, False, False]


def test_kept_set_is_the_smallest_prefix_that_reaches_top_p():
    rng = np.random.default_rng(1)
    for dtype in ("f32", "bf16"):
        for T in (1.0, 0.3):
            raw = rng.normal(0, 2, (4, 3, 500)).astype(np.float32)
            if dtype == "bf16":
                rows = (raw.view(np.uint32) >> 16).astype(np.uint16)          # truncation is a fine way to get bf16 patterns
                vals = (rows.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
            else:
                rows, vals = raw, raw.astype(np.float64)
            for top_k, top_p in ((0, 0.95), (50, 0.9), (0, 0.3), (7, 1.0)):
                f = oracle.filter_rows(rows, top_k, top_p, temperature=T)
                for b in range(4):
                    for r in range(3):
                        keep = f["keep"][b, r]
                        order = np.lexsort((np.arange(500), -vals[b, r]))         # value desc, token asc
                        n = f["kept"][b, r]
                        assert set(order[:n]) == set(np.flatnonzero(keep))       # a prefix of the sorted order
                        pool = order[:top_k] if 0 < top_k < 500 else order
                        p = _softmax(vals[b, r][pool] / T)
                        if top_p < 1.0:
                            assert p[:n].sum() >= top_p - 1e-12 and p[:n - 1].sum() < top_p + 1e-12
                            lo, hi = p[:n - 1].sum(), p[:n].sum()
                            assert abs(f["margin"][b, r] - min(hi - top_p, top_p - lo)) < 1e-9
                        else:
                            assert n == len(pool)


def test_first_pick_follows_the_renormalised_truncated_softmax_vocab_50():
    # Gumbel-Top-k on a filtered row samples from the warped distribution: temperature, top-k, nucleus, renormalised
    rng = np.random.default_rng(2)
    V, n, T = 50, 40000, 0.7
    row = rng.normal(0, 1.5, V).astype(np.float32)
    f = oracle.filter_rows(row[None, None, :], top_k=30, top_p=0.9, temperature=T)
    keep = f["keep"][0, 0]
    assert 3 < keep.sum() < 30
    masked = oracle.apply_filter(row[None, None, :], f["keep"])
    rows = np.broadcast_to(masked, (n, 1, V))
    d = oracle.gumbel_topk(rows, [2], [0], seed=3, step=1, temperature=T)
    first = d["token"][:, 0, 0]
    assert keep[first].all() and keep[d["token"][:, 0, 1]].all()               # never a filtered token
    q = _softmax(np.where(keep, row.astype(np.float64) / T, -np.inf))
    counts = np.bincount(first, minlength=V).astype(float)
    assert counts[~keep].sum() == 0
    obs, exp = counts[keep], q[keep] * n
    assert exp.min() > 5
    assert stats.chisquare(obs, exp).pvalue > 1e-3
