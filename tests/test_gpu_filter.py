"""rsd_filter_rows (top-k and nucleus filtering, Section 4's sampling settings) against the oracle, and the filtered
rows through drafting and verification."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from tests.parity import Tally, compare_topk, compare_verify

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rsd():
    import paper_2402_14160_b200 as m
    m.lib()
    return m


def _rows(shape, dtype, sigma, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    t = torch.randn(shape, generator=g, dtype=torch.float32) * sigma
    return t.to(torch.bfloat16 if dtype == "bf16" else torch.float32).cuda()


def _check_filter(rsd, rows, top_k, top_p, T, max_borderline=None):
    """GPU mask == oracle mask for every row whose nucleus cut is not borderline; returns the GPU's filtered rows."""
    g = rsd.rsd_filter_rows(rows, top_k, top_p, temperature=T)
    host = workloads.as_oracle_rows(rows.contiguous())
    o = oracle.filter_rows(host, top_k, top_p, temperature=T)
    want = oracle.apply_filter(host, o["keep"])
    got = workloads.as_oracle_rows(g["rows"])
    kept = g["kept"].cpu().numpy()
    B, R, _ = host.shape
    borderline = 0
    for b in range(B):
        for r in range(R):
            same = np.array_equal(got[b, r].view(np.uint32 if got.dtype == np.float32 else np.uint16),
                                  want[b, r].view(np.uint32 if want.dtype == np.float32 else np.uint16))
            if same:
                assert kept[b, r] == o["kept"][b, r]
                continue
            assert o["margin"][b, r] <= 1e-5, ("filter", b, r, int(kept[b, r]), int(o["kept"][b, r]), float(o["margin"][b, r]))
            borderline += 1
    assert borderline <= (max(1, B * R // 100) if max_borderline is None else max_borderline)
    return g


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [1, 17, 1000, 4099, 32000])
def test_filter_rows_matches_oracle(rsd, dtype, V):
    rows = _rows((3, 4, V), dtype, 2.0, 40 + V)
    for top_k, top_p, T in ((0, 0.95, 1.0), (min(50, V), 1.0, 1.0), (min(40, V), 0.9, 0.3), (0, 0.5, 2.0), (0, 1.0, 1.0),
                            (1, 1.0, 1.0), (0, 1e-6, 1.0)):
        g = _check_filter(rsd, rows, top_k, top_p, T)
        assert int(g["status"].sum()) == 0
        assert int(g["kept"].min()) >= 1


def test_filter_rows_ties_masked_entries_unaligned_rows_and_errors(rsd):
    V = 515
    # many equal values (a coarse grid): the cut falls inside a run of equal entries and the smaller tokens stay
    grid = (torch.randint(-3, 4, (2, 3, V), generator=torch.Generator().manual_seed(5)).float() * 0.5)
    for dtype in (torch.float32, torch.bfloat16):
        rows = grid.to(dtype).cuda()
        for top_k, top_p in ((100, 1.0), (0, 0.8), (37, 0.6)):
            _check_filter(rsd, rows, top_k, top_p, 1.0)
    # entries that are already -inf or NaN stay out; a row with a single finite entry keeps it
    rows = _rows((2, 2, V), "f32", 2.0, 9)
    rows[0, 0, 100:] = float("-inf")
    rows[0, 1, :] = float("-inf")
    rows[0, 1, 7] = 0.5
    rows[1, 0, 33] = float("nan")
    g = _check_filter(rsd, rows, 20, 0.9, 1.0)
    assert g["status"].cpu().tolist() == [0, rsd.ST_NAN_INPUT] and g["kept"][0, 1].item() == 1
    # rows at odd offsets and strides
    base = _rows((2, 3, V + 5), "bf16", 2.0, 10)
    _check_filter(rsd, base[:, :, 3:3 + V], 0, 0.9, 1.0)
    with pytest.raises(rsd.RsdError, match="top_p"):
        rsd.rsd_filter_rows(rows, 0, 0.0)
    with pytest.raises(rsd.RsdError, match="shared memory"):
        rsd.rsd_filter_rows(torch.zeros((1, 1, 120000), device="cuda"), 0, 0.9)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_filter_rows_degenerate_rows(rsd, dtype):
    # rows the histogram over values cannot split: all entries equal, zeros of both signs, one entry that carries all the
    # mass, two values only, a very wide spread; plus a vocabulary above 65,536 entries (no list of 16-bit indices)
    V = 4096
    g = torch.Generator(device="cpu").manual_seed(77)
    rows = torch.zeros((1, 7, V), dtype=torch.float32)
    rows[0, 0, :] = 0.25
    rows[0, 1, :] = torch.where(torch.rand(V, generator=g) < 0.5, torch.tensor(-0.0), torch.tensor(0.0))
    rows[0, 1, 5::400] = 1.0
    rows[0, 2, :] = torch.randn(V, generator=g)
    rows[0, 2, 1234] = 30.0
    rows[0, 3, :] = torch.where(torch.rand(V, generator=g) < 0.5, torch.tensor(-1.0), torch.tensor(1.0))
    rows[0, 4, :] = torch.randn(V, generator=g) * 8.0
    rows[0, 5, :] = torch.arange(V, dtype=torch.float32) / 64.0 - 40.0
    rows[0, 6, :] = torch.randn(V, generator=g) * 1e-3
    rows = rows.to(torch.bfloat16 if dtype == "bf16" else torch.float32).cuda()
    # (equal entries put cumulative masses exactly on round fractions: rows whose cut the oracle calls borderline may differ)
    for top_k, top_p, T in ((0, 0.9, 1.0), (0, 0.5, 1.0), (100, 1.0, 1.0), (3000, 0.7, 1.0), (0, 0.99, 0.3), (0, 0.999999, 1.0)):
        _check_filter(rsd, rows, top_k, top_p, T, max_borderline=3)
    big = _rows((1, 2, 70000), dtype, 2.0, 78) if dtype == "bf16" else _rows((1, 2, 50272), dtype, 2.0, 78)   # (fp32: OPT's vocabulary)
    _check_filter(rsd, big, 0, 0.9, 1.0)
    _check_filter(rsd, big, 500, 0.95, 1.0)


@pytest.mark.parametrize("dtype,V", [("bf16", 4099), ("f32", 1000)])
def test_filtered_rows_through_drafting_and_verification(rsd, dtype, V):
    # temperature 0.7, top-k 200, nucleus 0.9 on the draft rows and nucleus 0.95 on the target rows; drafting and the
    # walk then run on the filtered rows exactly as on any rows with masked entries
    B, branching, T = 12, (3, 2), 0.7
    parent = workloads.rsdc_parent_array(branching)
    k, nodes = workloads.rsdc_rows(branching)
    base = _rows((B, len(parent), V), "f32", 2.0, 70 + V)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    draft = base[:, :len(k)].to(tdt).contiguous()
    target = (base + _rows((B, len(parent), V), "f32", 1.0, 71 + V)).to(tdt).contiguous()
    fd = _check_filter(rsd, draft, 200, 0.9, T)["rows"]
    ft = _check_filter(rsd, target, 0, 0.95, T)["rows"]
    dh, th = workloads.as_oracle_rows(fd), workloads.as_oracle_rows(ft)
    g = rsd.rsd_gumbel_topk_draft(fd, k, nodes, 3, 1, temperature=T)
    o = oracle.gumbel_topk(dh, k, nodes, 3, 1, temperature=T)
    t = Tally()
    compare_topk(t, g["token"].cpu().numpy(), o, k)
    t.check()
    keep_d = np.isfinite(dh.astype(np.float32)) if dh.dtype == np.float32 else (dh != 0xFF80)
    picks = o["token"]
    for b in range(B):
        for r in range(len(k)):
            assert keep_d[b, r][picks[b, r, :k[r]]].all()          # only tokens the filter left are drafted
    token = workloads.rsdc_tokens_from_rows(branching, o["token"])
    gv = rsd.rsd_verify_tree(fd, ft, torch.from_numpy(parent).cuda(), torch.from_numpy(token).cuda(), 2, 3, 1,
                             want_theta=True, draft_temperature=T, target_temperature=T)
    gv = {kk: v.cpu().numpy() for kk, v in gv.items() if v is not None}
    ov = oracle.verify_tree(dh, th, parent, token, 2, 3, 1, draft_temperature=T, target_temperature=T)
    t = Tally()
    compare_verify(t, gv, ov, parent)
    t.check()
    keep_t = np.isfinite(th.astype(np.float32)) if th.dtype == np.float32 else (th != 0xFF80)
    for b in range(B):
        node = ov["accepted_node"][b, ov["accepted_len"][b] - 1] if ov["accepted_len"][b] > 0 else 0
        assert keep_t[b, node][ov["last_token"][b]]                # the last token comes from the target's nucleus
