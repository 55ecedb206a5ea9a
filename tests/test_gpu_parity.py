"""GPU-vs-oracle parity through the C ABI (needs a CUDA device)."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from tests.parity import Tally, close, compare_sbs_level, compare_topk, compare_verify

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rsd():
    import paper_2402_14160_b200 as m
    m.lib()
    return m


def _np(d):
    return {k: (v.cpu().numpy() if isinstance(v, torch.Tensor) else v) for k, v in d.items()}


def _rows(shape, dtype, sigma, seed, device="cuda"):
    g = torch.Generator(device="cpu").manual_seed(seed)
    t = torch.randn(shape, generator=g, dtype=torch.float32) * sigma
    return t.to(torch.bfloat16 if dtype == "bf16" else torch.float32).to(device)


# ---------------------------------------------------------------------------------------------------------
# Gumbel-Top-k drafting
# ---------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("V", [1, 5, 16, 17, 70, 1000, 4099, 32000, 50272])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_gumbel_topk_matches_oracle(rsd, V, dtype):
    B, R = 3, 4
    rows = _rows((B, R, V), dtype, 2.0, 100 + V)
    k = [min(V, kk) for kk in (1, 2, 4, 32)]
    nodes = [0, 3, 7, 1000]
    g = _np(rsd.rsd_gumbel_topk_draft(rows, k, nodes, seed=11, step=5, seq_base=9, max_k=max(k), want_values=True))
    o = oracle.gumbel_topk(workloads.as_oracle_rows(rows), k, nodes, 11, 5, seq_base=9, max_k=max(k))
    t = Tally()
    compare_topk(t, g["token"], o, k, g["perturbed"], g["logprob"])
    t.check()
    assert np.array_equal(g["status"], o["status"])
    # production form: no values asked, no normaliser computed, same picks
    g2 = _np(rsd.rsd_gumbel_topk_draft(rows, k, nodes, seed=11, step=5, seq_base=9, max_k=max(k)))
    assert np.array_equal(g2["token"], g["token"])


def test_gumbel_topk_unaligned_rows_and_logprob_input(rsd):
    B, R, V = 2, 3, 1003
    base = _rows((B, R, V + 5), "f32", 2.0, 7)
    rows = torch.log_softmax(base, -1)[:, :, 3:3 + V]            # odd offset, odd stride: scalar path
    k, nodes = [3, 3, 3], [1, 2, 3]
    g = _np(rsd.rsd_gumbel_topk_draft(rows, k, nodes, seed=1, step=0, is_logprob=True, want_values=True))
    o = oracle.gumbel_topk(workloads.as_oracle_rows(rows.contiguous()), k, nodes, 1, 0, is_logprob=True)
    t = Tally()
    compare_topk(t, g["token"], o, k, g["perturbed"], g["logprob"])
    t.check()
    bf = _rows((B, R, V + 8), "bf16", 2.0, 8)[:, :, 1:1 + V]
    g = _np(rsd.rsd_gumbel_topk_draft(bf, k, nodes, seed=1, step=0))
    o = oracle.gumbel_topk(workloads.as_oracle_rows(bf.contiguous()), k, nodes, 1, 0)
    t = Tally()
    compare_topk(t, g["token"], o, k)
    t.check()


def test_gumbel_topk_degenerate_rows(rsd):
    V = 300
    rows = torch.full((2, 2, V), float("-inf"), device="cuda")
    rows[0, 0, [5, 77]] = torch.tensor([0.5, 1.0], device="cuda")
    rows[0, 1, :] = 0.0                                           # all equal: noise alone decides
    rows[1, 0, 10:20] = 1.0
    rows[1, 0, 15] = float("nan")
    rows[1, 1, :] = torch.arange(V, device="cuda") * 0.1          # increasing: every element beats the running bound
    k, nodes = [4, 4], [0, 1]
    g = _np(rsd.rsd_gumbel_topk_draft(rows, k, nodes, seed=3, step=0, want_values=True))
    o = oracle.gumbel_topk(workloads.as_oracle_rows(rows), k, nodes, 3, 0)
    t = Tally()
    compare_topk(t, g["token"], o, k, g["perturbed"], g["logprob"])
    t.check()
    assert np.array_equal(g["status"], o["status"])
    assert g["status"][0] & rsd.ST_FEWER_THAN_K and g["status"][1] & rsd.ST_NAN_INPUT
    assert g["token"][0, 0, 2] == -1 and 15 not in g["token"][1, 0]


def test_gumbel_topk_is_deterministic_and_shardable(rsd):
    rows = _rows((8, 3, 5000), "bf16", 2.0, 21)
    k, nodes = [4, 2, 8], [0, 1, 2]
    a = _np(rsd.rsd_gumbel_topk_draft(rows, k, nodes, seed=5, step=1, want_values=True))
    b = _np(rsd.rsd_gumbel_topk_draft(rows, k, nodes, seed=5, step=1, want_values=True))
    assert all(np.array_equal(a[x], b[x]) for x in ("token", "perturbed", "logprob"))
    lo = _np(rsd.rsd_gumbel_topk_draft(rows[:3], k, nodes, seed=5, step=1, seq_base=0))
    hi = _np(rsd.rsd_gumbel_topk_draft(rows[3:], k, nodes, seed=5, step=1, seq_base=3))
    assert np.array_equal(np.concatenate([lo["token"], hi["token"]]), a["token"])


def test_argument_errors_are_reported_not_trapped(rsd):
    rows = _rows((1, 1, 64), "f32", 1.0, 1)
    with pytest.raises(rsd.RsdError, match="max_k"):
        rsd.rsd_gumbel_topk_draft(rows, [40], [0], seed=0, step=0)
    with pytest.raises(rsd.RsdError, match="workspace"):
        rsd.rsd_sbs_step(rows, 2, 0, None, None, 0, 0, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    with pytest.raises(rsd.RsdError):
        rsd.rsd_gumbel_topk_draft(rows.double(), [1], [0], seed=0, step=0)


# ---------------------------------------------------------------------------------------------------------
# Stochastic Beam Search
# ---------------------------------------------------------------------------------------------------------
def _sbs_chain(rsd, draft, W, L, seed, step, is_logprob, seq_base=0):
    """Run L levels on both sides, each from its own previous level; returns (tally, gpu levels, oracle levels)."""
    B = draft.shape[0]
    host = workloads.as_oracle_rows(draft)
    t = Tally()
    skip = set()
    g_prev = o_prev = None
    g_levels, o_levels = [], []
    for l in range(L):
        first = 0 if l == 0 else 1 + (l - 1) * W
        n_par = 1 if l == 0 else W
        g = rsd.rsd_sbs_step(draft[:, first:first + n_par], W, first,
                             None if l == 0 else g_prev["sum_logprob"], None if l == 0 else g_prev["trunc_gumbel"],
                             seed, step, is_logprob=is_logprob, seq_base=seq_base)
        o = oracle.sbs_step(host[:, first:first + n_par], W, first,
                            None if l == 0 else o_prev["sum_logprob"], None if l == 0 else o_prev["trunc_gumbel"],
                            seed, step, is_logprob=is_logprob, seq_base=seq_base)
        skip |= compare_sbs_level(t, _np(g), o, W, skip)
        g_prev, o_prev = g, o
        g_levels.append(_np(g))
        o_levels.append(o)
    return t, g_levels, o_levels, skip


def _sbs_tree(levels, W):
    """parent [B, N+1] (flat) and token [B, N+1] from per-level (token, parent) outputs."""
    B = levels[0]["token"].shape[0]
    L = len(levels)
    parent = np.full((B, 1 + L * W), -1, np.int32)
    token = np.full((B, 1 + L * W), -1, np.int32)
    for l, lv in enumerate(levels):
        off_prev = 0 if l == 0 else 1 + (l - 1) * W
        sl = slice(1 + l * W, 1 + (l + 1) * W)
        token[:, sl] = lv["token"]
        parent[:, sl] = np.where(lv["parent"] >= 0, off_prev + lv["parent"], -1)
    return parent, token


@pytest.mark.parametrize("dtype,V,W,L,is_logprob", [("f32", 1000, 3, 3, False), ("bf16", 4099, 8, 4, False),
                                                    ("f32", 515, 4, 3, True), ("bf16", 32000, 6, 3, False)])
def test_sbs_levels_match_oracle(rsd, dtype, V, W, L, is_logprob):
    B = 6
    P = 1 + (L - 1) * W
    draft = _rows((B, P, V), dtype, 2.0, 300 + V)
    if is_logprob:
        draft = torch.log_softmax(draft.float(), -1).to(draft.dtype)
    t, g_levels, o_levels, _ = _sbs_chain(rsd, draft, W, L, seed=17, step=2, is_logprob=is_logprob, seq_base=4)
    t.check()
    assert all(np.all(g["count"] == W) for g in g_levels)


@pytest.mark.parametrize("dtype,V,W,L,is_logprob", [("f32", 1000, 3, 3, False), ("bf16", 4099, 8, 4, False),
                                                    ("f32", 515, 5, 1, True), ("bf16", 32000, 6, 5, False),
                                                    ("f32", 300, 32, 3, False),    # finalists too many for shared memory
                                                    ("bf16", 520, 16, 6, False)])  # 1296 finalists, staged
def test_sbs_draft_tree_is_the_chain_of_level_calls(rsd, dtype, V, W, L, is_logprob):
    # rsd_sbs_draft_tree (all levels from rows that exist up front) must give what L rsd_sbs_step calls give, bit for
    # bit, and through them what the oracle's level-by-level chain gives
    B = 7
    P = 1 + (L - 1) * W
    draft = _rows((B, P, V), dtype, 2.5, 700 + V)
    if is_logprob:
        draft = torch.log_softmax(draft.float(), -1).to(draft.dtype)
    t, g_levels, o_levels, skip = _sbs_chain(rsd, draft, W, L, seed=23, step=6, is_logprob=is_logprob, seq_base=11)
    t.check()
    parent, token = _sbs_tree(g_levels, W)
    node_token = torch.full((B, 3 + L * W), -7, dtype=torch.int32, device="cuda")      # wider than needed: stride kept
    node_parent = torch.full((B, 3 + L * W), -7, dtype=torch.int32, device="cuda")
    out = _np(rsd.rsd_sbs_draft_tree(draft, W, L, 23, 6, node_token, node_parent, is_logprob=is_logprob, seq_base=11))
    torch.cuda.synchronize()
    nt, npar = node_token.cpu().numpy(), node_parent.cpu().numpy()
    assert np.array_equal(nt[:, 1:1 + L * W], token[:, 1:]) and np.array_equal(npar[:, 1:1 + L * W], parent[:, 1:])
    assert np.all(nt[:, 0] == -7) and np.all(nt[:, 1 + L * W:] == -7) and np.all(npar[:, 1 + L * W:] == -7)   # untouched
    assert np.array_equal(out["sum_logprob"], g_levels[-1]["sum_logprob"])
    assert np.array_equal(out["trunc_gumbel"], g_levels[-1]["trunc_gumbel"])
    assert np.array_equal(out["count"], np.stack([g["count"] for g in g_levels]))
    assert np.array_equal(out["status"], np.bitwise_or.reduce(np.stack([g["status"] for g in g_levels]), axis=0))


def test_sbs_draft_tree_with_underfull_levels_and_bad_arguments(rsd):
    W, L, V = 4, 3, 64
    draft = _rows((3, 1 + (L - 1) * W, V), "f32", 2.0, 31)
    draft[0, 0, :] = float("-inf")
    draft[0, 0, [5, 9]] = 0.25                                   # the root of sequence 0 offers two tokens only
    node_token = torch.full((3, 1 + L * W), -1, dtype=torch.int32, device="cuda")
    node_parent = torch.full((3, 1 + L * W), -1, dtype=torch.int32, device="cuda")
    out = _np(rsd.rsd_sbs_draft_tree(draft, W, L, 2, 0, node_token, node_parent))
    host = workloads.as_oracle_rows(draft)
    prev = None
    for l in range(L):
        first = 0 if l == 0 else 1 + (l - 1) * W
        o = oracle.sbs_step(host[:, first:first + (1 if l == 0 else W)], W, first, None if l == 0 else prev["sum_logprob"],
                            None if l == 0 else prev["trunc_gumbel"], 2, 0)
        sl = slice(1 + l * W, 1 + (l + 1) * W)
        assert np.array_equal(node_token[:, sl].cpu().numpy(), o["token"]), l
        assert np.array_equal(node_parent[:, sl].cpu().numpy(), np.where(o["parent"] >= 0, first + o["parent"], -1)), l
        assert np.array_equal(out["count"][l], o["count"])
        prev = o
    assert out["count"][0, 0] == 2 and out["status"][0] & rsd.ST_FEWER_THAN_K and out["status"][1] == 0
    with pytest.raises(rsd.RsdError, match="rows per sequence"):
        rsd.rsd_sbs_draft_tree(draft[:, :5], W, L, 2, 0, node_token, node_parent)
    with pytest.raises(rsd.RsdError, match="node_stride"):
        rsd.rsd_sbs_draft_tree(draft, W, L, 2, 0, node_token[:, :6].contiguous(), node_parent[:, :6].contiguous())


def test_sbs_drops_minus_infinity_candidates(rsd):
    rows = torch.full((1, 2, 64), float("-inf"), device="cuda")
    rows[0, 0, [2, 9]] = torch.tensor([0.0, 1.0], device="cuda")
    rows[0, 1, 5] = 0.3
    sig = torch.zeros((1, 2), device="cuda")
    gam = torch.tensor([[0.0, -0.5]], device="cuda")
    g = _np(rsd.rsd_sbs_step(rows, 4, 1, sig, gam, 3, 0))
    o = oracle.sbs_step(workloads.as_oracle_rows(rows), 4, 1, sig.cpu().numpy(), gam.cpu().numpy(), 3, 0)
    assert np.array_equal(g["token"], o["token"]) and np.array_equal(g["parent"], o["parent"])
    assert g["count"][0] == 3 and g["status"][0] & rsd.ST_FEWER_THAN_K
    assert close(g["trunc_gumbel"][0, :3], o["trunc_gumbel"][0, :3]).all()


@pytest.mark.parametrize("dtype,V,W,L,sigma", [("f32", 200, 8, 5, 3.5), ("bf16", 4099, 8, 4, 4.5), ("f32", 64, 4, 6, 3.0)])
def test_sbs_peaked_rows_branch_inside_a_parent(rsd, dtype, V, W, L, sigma):
    # peaked next-token distributions: several children of one parent enter the beam and other parents drop out, so
    # the epilogue's early rejection of finalists (psi below the W-th largest Gamma) has to keep exactly the right ones
    B = 16
    draft = _rows((B, 1 + (L - 1) * W, V), dtype, sigma, 900 + V)
    t, g_levels, o_levels, _ = _sbs_chain(rsd, draft, W, L, seed=5, step=1, is_logprob=False)
    t.check()
    parents = np.concatenate([o["parent"] for o in o_levels[1:]])
    counts = [len(set(row.tolist())) for row in parents]
    assert min(counts) < W and np.mean(counts) < W - 0.25      # parents really are shared and dropped


def test_sbs_parent_with_a_fully_masked_row(rsd):
    # W valid parents, one of which has no selectable child: only W - 1 parents deliver their best child, so second
    # and third children of the others must still be found
    W, V = 4, 96
    rows = _rows((3, W, V), "f32", 2.0, 77)
    rows[:, 2, :] = float("-inf")
    sig = _rows((3, W), "f32", 1.0, 78) - 3.0
    gam = _rows((3, W), "f32", 1.0, 79)
    g = _np(rsd.rsd_sbs_step(rows, W, 1, sig, gam, 11, 0))
    o = oracle.sbs_step(workloads.as_oracle_rows(rows), W, 1, sig.cpu().numpy().astype(np.float64),
                        gam.cpu().numpy().astype(np.float64), 11, 0)
    t = Tally()
    compare_sbs_level(t, g, o, W, set())
    t.check()
    assert np.all(g["count"] == W) and not np.any(g["parent"] == 2)


def test_sbs_level_after_an_underfull_level(rsd):
    # A level that finds fewer than W finite candidates pads its outputs with -1 / -inf.  Fed to the next level,
    # those slots are empty parents: they must contribute no children (no NaN, no pick pointing at them), like the
    # oracle, which drops every candidate whose sequence log-probability is -inf.
    W, V = 4, 80
    root = torch.full((2, 1, V), float("-inf"), device="cuda")
    root[0, 0, [3, 17, 40]] = torch.tensor([0.5, -0.25, 1.0], device="cuda")      # W - 1 finite entries
    root[1, 0, [5, 6]] = torch.tensor([0.0, 0.1], device="cuda")                  # W - 2
    g0 = _np(rsd.rsd_sbs_step(root, W, 0, None, None, 8, 2))
    o0 = oracle.sbs_step(workloads.as_oracle_rows(root), W, 0, None, None, 8, 2)
    assert np.array_equal(g0["token"], o0["token"]) and list(g0["count"]) == [3, 2]
    assert np.all(np.isneginf(g0["sum_logprob"][0, 3:])) and np.all(np.isneginf(g0["trunc_gumbel"][1, 2:]))
    rows = _rows((2, W, V), "f32", 2.0, 4242)
    g1 = _np(rsd.rsd_sbs_step(rows, W, 1, torch.from_numpy(g0["sum_logprob"]).cuda(),
                              torch.from_numpy(g0["trunc_gumbel"]).cuda(), 8, 2, parent_base=1))
    o1 = oracle.sbs_step(workloads.as_oracle_rows(rows), W, 1, o0["sum_logprob"], o0["trunc_gumbel"], 8, 2)
    t = Tally()
    g1_rel = dict(g1, parent=np.where(g1["parent"] >= 0, g1["parent"] - 1, -1))
    compare_sbs_level(t, g1_rel, o1, W, set())
    t.check()
    assert np.all(g1["count"] == W) and not np.any(np.isnan(g1["trunc_gumbel"]))
    assert np.all(g1_rel["parent"][0] < 3) and np.all(g1_rel["parent"][1] < 2)   # never an empty slot


# ---------------------------------------------------------------------------------------------------------
# verification
# ---------------------------------------------------------------------------------------------------------
def _verify_both(rsd, draft, target, parent, token, L, seed, step, seq_base=0):
    par_t = torch.from_numpy(parent).cuda()
    tok_t = torch.from_numpy(token).cuda()
    g = _np(rsd.rsd_verify_tree(draft, target, par_t, tok_t, L, seed, step, seq_base=seq_base, want_theta=True))
    o = oracle.verify_tree(workloads.as_oracle_rows(draft), workloads.as_oracle_rows(target), parent, token, L,
                           seed, step, seq_base=seq_base)
    return g, o


@pytest.mark.parametrize("dtype,V,branching,noise", [("f32", 64, (3, 2, 2), 1.0), ("bf16", 515, (4, 2, 1), 1.5),
                                                      ("f32", 4099, (3, 3), 2.0), ("bf16", 32000, (3, 2, 2, 1), 1.0),
                                                      ("f32", 32000, (2, 2, 2), 0.5), ("bf16", 50272, (4, 2), 1.0)])
def test_verify_tree_matches_oracle_constant_branching(rsd, dtype, V, branching, noise):
    B = 48 if V <= 5000 else 12
    L = len(branching)
    parent = workloads.rsdc_parent_array(branching)
    n_nodes = len(parent)
    k, nodes = workloads.rsdc_rows(branching)
    P = len(k)
    base = _rows((B, n_nodes, V), "f32", 2.0, 500 + V)
    draft = base[:, :P].to(torch.bfloat16 if dtype == "bf16" else torch.float32).contiguous()
    target = (base + _rows((B, n_nodes, V), "f32", noise, 501 + V)).to(draft.dtype).contiguous()
    o_draft = oracle.gumbel_topk(workloads.as_oracle_rows(draft), k, nodes, 23, 1, seq_base=2)
    token = workloads.rsdc_tokens_from_rows(branching, o_draft["token"])
    g, o = _verify_both(rsd, draft, target, parent, token, L, 23, 1, seq_base=2)
    t = Tally()
    compare_verify(t, g, o, parent)
    t.check()
    assert t.final_mismatch <= max(1, 0.02 * B)
    assert np.array_equal(g["status"], o["status"])
    assert len(set(o["accepted_len"].tolist())) > 1 or B < 20     # the cases exercise several path lengths


def test_verify_tree_special_trees(rsd):
    rng = np.random.default_rng(3)
    V = 200
    parent = np.array([[-1, 0, 0, 1, 1, 2]] * 4, np.int32)       # per-sequence topology
    token = np.array([[-1, 4, 7, 1, -1, 3]] * 4, np.int32)
    token[1, 1:] = -1                                             # sequence 1: the root has no children
    token[2, 2] = 250                                             # sequence 2: a token outside the vocabulary is absent
    draft = torch.from_numpy(rng.normal(0, 1, (4, 3, V)).astype(np.float32)).cuda()
    target = torch.from_numpy(rng.normal(0, 1, (4, 6, V)).astype(np.float32)).cuda()
    target[3] = torch.cat([draft[3], draft[3]], 0)                # sequence 3: target == draft on the visited rows
    tok_o = token.copy()
    tok_o[2, 2] = -1
    par_t, tok_t = torch.from_numpy(parent).cuda(), torch.from_numpy(token).cuda()
    g = _np(rsd.rsd_verify_tree(draft, target, par_t, tok_t, 2, 9, 0, want_theta=True))
    o = oracle.verify_tree(workloads.as_oracle_rows(draft), workloads.as_oracle_rows(target), parent, tok_o, 2, 9, 0)
    t = Tally()
    compare_verify(t, g, o, parent)
    t.check()
    assert g["stop_reason"][1] == rsd.STOP_NO_CHILDREN and g["accepted_len"][1] == 0
    assert g["accepted_len"][3] == 2 and g["stop_reason"][3] == rsd.STOP_LEAF
    assert np.array_equal(g["last_token"], o["last_token"])


@pytest.mark.parametrize("dtype,V,branching,aligned", [("bf16", 64, (20, 20), True), ("f32", 48, (40,), True),
                                                       ("f32", 50, (20, 20), False), ("bf16", 1000, (40, 2), True),
                                                       ("f32", 51, (40,), False)])
def test_verify_tree_wide_and_large_trees(rsd, dtype, V, branching, aligned):
    # b = (20, 20): 421 nodes, more than the walk kernels keep in shared memory, so the children are searched in
    # global memory; b = (40, ...): a node with 40 children, more rejections than a warp has lanes (the row values
    # of the later children are no longer fetched ahead) and, with the draft far from the target, more removed
    # tokens than the 32 the register-fed walk remembers.  aligned=False: rows at odd offsets (register-fed walk).
    B = 24
    L = len(branching)
    parent = workloads.rsdc_parent_array(branching)
    n_nodes = len(parent)
    k, nodes = workloads.rsdc_rows(branching)
    P = len(k)
    pad = 0 if aligned else 3
    base = _rows((B, n_nodes, V + pad), "f32", 1.5, 800 + V)
    tgt = -1.5 * base + _rows((B, n_nodes, V + pad), "f32", 0.5, 801 + V)     # what the draft likes the target does not
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    draft = base[:, :P].to(tdt).contiguous()[:, :, pad:]
    target = tgt.to(tdt).contiguous()[:, :, pad:]
    o_draft = oracle.gumbel_topk(workloads.as_oracle_rows(draft.contiguous()), k, nodes, 4, 3)
    token = workloads.rsdc_tokens_from_rows(branching, o_draft["token"])
    par_t, tok_t = torch.from_numpy(parent).cuda(), torch.from_numpy(token).cuda()
    g = _np(rsd.rsd_verify_tree(draft, target, par_t, tok_t, L, 4, 3, want_theta=True))
    o = oracle.verify_tree(workloads.as_oracle_rows(draft.contiguous()), workloads.as_oracle_rows(target.contiguous()),
                           parent, token, L, 4, 3)
    t = Tally()
    compare_verify(t, g, o, parent)
    t.check()
    assert np.array_equal(g["status"], o["status"])
    tested = (~np.isnan(o["theta"])).sum(axis=1)
    assert tested.max() >= branching[0] // 2                       # some walk went through many children of a node


@pytest.mark.parametrize("V", [128, 127])      # rows on and off 16-byte boundaries: the two walks
def test_verify_tree_repeated_sibling_tokens(rsd, V):
    # Two children of a node carry the same token (a caller's tree; Gumbel-Top-k never drafts one): once the first is
    # rejected its draft mass is gone (Eq. 1), so the second is a child the draft could not have produced: threshold 0
    # (its residual mass is 0 too) and RSD_ST_ZERO_DRAFT_PROB, exactly as the oracle reports it.
    rng = np.random.default_rng(8)
    B = 16
    parent = np.array([-1, 0, 0, 0, 0], np.int32)
    draft_h = rng.normal(0, 1, (B, 1, V)).astype(np.float32)
    target_h = rng.normal(0, 1, (B, 5, V)).astype(np.float32)
    token = np.tile(np.array([[-1, 5, 9, 5, 11]], np.int32), (B, 1))
    target_h[:, 0, 5] -= 6.0                                       # token 5 is rejected almost surely
    target_h[:, 0, 9] -= 6.0
    for dtype in (torch.float32, torch.bfloat16):
        draft, target = torch.from_numpy(draft_h).to(dtype).cuda(), torch.from_numpy(target_h).to(dtype).cuda()
        g, o = _verify_both(rsd, draft, target, parent, token, 1, 31, 2)
        t = Tally()
        compare_verify(t, g, o, parent)
        t.check()
        assert np.array_equal(g["status"], o["status"])
        reached = ~np.isnan(o["theta"][:, 3])
        assert reached.sum() >= B // 2 and np.all(o["status"][reached] & rsd.ST_ZERO_DRAFT_PROB)
        assert np.all(g["theta"][reached, 3] == 0.0)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_verify_tree_rows_far_from_zero_and_nan_logits(rsd, dtype):
    # The copy-engine walk takes its first pass relative to a reference of 0: rows shifted by +-120 (sums over- or
    # underflow), rows of which only one far-away entry is finite, and rows with NaN logits make it fall back on the
    # rows' maxima and on its cleaning passes.
    B, V, branching = 20, 4096 + 40, (3, 2)
    parent = workloads.rsdc_parent_array(branching)
    k, nodes = workloads.rsdc_rows(branching)
    base = _rows((B, len(parent), V), "f32", 2.0, 61)
    tgt = base + _rows((B, len(parent), V), "f32", 1.0, 62)
    shift = torch.tensor([0.0, 120.0, -120.0, 300.0, -90.0] * 4, device="cuda").view(B, 1, 1)
    base, tgt = base + shift, tgt - shift
    base[5, 1, 100:] = float("-inf")                               # a draft row with 100 finite entries
    tgt[6, 0, :] = float("-inf")
    tgt[6, 0, 77] = -250.0                                         # a target row with one finite, far-away entry
    tgt[7, 0, 1000] = float("nan")
    base[8, 0, 2000] = float("nan")
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    draft, target = base[:, :len(k)].to(tdt).contiguous(), tgt.to(tdt).contiguous()
    o_draft = oracle.gumbel_topk(workloads.as_oracle_rows(draft), k, nodes, 6, 0)
    token = workloads.rsdc_tokens_from_rows(branching, o_draft["token"])
    g, o = _verify_both(rsd, draft, target, parent, token, 2, 6, 0)
    t = Tally()
    compare_verify(t, g, o, parent)
    t.check()
    assert np.array_equal(g["status"], o["status"])
    assert o["status"][7] & rsd.ST_NAN_INPUT and o["status"][8] & rsd.ST_NAN_INPUT


def test_verify_tree_on_stochastic_beam_trees(rsd):
    w = workloads.scaled(workloads.WORKLOADS[3], batch=8, vocab=4000)
    draft, target = workloads.make_logits(w, step=0, device="cuda")
    W, L = w.beam_width, w.depth
    _, g_levels, o_levels, skip = _sbs_chain(rsd, draft, W, L, seed=5, step=0, is_logprob=True)
    parent, token = _sbs_tree(o_levels, W)
    g, o = _verify_both(rsd, draft, target, parent, token, L, 5, 0)
    t = Tally()
    compare_verify(t, g, o, parent)
    t.check()


# ---------------------------------------------------------------------------------------------------------
# residual draw
# ---------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,V", [("f32", 70), ("bf16", 4099), ("f32", 32000)])
def test_resample_residual_matches_oracle(rsd, dtype, V):
    B = 16
    d = _rows((B, V), dtype, 2.0, 900 + V)
    tg = (d.float() + _rows((B, V), "f32", 1.0, 901 + V)).to(d.dtype)
    nodes = torch.arange(B, dtype=torch.int32, device="cuda") + 3
    rng = np.random.default_rng(V)
    rej = np.full((B, 4), -1, np.int32)
    for b in range(B):
        n = b % 4
        rej[b, :n] = rng.choice(V, n, replace=False)
    rej[:, 0][rej[:, 0] < 0] = -1
    g = _np(rsd.rsd_resample_residual(d, tg, torch.from_numpy(rej).cuda(), nodes, 13, 2, seq_base=1, want_residual=True))
    o = oracle.resample_residual(workloads.as_oracle_rows(d), workloads.as_oracle_rows(tg), rej, nodes.cpu().numpy(),
                                 13, 2, seq_base=1)
    peak = o["residual"].max(axis=1, keepdims=True)
    assert np.all(np.abs(g["residual"] - o["residual"]) <= 1e-5 * peak)
    mism = g["token"] != o["token"]
    assert np.all(o["margin"][mism] <= 1e-5) and mism.sum() <= 1
    plain = _np(rsd.rsd_resample_residual(None, tg, None, nodes, 13, 2, seq_base=1, want_residual=True))
    o2 = oracle.resample_residual(None, workloads.as_oracle_rows(tg), None, nodes.cpu().numpy(), 13, 2, seq_base=1)
    assert np.all(np.abs(plain["residual"] - o2["residual"]) <= 1e-5 * o2["residual"].max(axis=1, keepdims=True))
    assert (plain["token"] != o2["token"]).sum() <= 1


# ---------------------------------------------------------------------------------------------------------
# sampling temperature (Section 4: 0.3 and 1.0)
# ---------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,V,T", [("f32", 4099, 0.3), ("bf16", 32000, 0.3), ("bf16", 515, 0.7), ("f32", 1000, 2.0)])
def test_gumbel_topk_with_temperature(rsd, dtype, V, T):
    B, R = 3, 4
    rows = _rows((B, R, V), dtype, 2.0, 1200 + V)
    k = [min(V, x) for x in (1, 4, 8, 32)]
    T = float(np.float32(T))                                     # the library takes the temperature as fp32
    # value / T and the log-sum-exp are fp32 numbers of this size: two ulps of it bound their difference's error
    tol = 2.0 * float(np.spacing(np.float32(rows.float().abs().max().item() / T)))
    g = rsd.rsd_gumbel_topk_draft(rows, k, [0, 3, 7, 11], 9, 2, max_k=max(k), want_values=True, temperature=T)
    o = oracle.gumbel_topk(workloads.as_oracle_rows(rows), k, [0, 3, 7, 11], 9, 2, max_k=max(k), temperature=T)
    t = Tally()
    compare_topk(t, g["token"].cpu().numpy(), o, k, g["perturbed"].cpu().numpy(), g["logprob"].cpu().numpy(),
                 logprob_abs_tol=tol)
    t.check()
    # log-probability rows are re-scored under a temperature: same picks as the raw rows give
    lp = torch.log_softmax(rows.float(), -1)
    g2 = rsd.rsd_gumbel_topk_draft(lp, k, [0, 3, 7, 11], 9, 2, max_k=max(k), want_values=True, is_logprob=True,
                                   temperature=T)
    o2 = oracle.gumbel_topk(workloads.as_oracle_rows(lp), k, [0, 3, 7, 11], 9, 2, max_k=max(k), is_logprob=True,
                            temperature=T)
    t = Tally()
    compare_topk(t, g2["token"].cpu().numpy(), o2, k, g2["perturbed"].cpu().numpy(), g2["logprob"].cpu().numpy(),
                 logprob_abs_tol=tol)
    t.check()


@pytest.mark.parametrize("dtype,V,W,L,T", [("bf16", 4099, 8, 4, 0.3), ("f32", 1000, 4, 4, 0.3), ("bf16", 32000, 6, 3, 0.5)])
def test_sbs_and_walk_with_temperature(rsd, dtype, V, W, L, T):
    # low temperature sharpens the rows: beams branch inside parents, acceptance tests see tempered ratios
    B = 8
    T = float(np.float32(T))
    P = 1 + (L - 1) * W
    draft = _rows((B, P, V), dtype, 1.5, 1300 + V)
    target = (torch.cat([draft.float(), _rows((B, W, V), "f32", 1.5, 1301 + V)], 1)
              + _rows((B, P + W, V), "f32", 0.5, 1302 + V)).to(draft.dtype)
    host = workloads.as_oracle_rows(draft)
    t = Tally()
    skip = set()
    g_prev = o_prev = None
    o_levels = []
    for l in range(L):
        first = 0 if l == 0 else 1 + (l - 1) * W
        n_par = 1 if l == 0 else W
        g = rsd.rsd_sbs_step(draft[:, first:first + n_par], W, first, None if l == 0 else g_prev["sum_logprob"],
                             None if l == 0 else g_prev["trunc_gumbel"], 21, 3, temperature=T)
        o = oracle.sbs_step(host[:, first:first + n_par], W, first, None if l == 0 else o_prev["sum_logprob"],
                            None if l == 0 else o_prev["trunc_gumbel"], 21, 3, temperature=T)
        skip |= compare_sbs_level(t, _np(g), o, W, skip)
        g_prev, o_prev = g, o
        o_levels.append(o)
    t.check()
    parent, token = _sbs_tree(o_levels, W)
    par_t, tok_t = torch.from_numpy(parent).cuda(), torch.from_numpy(token).cuda()
    gv = _np(rsd.rsd_verify_tree(draft, target, par_t, tok_t, L, 21, 3, want_theta=True, draft_temperature=T,
                                 target_temperature=T))
    ov = oracle.verify_tree(host, workloads.as_oracle_rows(target), parent, token, L, 21, 3, draft_temperature=T,
                            target_temperature=T)
    t = Tally()
    compare_verify(t, gv, ov, parent)
    t.check()
    # and with different temperatures for the two models
    gv = _np(rsd.rsd_verify_tree(draft, target, par_t, tok_t, L, 21, 3, want_theta=True, draft_temperature=T,
                                 target_temperature=1.0))
    ov = oracle.verify_tree(host, workloads.as_oracle_rows(target), parent, token, L, 21, 3, draft_temperature=T)
    t = Tally()
    compare_verify(t, gv, ov, parent)
    t.check()


def test_temperature_arguments_are_checked(rsd):
    rows = _rows((1, 1, 64), "f32", 1.0, 1)
    for bad in (-0.5, float("nan"), float("inf")):
        with pytest.raises(rsd.RsdError, match="temperature"):
            rsd.rsd_gumbel_topk_draft(rows, [1], [0], seed=0, step=0, temperature=bad)
    a = rsd.rsd_gumbel_topk_draft(rows, [4], [0], seed=0, step=0, temperature=0.0)     # 0 = none
    b = rsd.rsd_gumbel_topk_draft(rows, [4], [0], seed=0, step=0)
    assert torch.equal(a["token"], b["token"])


# ---------------------------------------------------------------------------------------------------------
# baseline verifiers on the same kernel: multi-round rejection sampling and K-SEQ (Section 2)
# ---------------------------------------------------------------------------------------------------------
def _iid_tree(draft_h, branching, seed):
    """Tree with constant branching factors whose children are independent draws (repeats allowed) from the softmax of
    the parent's draft row, as the two baseline verifiers assume."""
    parent = workloads.rsdc_parent_array(branching)
    B, P, V = draft_h.shape
    rng = np.random.default_rng(seed)
    token = np.full((B, len(parent)), -1, np.int32)
    if draft_h.dtype == np.uint16:   # bf16 rows come as bit patterns
        draft_h = (draft_h.astype(np.uint32) << 16).view(np.float32)
    for b in range(B):
        for n in range(1, len(parent)):
            row = draft_h[b, parent[n]].astype(np.float64)
            p = np.exp(row - row.max())
            token[b, n] = rng.choice(V, p=p / p.sum())
    return parent, token


@pytest.mark.parametrize("rule,gamma,sampler", [(1, 1.0, 0), (2, 3.0, 0), (2, 1.5, 0), (0, 1.0, 1), (1, 1.0, 1), (2, 2.0, 1)])
@pytest.mark.parametrize("dtype,V,branching", [("f32", 97, (3, 3)), ("bf16", 4099, (3, 2, 2)), ("bf16", 32000, (4, 2))])
def test_verify_tree_baseline_rules_match_oracle(rsd, rule, gamma, sampler, dtype, V, branching):
    B = 40 if V <= 5000 else 12
    L = len(branching)
    n_nodes = len(workloads.rsdc_parent_array(branching))
    P = n_nodes - int(np.prod(branching))
    # peaked drafts (sigma 3) so that repeated children occur; a target close enough for walks of several lengths
    base = _rows((B, n_nodes, V), "f32", 3.0, 700 + V)
    draft = base[:, :P].to(torch.bfloat16 if dtype == "bf16" else torch.float32).contiguous()
    target = (base + _rows((B, n_nodes, V), "f32", 1.0, 701 + V)).to(draft.dtype).contiguous()
    draft_h = workloads.as_oracle_rows(draft)
    if rule == 0:   # recursive rejection sampling verifies drafts without replacement
        k, nodes = workloads.rsdc_rows(branching)
        parent = workloads.rsdc_parent_array(branching)
        token = workloads.rsdc_tokens_from_rows(branching, oracle.gumbel_topk(draft_h, k, nodes, 31, 2, seq_base=7)["token"])
    else:
        parent, token = _iid_tree(draft_h, branching, 5 + rule)
    par_t, tok_t = torch.from_numpy(parent).cuda(), torch.from_numpy(token).cuda()
    g = _np(rsd.rsd_verify_tree_rule(draft, target, par_t, tok_t, L, rule, gamma, sampler, 31, 2, seq_base=7, want_theta=True))
    o = oracle.verify_tree(draft_h, workloads.as_oracle_rows(target), parent, token, L, 31, 2, seq_base=7,
                           rule=rule, gamma=gamma, final_sampler=sampler)
    t = Tally()
    compare_verify(t, g, o, parent)
    t.check()
    assert t.final_mismatch <= max(1, 0.02 * B)
    assert np.array_equal(g["status"], o["status"])
    assert len(set(o["accepted_len"].tolist())) > 1
    assert (o["stop_reason"] == 0).any()                       # some walks end in the rule's residual


def test_verify_tree_rule_rrs_is_verify_tree_and_bad_rules_are_refused(rsd):
    B, V, branching = 8, 515, (3, 2)
    parent = workloads.rsdc_parent_array(branching)
    base = _rows((B, len(parent), V), "f32", 2.0, 900)
    draft = base[:, :4].contiguous()
    target = (base + _rows((B, len(parent), V), "f32", 1.0, 901)).contiguous()
    _, token = _iid_tree(workloads.as_oracle_rows(draft), branching, 3)
    par_t, tok_t = torch.from_numpy(parent).cuda(), torch.from_numpy(token).cuda()
    a = _np(rsd.rsd_verify_tree(draft, target, par_t, tok_t, 2, 5, 0, want_theta=True))
    b = _np(rsd.rsd_verify_tree_rule(draft, target, par_t, tok_t, 2, rsd.RULE_RRS, 1.0, rsd.FINAL_INVERSE_CDF, 5, 0, want_theta=True))
    for k in a:
        assert np.array_equal(a[k], b[k], equal_nan=True), k
    with pytest.raises(rsd.RsdError):
        rsd.rsd_verify_tree_rule(draft, target, par_t, tok_t, 2, 7, 1.0, 0, 5, 0)
    with pytest.raises(rsd.RsdError):
        rsd.rsd_verify_tree_rule(draft, target, par_t, tok_t, 2, rsd.RULE_KSEQ, 0.5, 0, 5, 0)
    with pytest.raises(rsd.RsdError):
        rsd.rsd_verify_tree_rule(draft, target, par_t, tok_t, 2, rsd.RULE_RRS, 1.0, 3, 5, 0)


@pytest.mark.parametrize("dtype,V", [("f32", 140000), ("bf16", 262144)])
def test_verify_tree_longest_rows(rsd, dtype, V):
    # 4-byte rows of more than 131,072 entries are more than 64 chunks of the copy-engine ring: they take the other walk
    B, branching = 2, (2, 2)
    L = len(branching)
    n_nodes = len(workloads.rsdc_parent_array(branching))
    base = _rows((B, n_nodes, V), "f32", 2.5, 1500)
    draft = base[:, :3].to(torch.bfloat16 if dtype == "bf16" else torch.float32).contiguous()
    target = (base + _rows((B, n_nodes, V), "f32", 1.0, 1501)).to(draft.dtype).contiguous()
    draft_h = workloads.as_oracle_rows(draft)
    k, nodes = workloads.rsdc_rows(branching)
    parent = workloads.rsdc_parent_array(branching)
    token = workloads.rsdc_tokens_from_rows(branching, oracle.gumbel_topk(draft_h, k, nodes, 3, 1)["token"])
    g = _np(rsd.rsd_verify_tree(draft, target, torch.from_numpy(parent).cuda(), torch.from_numpy(token).cuda(), L, 3, 1,
                                want_theta=True))
    o = oracle.verify_tree(draft_h, workloads.as_oracle_rows(target), parent, token, L, 3, 1)
    t = Tally()
    compare_verify(t, g, o, parent)
    t.check()
    assert np.array_equal(g["status"], o["status"])


@pytest.mark.parametrize("dtype,V,branching", [("f32", 96, (4,)), ("bf16", 1000, (2, 2, 3)), ("f32", 33, (2, 1)),
                                               ("bf16", 515, (4, 1, 4)), ("bf16", 32000, (3, 2))])
def test_verify_tree_peaked_draft_flat_target(rsd, dtype, V, branching):
    # Draft at temperature 0.3 on wide logits, target at temperature 2: the first child often holds all but 1e-6 or
    # less of the draft mass and is rejected, so the thresholds of its siblings hang on 1 - P, the mass that is left.
    # Taken as a difference of rounded sums it would be noise; the thresholds must still agree with the oracle's.
    B = 24 if V <= 5000 else 6
    L = len(branching)
    n_nodes = len(workloads.rsdc_parent_array(branching))
    P = n_nodes - int(np.prod(branching))
    base = _rows((B, n_nodes, V), "f32", 3.0, 1300 + V)
    draft = base[:, :P].to(torch.bfloat16 if dtype == "bf16" else torch.float32).contiguous()
    target = (base + _rows((B, n_nodes, V), "f32", 2.0, 1301 + V)).to(draft.dtype).contiguous()
    draft_h = workloads.as_oracle_rows(draft)
    k, nodes = workloads.rsdc_rows(branching)
    parent = workloads.rsdc_parent_array(branching)
    t = Tally()
    small = 0
    for seed in range(4):
        token = workloads.rsdc_tokens_from_rows(
            branching, oracle.gumbel_topk(draft_h, k, nodes, seed, 2, seq_base=7, temperature=0.3)["token"])
        par_t, tok_t = torch.from_numpy(parent).cuda(), torch.from_numpy(token).cuda()
        g = _np(rsd.rsd_verify_tree(draft, target, par_t, tok_t, L, seed, 2, seq_base=7, want_theta=True,
                                    draft_temperature=0.3, target_temperature=2.0))
        o = oracle.verify_tree(draft_h, workloads.as_oracle_rows(target), parent, token, L, seed, 2, seq_base=7,
                               draft_temperature=0.3, target_temperature=2.0)
        compare_verify(t, g, o, parent)
        assert np.array_equal(g["status"], o["status"])
        # how peaked: draft mass outside the root's first child
        row = draft_h[:, 0].astype(np.float64) / 0.3
        pr = np.exp(row - row.max(axis=1, keepdims=True))
        pr /= pr.sum(axis=1, keepdims=True)
        small += int(np.sum(1.0 - pr[np.arange(B), token[:, 1]] < 1e-4))
    t.check()
    if V <= 100:
        assert small > 0          # the regime the test is about does occur


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_verify_tree_more_sequences_than_sms(rsd, dtype):
    # batches above one sequence per SM run the walk in blocks of 256 threads, smaller ones in blocks of 512: the
    # other verification tests here are small batches, this one is not
    B, V, branching = 200, 1030, (3, 2, 2)
    L = len(branching)
    parent = workloads.rsdc_parent_array(branching)
    n_nodes = len(parent)
    k, nodes = workloads.rsdc_rows(branching)
    base = _rows((B, n_nodes, V), "f32", 2.0, 1500)
    draft = base[:, :len(k)].to(torch.bfloat16 if dtype == "bf16" else torch.float32).contiguous()
    target = (base + _rows((B, n_nodes, V), "f32", 1.0, 1501)).to(draft.dtype).contiguous()
    o_draft = oracle.gumbel_topk(workloads.as_oracle_rows(draft), k, nodes, 29, 0)
    token = workloads.rsdc_tokens_from_rows(branching, o_draft["token"])
    g, o = _verify_both(rsd, draft, target, parent, token, L, 29, 0)
    t = Tally()
    compare_verify(t, g, o, parent)
    t.check()
    assert t.final_mismatch <= 0.02 * B
    assert np.array_equal(g["status"], o["status"])
