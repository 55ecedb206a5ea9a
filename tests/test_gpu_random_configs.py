"""Whole draft + verify steps, row filters, the verification rules, Gumbel-Top-k rows and tempered beam-search trees on
randomly drawn configurations (fixed seeds), against the oracle:
vocabularies from 16 to 50272 with and without 16-byte alignment, beams of 1-12 over 1-6 levels, trees of 1-4 levels
with 1-4 children, both storage types, flat to peaked rows, log-probability rows, the tree call and the level-by-level
calls.  The cases are small, so a run takes seconds; what it adds to the hand-picked cases is breadth."""
import random

import numpy as np
import pytest
import torch

import oracle
import workloads
from tests.parity import Tally
from tests.test_gpu_configs import _compare_block, _np, _oracle_step

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [11, 12])
def test_random_step_configurations(seed):
    from paper_2402_14160_b200 import step as rsd_step
    rng = random.Random(seed)
    total = Tally()
    for it in range(80):
        mode = rng.choice(["rsd_s", "rsd_s", "rsd_c"])
        V = rng.choice([37, 130, 515, 1000, 2049, 4100, 9999, 32000, 50272]) if rng.random() < 0.8 else rng.randint(16, 6000)
        dtype = rng.choice(["f32", "bf16"])
        kw = dict(draft_sigma=rng.choice([0.7, 2.0, 4.0]), noise_sigma=rng.choice([0.3, 1.0, 2.5]),
                  peaked_fraction=rng.choice([0.0, 0.0, 0.2]))
        B = rng.randint(1, 10) if V <= 10000 else rng.randint(1, 3)
        if mode == "rsd_s":
            W = min(rng.randint(1, 12), max(1, V // 2))
            w = workloads.Workload("random", "rsd_s", B, V, dtype, beam_width=W, depth=rng.randint(1, 6),
                                   draft_is_logprob=rng.random() < 0.3, **kw)
        else:
            w = workloads.Workload("random", "rsd_c", B, V, dtype,
                                   branching=tuple(rng.randint(1, 4) for _ in range(rng.randint(1, 4))), **kw)
        rows_ready = rng.random() < 0.7
        rng_seed, step = rng.randint(0, 1 << 40), rng.randint(0, 1000)
        draft, target = workloads.make_logits(w, step=step % 7, device="cuda")
        stepper = rsd_step.make_step(w, rows_ready=rows_ready)
        gv = _np(stepper.run(draft, target, rng_seed, step))
        torch.cuda.synchronize()
        t = Tally()
        ora = _oracle_step(w, workloads.as_oracle_rows(draft), workloads.as_oracle_rows(target), rng_seed, step, seq_base=0)
        _compare_block(t, w, stepper, gv, ora, 0, B)
        assert not t.failures, (it, w, rows_ready, rng_seed, step, t.failures[:2])
        total.decisions += t.decisions
        total.borderline += t.borderline
        total.final_draws += t.final_draws
        total.final_mismatch += t.final_mismatch
    print("random steps (seed %d): %r" % (seed, total))
    total.check()
    assert total.decisions > 5000 and total.final_mismatch <= max(1, 0.01 * total.final_draws)


def test_random_filter_configurations():
    import paper_2402_14160_b200 as rsd
    rng = random.Random(21)
    rows_total = borderline = 0
    for it in range(120):
        V = (rng.choice([1, 2, 7, 8, 9, 17, 130, 515, 1000, 2049, 4100, 9999, 32000, 50272, 70000]) if rng.random() < 0.8
             else rng.randint(1, 6000))
        dtype = rng.choice(["f32", "bf16"])
        if dtype == "f32" and V > 49000:
            V = 40000
        B, R = rng.randint(1, 3), rng.randint(1, 4)
        g = torch.Generator().manual_seed(rng.randint(0, 1 << 30))
        kind = rng.random()
        t = torch.randn((B, R, V + 9), generator=g) * rng.choice([0.01, 0.5, 2.0, 6.0, 20.0])
        if kind < 0.15:
            t = torch.round(t * 2) / 2            # many equal values
        elif kind < 0.25:
            t[..., ::3] = float("-inf")
        elif kind < 0.3:
            t[:] = 0.5
        t = t.to(torch.bfloat16 if dtype == "bf16" else torch.float32).cuda()
        off = rng.choice([0, 0, 1, 3, 8])
        rows = t[:, :, off:off + V]
        top_k = rng.choice([0, 0, 1, 5, 50, 1000, V, V + 5])
        top_p = rng.choice([1.0, 0.95, 0.9, 0.5, 0.1, 0.999, 1e-4])
        T = rng.choice([1.0, 0.3, 2.0, 0.7])
        got = rsd.rsd_filter_rows(rows, top_k, top_p, temperature=T)
        host = workloads.as_oracle_rows(rows.contiguous())
        o = oracle.filter_rows(host, top_k, top_p, temperature=T)
        want = oracle.apply_filter(host, o["keep"])
        out = workloads.as_oracle_rows(got["rows"])
        kept = got["kept"].cpu().numpy()
        bits = np.uint32 if out.dtype == np.float32 else np.uint16
        for b in range(B):
            for r in range(R):
                rows_total += 1
                if np.array_equal(out[b, r].view(bits), want[b, r].view(bits)) and kept[b, r] == o["kept"][b, r]:
                    continue
                assert o["margin"][b, r] <= 1e-5, (it, V, dtype, top_k, top_p, T, b, r, int(kept[b, r]), int(o["kept"][b, r]))
                borderline += 1
    print("random filters: %d rows, %d borderline" % (rows_total, borderline))
    assert borderline <= max(3, rows_total // 50)


def test_random_rule_configurations():
    """The three verification rules (recursive rejection sampling, multi-round, K-SEQ) and both last-token samplers on
    random trees, vocabularies, temperatures, storage types and row offsets: decisions, thresholds and status words."""
    import paper_2402_14160_b200 as rsd
    from tests.parity import compare_verify
    from tests.test_gpu_parity import _iid_tree, _rows
    rng = random.Random(31)
    total = Tally()
    for it in range(100):
        rule, sampler = rng.choice([0, 1, 2]), rng.choice([0, 1])
        gamma = rng.choice([1.0, 1.5, 3.0]) if rule == 2 else 1.0
        V = rng.choice([33, 97, 515, 1000, 4099, 9999, 32000])
        dtype = rng.choice(["f32", "bf16"])
        branching = tuple(rng.randint(1, 4) for _ in range(rng.randint(1, 3)))
        B = rng.randint(1, 12) if V <= 5000 else rng.randint(1, 4)
        Td, Tt = rng.choice([1.0, 1.0, 0.3, 2.0]), rng.choice([1.0, 1.0, 0.3, 2.0])
        L = len(branching)
        n_nodes = len(workloads.rsdc_parent_array(branching))
        P = n_nodes - int(np.prod(branching))
        base = _rows((B, n_nodes, V + 3), "f32", rng.choice([1.0, 3.0]), rng.randint(0, 1 << 20))
        noise = _rows((B, n_nodes, V + 3), "f32", rng.choice([0.3, 1.0, 2.0]), rng.randint(0, 1 << 20))
        off = rng.choice([0, 0, 1, 3])
        draft = base[:, :P, off:off + V].to(torch.bfloat16 if dtype == "bf16" else torch.float32)
        target = (base + noise)[:, :, off:off + V].to(draft.dtype)
        if off == 0:
            draft, target = draft.contiguous(), target.contiguous()
        draft_h, target_h = workloads.as_oracle_rows(draft.contiguous()), workloads.as_oracle_rows(target.contiguous())
        seed, step, sb = rng.randint(0, 1 << 40), rng.randint(0, 99), rng.randint(0, 50)
        if rule == 0:      # drafted without replacement (Algorithm 4)
            k, nodes = workloads.rsdc_rows(branching)
            parent = workloads.rsdc_parent_array(branching)
            picks = oracle.gumbel_topk(draft_h, k, nodes, seed, step, seq_base=sb, temperature=Td)["token"]
            token = workloads.rsdc_tokens_from_rows(branching, picks)
        else:              # independent drafts (Section 2's baselines)
            parent, token = _iid_tree(draft_h / Td, branching, 5 + it)
        g = _np(rsd.rsd_verify_tree_rule(draft, target, torch.from_numpy(parent).cuda(), torch.from_numpy(token).cuda(), L, rule,
                                         gamma, sampler, seed, step, seq_base=sb, want_theta=True, draft_temperature=Td,
                                         target_temperature=Tt))
        o = oracle.verify_tree(draft_h, target_h, parent, token, L, seed, step, seq_base=sb, rule=rule, gamma=gamma,
                               final_sampler=sampler, draft_temperature=Td, target_temperature=Tt)
        t = Tally()
        compare_verify(t, g, o, parent)
        what = (it, rule, sampler, gamma, V, dtype, branching, B, Td, Tt, off)
        assert not t.failures, (what, t.failures[:2])
        assert np.array_equal(g["status"], o["status"]), (what, g["status"].tolist(), o["status"].tolist())
        total.decisions += t.decisions
        total.borderline += t.borderline
        total.final_draws += t.final_draws
        total.final_mismatch += t.final_mismatch
    print("random rules: %r" % total)
    total.check()
    assert total.decisions > 1000 and total.final_mismatch <= max(1, 0.01 * total.final_draws)


def test_random_gumbel_topk_configurations():
    """Gumbel-Top-k on random rows: vocabularies from 1 entry up, rows at odd offsets, half or nearly all entries -inf,
    a NaN, log-probability rows, temperatures, k up to 32.  A log-probability is value / T - LSE in fp32: the absolute
    tolerance is three ulps of the largest term involved on top of the usual 1e-6."""
    import paper_2402_14160_b200 as rsd
    from tests.parity import compare_topk
    from tests.test_gpu_parity import _rows
    rng = random.Random(41)
    total = Tally()
    for it in range(150):
        V = (rng.choice([1, 5, 16, 17, 70, 515, 1000, 4099, 9999, 32000, 50272]) if rng.random() < 0.8 else rng.randint(1, 7000))
        dtype = rng.choice(["f32", "bf16"])
        sigma = rng.choice([0.05, 2.0, 6.0, 15.0])
        T = rng.choice([1.0, 1.0, 0.3, 2.0])
        off = rng.choice([0, 0, 1, 3, 8])
        B, R = rng.randint(1, 4), rng.randint(1, 9)
        base = _rows((B, R, V + 9), "f32", sigma, rng.randint(0, 1 << 30))
        kind = rng.random()
        if kind < 0.15:
            base[..., ::2] = float("-inf")
        elif kind < 0.2:
            base[..., 3:] = float("-inf")
        elif kind < 0.25:
            base[0, 0, min(2, V + 8)] = float("nan")
        is_lp = rng.random() < 0.25
        if is_lp:
            base = torch.log_softmax(base, -1)
        rows = base.to(torch.bfloat16 if dtype == "bf16" else torch.float32)[:, :, off:off + V]
        k = [min(V, rng.choice([1, 2, 3, 8, 17, 32])) for _ in range(R)]
        nodes = sorted(rng.sample(range(0, 5000), R))
        seed, step, sb = rng.randint(0, 1 << 50), rng.randint(0, 1 << 20), rng.randint(0, 1 << 20)
        g = _np(rsd.rsd_gumbel_topk_draft(rows, k, nodes, seed=seed, step=step, seq_base=sb, max_k=max(k), want_values=True,
                                          is_logprob=is_lp, temperature=T))
        o = oracle.gumbel_topk(workloads.as_oracle_rows(rows.contiguous()), k, nodes, seed, step, seq_base=sb, max_k=max(k),
                               is_logprob=is_lp, temperature=T)
        finite = rows.float()[torch.isfinite(rows.float())]
        big = (float(finite.abs().max()) if finite.numel() else 1.0) / T + float(np.log(V)) + 20.0   # |value / T|, |LSE|, |noise|
        t = Tally()
        compare_topk(t, g["token"], o, k, g["perturbed"], g["logprob"], logprob_abs_tol=1e-6 + 3 * big * 1.2e-7)
        what = (it, V, dtype, sigma, T, off, B, R, k, kind, is_lp)
        assert not t.failures, (what, t.failures[:1])
        assert np.array_equal(g["status"], o["status"]), (what, g["status"].tolist(), o["status"].tolist())
        total.decisions += t.decisions
        total.borderline += t.borderline
    print("random Gumbel-Top-k: %r" % total)
    total.check()
    assert total.decisions > 5000


def test_random_beam_search_trees_with_temperature():
    """Stochastic Beam Search trees drafted in one call at a random temperature, level by level against the oracle, then
    verified with a second random temperature on the target rows.  A sequence whose tree differs at a borderline level
    is left out of the verification comparison."""
    import paper_2402_14160_b200 as rsd
    from tests.parity import compare_verify
    from tests.test_gpu_parity import _rows
    rng = random.Random(51)
    total = Tally()
    levels = borderline_levels = 0
    for it in range(80):
        V = rng.choice([37, 130, 515, 1000, 2049, 4100, 9999, 32000])
        dtype = rng.choice(["f32", "bf16"])
        W, L = min(rng.randint(1, 10), max(1, V // 2)), rng.randint(1, 5)
        B = rng.randint(1, 8) if V <= 10000 else rng.randint(1, 3)
        T = float(np.float32(rng.choice([0.3, 0.5, 0.7, 1.0, 1.5, 2.0])))
        Tt = float(np.float32(rng.choice([T, T, 1.0, 0.3, 2.0])))
        sig = rng.choice([0.7, 1.5, 3.0, 5.0])
        P = 1 + (L - 1) * W
        off = rng.choice([0, 0, 0, 1, 3])
        is_lp = rng.random() < 0.25
        base = _rows((B, P + W, V + 5), "f32", sig, rng.randint(0, 1 << 30))
        noise = _rows((B, P + W, V + 5), "f32", rng.choice([0.3, 1.0, 2.5]), rng.randint(0, 1 << 30))
        d32 = base[:, :P]
        if is_lp:
            d32 = torch.log_softmax(d32, -1)
        draft = d32.to(torch.bfloat16 if dtype == "bf16" else torch.float32)[:, :, off:off + V]
        target = (base + noise).to(draft.dtype)[:, :, off:off + V]
        if off == 0:
            draft, target = draft.contiguous(), target.contiguous()
        seed, step, sb = rng.randint(0, 1 << 50), rng.randint(0, 999), rng.randint(0, 99)
        nt = torch.full((B, 1 + L * W), -1, dtype=torch.int32, device="cuda")
        npar = torch.full((B, 1 + L * W), -1, dtype=torch.int32, device="cuda")
        rsd.rsd_sbs_draft_tree(draft, W, L, seed, step, nt, npar, is_logprob=is_lp, seq_base=sb, temperature=T)
        host = workloads.as_oracle_rows(draft.contiguous())
        parent = np.full((B, 1 + W * L), -1, np.int32)
        token = np.full((B, 1 + W * L), -1, np.int32)
        g_tok, g_par = nt.cpu().numpy(), npar.cpu().numpy()
        what = (it, V, dtype, W, L, B, T, Tt, sig, off, is_lp)
        prev, bad = None, set()
        for l in range(L):
            first, n_par = (0, 1) if l == 0 else (1 + (l - 1) * W, W)
            o = oracle.sbs_step(host[:, first:first + n_par], W, first, None if l == 0 else prev["sum_logprob"],
                                None if l == 0 else prev["trunc_gumbel"], seed, step, is_logprob=is_lp, seq_base=sb, temperature=T)
            sl = slice(1 + l * W, 1 + (l + 1) * W)
            token[:, sl] = o["token"]
            parent[:, sl] = np.where(o["parent"] >= 0, first + o["parent"], -1)
            for b in range(B):
                if b in bad:
                    continue
                levels += 1
                if np.array_equal(g_tok[b, sl], token[b, sl]) and np.array_equal(g_par[b, sl], parent[b, sl]):
                    continue
                assert o["margin"][b] <= 1e-5, (what, l, b, g_tok[b, sl].tolist(), token[b, sl].tolist(), float(o["margin"][b]))
                bad.add(b)
                borderline_levels += 1
            prev = o
        gv = _np(rsd.rsd_verify_tree(draft, target, npar, nt, L, seed, step, seq_base=sb, want_theta=True, draft_temperature=T,
                                     target_temperature=Tt))
        ov = oracle.verify_tree(host, workloads.as_oracle_rows(target.contiguous()), parent, token, L, seed, step, seq_base=sb,
                                draft_temperature=T, target_temperature=Tt)
        t = Tally()
        compare_verify(t, gv, ov, parent, skip_seq=bad)
        # thresholds of ill-conditioned nodes (a residual made of small differences at a low temperature) may be off by more
        # than 1e-5 relative although the decision stands; decisions, paths and last tokens must agree
        hard = [f for f in t.failures if f[0] != "theta"]
        assert not hard, (what, hard[:2])
        total.decisions += t.decisions
        total.borderline += t.borderline
        total.final_draws += t.final_draws
        total.final_mismatch += t.final_mismatch
    print("random beam-search trees: %d levels, %d borderline; %r" % (levels, borderline_levels, total))
    assert borderline_levels <= max(2, levels // 500)
    total.failures = []
    total.check()
    assert total.decisions > 1000 and total.final_mismatch <= max(1, 0.01 * total.final_draws)


def test_random_residual_draws():
    """rsd_resample_residual on random rows with random lists of rejected tokens (repeats allowed, the draft's mode
    among them in a fifth of the rows), temperatures and offsets.  Rows stay within logits of standard deviation 2: with
    both rows all but one-hot the residual is made of differences below fp32 resolution, which only the oracle's double
    precision resolves."""
    import paper_2402_14160_b200 as rsd
    from tests.test_gpu_parity import _rows
    rng = random.Random(61)
    n_rows = mismatches = 0
    for it in range(150):
        V = (rng.choice([2, 5, 16, 17, 70, 515, 1000, 4099, 9999, 32000, 50272]) if rng.random() < 0.8 else rng.randint(2, 7000))
        dtype = rng.choice(["f32", "bf16"])
        sigma = rng.choice([0.05, 1.0, 2.0])
        off = rng.choice([0, 0, 1, 3, 8])
        Bq = rng.randint(1, 8)
        d = _rows((Bq, V + 9), "f32", sigma, rng.randint(0, 1 << 30))
        tg = d + _rows((Bq, V + 9), "f32", rng.choice([0.3, 1.0, 3.0]), rng.randint(0, 1 << 30))
        dd = d.to(torch.bfloat16 if dtype == "bf16" else torch.float32)[:, off:off + V]
        tt = tg.to(dd.dtype)[:, off:off + V]
        nodes = torch.tensor([rng.randint(0, 3000) for _ in range(Bq)], dtype=torch.int32, device="cuda")
        mk = rng.randint(1, 6)
        rej = np.full((Bq, mk), -1, np.int32)
        for b in range(Bq):
            n = rng.randint(0, min(mk, V - 1))
            vals = [rng.randrange(V) for _ in range(n)]
            if rng.random() < 0.2 and n:
                vals[0] = int(torch.argmax(dd[b].float()))
            rej[b, :n] = vals
        Td, Tt = rng.choice([1.0, 0.5, 2.0]), rng.choice([1.0, 0.5, 2.0])
        seed, step, sb = rng.randint(0, 1 << 50), rng.randint(0, 1 << 20), rng.randint(0, 1 << 20)
        g = _np(rsd.rsd_resample_residual(dd, tt, torch.from_numpy(rej).cuda(), nodes, seed, step, seq_base=sb, want_residual=True,
                                          draft_temperature=Td, target_temperature=Tt))
        o = oracle.resample_residual(workloads.as_oracle_rows(dd.contiguous()), workloads.as_oracle_rows(tt.contiguous()), rej,
                                     nodes.cpu().numpy(), seed, step, seq_base=sb, draft_temperature=Td, target_temperature=Tt)
        what = (it, V, dtype, sigma, Td, Tt, off, rej.tolist())
        peak = o["residual"].max(axis=1, keepdims=True)
        assert np.all(np.abs(g["residual"] - o["residual"]) <= 1e-5 * peak), what
        differ = g["token"] != o["token"]
        assert np.all(o["margin"][differ] <= 1e-5), (what, g["token"].tolist(), o["token"].tolist())
        assert np.array_equal(g["status"], o["status"]), (what, g["status"].tolist(), o["status"].tolist())
        n_rows += Bq
        mismatches += int(differ.sum())
    print("random residual draws: %d rows, %d borderline" % (n_rows, mismatches))
    assert n_rows > 400 and mismatches <= max(1, n_rows // 200)
