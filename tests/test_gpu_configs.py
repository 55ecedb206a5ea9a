"""The five benchmark workloads at full size: one draft + verify step on the GPU in the launch configuration the
benchmark times, compared with the oracle on every sequence (the large workloads in blocks of 128 sequences, which
bounds the host memory the oracle's copies of the rows take)."""
import os

import numpy as np
import pytest
import torch

import oracle
import workloads
from tests.parity import Tally, compare_topk, compare_verify

pytestmark = pytest.mark.gpu


def _np(d):
    return {k: (v.cpu().numpy() if isinstance(v, torch.Tensor) else v) for k, v in d.items() if v is not None}


def _oracle_step(w, draft_h, target_h, seed, step, seq_base):
    """Draft and verify a block of sequences with the oracle alone."""
    if w.mode == "rsd_c":
        k, nodes = workloads.rsdc_rows(w.branching)
        d = oracle.gumbel_topk(draft_h, k, nodes, seed, step, seq_base=seq_base)
        parent = workloads.rsdc_parent_array(w.branching)
        token = workloads.rsdc_tokens_from_rows(w.branching, d["token"])
        v = oracle.verify_tree(draft_h, target_h, parent, token, w.num_levels, seed, step, seq_base=seq_base)
        return dict(draft=d, parent=parent, token=token, verify=v)
    W, L = w.beam_width, w.depth
    nb = draft_h.shape[0]
    parent = np.full((nb, 1 + W * L), -1, np.int32)
    token = np.full((nb, 1 + W * L), -1, np.int32)
    levels, prev = [], None
    for l in range(L):
        first = 0 if l == 0 else 1 + (l - 1) * W
        n_par = 1 if l == 0 else W
        o = oracle.sbs_step(draft_h[:, first:first + n_par], W, first, None if l == 0 else prev["sum_logprob"],
                            None if l == 0 else prev["trunc_gumbel"], seed, step, is_logprob=w.draft_is_logprob,
                            seq_base=seq_base)
        sl = slice(1 + l * W, 1 + (l + 1) * W)
        token[:, sl] = o["token"]
        parent[:, sl] = np.where(o["parent"] >= 0, first + o["parent"], -1)
        levels.append(o)
        prev = o
    v = oracle.verify_tree(draft_h, target_h, parent, token, L, seed, step, seq_base=seq_base)
    return dict(levels=levels, parent=parent, token=token, verify=v)


def _compare_block(t, w, stepper, gpu_verify, ora, lo, hi):
    """Compare sequences lo..hi of the GPU step with the oracle's results for the same block."""
    nb = hi - lo
    if w.mode == "rsd_c":
        g_tok = stepper.draft_out["token"][lo:hi].cpu().numpy()
        bad = compare_topk(t, g_tok, ora["draft"], stepper.k_per_row)
        assert np.array_equal(stepper.token[lo:hi].cpu().numpy()[[b for b in range(nb) if b not in bad]],
                              ora["token"][[b for b in range(nb) if b not in bad]])
    else:
        W = w.beam_width
        g_token = stepper.token[lo:hi].cpu().numpy()
        g_parent = stepper.parent[lo:hi].cpu().numpy()
        bad = set()
        for l, lv in enumerate(ora["levels"]):
            sl = slice(1 + l * W, 1 + (l + 1) * W)
            for b in range(nb):
                if b in bad:
                    continue
                t.decisions += W
                if np.array_equal(g_token[b, sl], ora["token"][b, sl]) and np.array_equal(g_parent[b, sl], ora["parent"][b, sl]):
                    continue
                bad.add(b)
                if lv["margin"][b] <= 1e-5:
                    t.borderline += 1
                else:
                    t.failures.append(("sbs level", l, lo + b, g_token[b, sl].tolist(), ora["token"][b, sl].tolist(),
                                       float(lv["margin"][b])))
    g = {k: v[lo:hi] for k, v in gpu_verify.items()}
    compare_verify(t, g, ora["verify"], ora["parent"], skip_seq=bad)
    return bad


def _run_config(cid, steps, blocks, rows_ready=True):
    import paper_2402_14160_b200 as rsd
    from paper_2402_14160_b200 import step as rsd_step
    w = workloads.WORKLOADS[cid]
    stepper = rsd_step.make_step(w, rows_ready=rows_ready)
    t = Tally()
    acc_len = []
    for s in range(steps):
        draft, target = workloads.make_logits(w, step=s, device="cuda")
        seed = s if cid == 2 else 0                      # workload 2: a fresh seed every step
        gv = _np(stepper.run(draft, target, seed, s))
        torch.cuda.synchronize()
        assert np.all((gv["status"] & ~rsd.ST_ZERO_RESIDUAL) == 0)
        acc_len.append(gv["accepted_len"].mean())
        for lo, hi in blocks:
            dh = workloads.as_oracle_rows(draft[lo:hi])
            th = workloads.as_oracle_rows(target[lo:hi])
            ora = _oracle_step(w, dh, th, seed, s, seq_base=lo)
            _compare_block(t, w, stepper, gv, ora, lo, hi)
        del draft, target
    print("workload %d: %r mean accepted length %.3f" % (cid, t, float(np.mean(acc_len))))
    t.check()
    assert t.final_mismatch <= max(1, 0.01 * t.final_draws)
    return t


def test_workload_1_rsd_c_tiny():
    _run_config(1, 1, [(0, 1)])


def test_workload_2_rsd_c_batch():
    steps = 100 if os.environ.get("RSD_ALL_STEPS", "1") == "1" else 10
    t = _run_config(2, steps, [(0, 64)])
    assert t.decisions > 64 * 33 * steps


def test_workload_3_rsd_s():
    _run_config(3, 1, [(0, 32)])


def test_workload_3_rsd_s_level_by_level():
    _run_config(3, 1, [(0, 32)], rows_ready=False)      # one rsd_sbs_step call per level instead of rsd_sbs_draft_tree


def test_workload_4_opt_vocab_rsd_c():
    t = _run_config(4, 1, [(lo, lo + 128) for lo in range(0, 256, 128)])
    assert t.decisions > 256 * 60


def test_workload_5_serving_rsd_s():
    t = _run_config(5, 1, [(lo, lo + 128) for lo in range(0, 1024, 128)])
    assert t.decisions > 1024 * 64
