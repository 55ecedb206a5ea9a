"""Whole draft + verify steps and row filters on randomly drawn configurations (fixed seeds), against the oracle:
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
