"""rsd_sbs_step_static: the Stochastic Beam Search level for callers that cannot allocate device memory.

A serving engine that fixes its memory pool at start-up, or a plug-in that is given a stream but no allocator, cannot
hand the library a scratch buffer.  The static entry point keeps its scratch inside the library, so it must give the
same answers as rsd_sbs_step with caller-owned scratch.  Checked on two calls in a row, because the built-in scratch
is shared by every call and keeps what the previous call left in it.  Runs last on purpose.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads
from tests.parity import Tally, compare_sbs_level

pytestmark = pytest.mark.gpu


def _outputs(B, W):
    return dict(token=torch.empty((B, W), dtype=torch.int32, device="cuda"),
                parent=torch.empty((B, W), dtype=torch.int32, device="cuda"),
                sum_logprob=torch.empty((B, W), dtype=torch.float32, device="cuda"),
                trunc_gumbel=torch.empty((B, W), dtype=torch.float32, device="cuda"),
                count=torch.empty((B,), dtype=torch.int32, device="cuda"),
                status=torch.empty((B,), dtype=torch.int32, device="cuda"))


def test_static_scratch_entry_point_matches_the_caller_scratch_one_twice():
    import paper_2402_14160_b200 as rsd
    rsd.lib()
    g = torch.Generator(device="cpu").manual_seed(77)
    W = 6
    # two calls in a row with different shapes, so the second finds the first one's leftovers in the scratch
    cases = [((9, 1, 4099), 0, False, 3), ((5, W, 2000), 1, True, 4)]
    done = 0
    for shape, first_node, with_state, step in cases:
        rows = (torch.randn(shape, generator=g) * 2.0).to(torch.bfloat16).cuda()
        B = shape[0]
        sig = gam = None
        if with_state:
            sig = -torch.rand((B, W), generator=g).cuda() * 5.0
            gam = -torch.sort(torch.rand((B, W), generator=g), dim=1).values.cuda()
        ref = rsd.rsd_sbs_step(rows, W, first_node, sig, gam, 21, step, seq_base=3, parent_base=first_node)
        outs = _outputs(B, W)
        torch.cuda.synchronize()
        # the property the entry point exists for: the call takes no device memory, neither from torch's pool nor
        # from the driver (the first call on a device only looks an address up)
        torch_before, (free_before, _) = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()
        rsd.rsd_sbs_step_static(rows, W, first_node, sig, gam, 21, step, outs, seq_base=3, parent_base=first_node)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == torch_before   # (no name is rebound in between: nothing is freed either)
        got = outs
        if done > 0:   # (the very first call on a device may still page the library's image in)
            assert torch.cuda.mem_get_info()[0] >= free_before
        for key in ("token", "parent", "count", "status"):
            assert torch.equal(ref[key], got[key]), key
        for key in ("sum_logprob", "trunc_gumbel"):
            a, b = ref[key].cpu().numpy().astype(np.float64), got[key].cpu().numpy().astype(np.float64)
            assert np.all(np.abs(a - b) <= 1e-6 + 1e-5 * np.abs(a)), key
        assert int(got["count"].min()) == W
        # and against the oracle itself, decision by decision with its margins
        host = workloads.as_oracle_rows(rows)
        o = oracle.sbs_step(host, W, first_node, None if sig is None else sig.cpu().numpy(),
                            None if gam is None else gam.cpu().numpy(), 21, step, seq_base=3)
        o["parent"] = np.where(o["parent"] >= 0, o["parent"] + first_node, -1)    # (parent_base of the call)
        t = Tally()
        compare_sbs_level(t, {k: v.cpu().numpy() for k, v in got.items()}, o, W, set())
        t.check()
        done += 1
    assert done == 2


def test_static_scratch_entry_point_rejects_oversized_calls():
    import paper_2402_14160_b200 as rsd
    rows = torch.zeros((1, 1, 64), dtype=torch.float32, device="cuda")
    B, n_par, W = 4096, 8, 8                                   # 4096 * 8 * 8 * 8 bytes > 1 MiB
    assert rsd.rsd_sbs_workspace_bytes(B, n_par, W) > rsd.api.SBS_STATIC_SCRATCH_BYTES
    big = rows.expand(B, n_par, 64)
    with pytest.raises(rsd.RsdError, match="built-in scratch"):
        rsd.rsd_sbs_step_static(big, W, 1, None, None, 0, 0, _outputs(B, W))


def test_static_scratch_entry_point_takes_the_largest_documented_batch():
    # B = 1024, n_par = 8, W = 8 needs 851,968 bytes: the example the header gives as fitting
    import paper_2402_14160_b200 as rsd
    B, n_par, W, V = 1024, 8, 8, 256
    assert rsd.rsd_sbs_workspace_bytes(B, n_par, W) == 851968 <= rsd.api.SBS_STATIC_SCRATCH_BYTES
    g = torch.Generator(device="cpu").manual_seed(5)
    rows = (torch.randn((B, n_par, V), generator=g) * 2.0).cuda()
    sig = -torch.rand((B, n_par), generator=g).cuda() * 3.0
    gam = -torch.sort(torch.rand((B, n_par), generator=g), dim=1).values.cuda()
    ref = rsd.rsd_sbs_step(rows, W, 1, sig, gam, 2, 9, parent_base=1)
    got = rsd.rsd_sbs_step_static(rows, W, 1, sig, gam, 2, 9, _outputs(B, W), parent_base=1)
    torch.cuda.synchronize()
    for key in ("token", "parent", "count", "status"):
        assert torch.equal(ref[key], got[key]), key
    for key in ("sum_logprob", "trunc_gumbel"):
        assert torch.allclose(ref[key], got[key], rtol=1e-5, atol=1e-6), key


def test_static_scratch_entry_point_names_argument_errors_before_the_size():
    import paper_2402_14160_b200 as rsd
    rows = torch.zeros((1, 1, 64), dtype=torch.float32, device="cuda").expand(2, 300, 64)
    with pytest.raises(rsd.RsdError, match="n_par = 300"):
        rsd.rsd_sbs_step_static(rows, 4, 1, None, None, 0, 0, _outputs(2, 4))
