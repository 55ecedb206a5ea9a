"""The scan kernel's overflow paths (candidate queue full, too many elements above the bound) give the same picks.

A variant of the library is built with tiny queues (-DRSD_SCAN_SMALL_QUEUES), so that ordinary rows overflow every
queue, and is compared with the oracle in a child process (the binding loads one library per process)."""
import os
import subprocess
import sys
import tempfile

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, %(root)r)
import numpy as np, torch
import oracle, workloads
import paper_2402_14160_b200 as rsd
from tests.parity import Tally, compare_topk
rsd.lib()
t = Tally()
for V, dtype, k in [(4099, torch.float32, [1, 8, 32]), (32000, torch.bfloat16, [4, 8, 32]), (70, torch.float32, [2, 16, 32])]:
    g = torch.Generator().manual_seed(V)
    rows = (torch.randn((4, 3, V), generator=g) * 2).to(dtype).cuda()
    kk = [min(V, x) for x in k]
    out = rsd.rsd_gumbel_topk_draft(rows, kk, [0, 5, 9], 3, 1, max_k=max(kk), want_values=True)
    o = oracle.gumbel_topk(workloads.as_oracle_rows(rows), kk, [0, 5, 9], 3, 1, max_k=max(kk))
    compare_topk(t, out["token"].cpu().numpy(), o, kk, out["perturbed"].cpu().numpy(), out["logprob"].cpu().numpy())
    assert np.array_equal(out["status"].cpu().numpy(), o["status"])
t.check()
print("ok", t)
"""


def test_small_queue_build_matches_the_oracle():
    from paper_2402_14160_b200 import build
    with tempfile.TemporaryDirectory() as d:
        lib = build.build(out=os.path.join(d, "librsd_small_queues.so"), defines=("RSD_SCAN_SMALL_QUEUES",))
        env = dict(os.environ, RSD_LIB_PATH=lib)
        r = subprocess.run([sys.executable, "-c", CHILD % {"root": ROOT}], env=env, capture_output=True, text=True,
                           timeout=600)
        assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
        assert "ok" in r.stdout
