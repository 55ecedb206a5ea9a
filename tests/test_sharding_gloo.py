"""Host logic of the multi-GPU path on CPU: two gloo ranks split a batch by sequence; because the random streams
are keyed by the global sequence index, the shards' results concatenate to the single-process result."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import oracle
    import workloads
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = workloads.scaled(workloads.WORKLOADS[2], batch=5, vocab=300)
    lo, hi = workloads.shard_range(w.batch, rank, world)
    draft, _ = workloads.make_logits(w, step=3, device="cpu", seq_begin=lo, seq_end=hi)
    k, nodes = workloads.rsdc_rows(w.branching)
    d = oracle.gumbel_topk(workloads.as_oracle_rows(draft), k, nodes, 9, 3, seq_base=lo)
    np.save(os.path.join(out_dir, "tok%d.npy" % rank), d["token"])
    # the benchmark's reduction: slowest rank decides
    t = torch.tensor([10.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    assert t.item() == 10.0 + world - 1
    dist.barrier()
    dist.destroy_process_group()


def test_shard_ranges_cover_the_batch():
    sys.path.insert(0, ROOT)
    import workloads
    for batch in (1, 5, 64, 1024):
        for world in (1, 2, 3, 8):
            ranges = [workloads.shard_range(batch, r, world) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == batch
            assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
            sizes = [b - a for a, b in ranges]
            assert max(sizes) - min(sizes) <= 1


def test_two_ranks_reproduce_the_single_process_result(tmp_path):
    sys.path.insert(0, ROOT)
    import oracle
    import workloads
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    w = workloads.scaled(workloads.WORKLOADS[2], batch=5, vocab=300)
    draft, _ = workloads.make_logits(w, step=3, device="cpu")
    k, nodes = workloads.rsdc_rows(w.branching)
    full = oracle.gumbel_topk(workloads.as_oracle_rows(draft), k, nodes, 9, 3)
    parts = np.concatenate([np.load(tmp_path / ("tok%d.npy" % r)) for r in range(2)])
    assert np.array_equal(parts, full["token"])
