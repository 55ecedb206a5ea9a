#!/usr/bin/env python
"""Benchmark of the RSD hot path: draft + verify steps per second over resident synthetic logits.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..5] [--impl reference]

One step = one pass of the whole hot path over one batch: every drafting level (Gumbel-Top-k scan, or L Stochastic
Beam Search levels) and the recursive-rejection-sampling walk.  Prints one JSON line (rank 0).
With N > 1 every rank runs the same per-GPU batch on its own sequences (weak scaling, no collective on the data
path; the global sequence index keys the random streams).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads  # noqa: E402

# DRAM bytes moved per algorithmic byte by the scan kernel, from the committed ncu summary of the scan kernel
# (dram__bytes_read + dram__bytes_write over rows x V x 2 bytes; the traffic grows in proportion to the rows scanned),
# together with the SHA-256 of the kernel sources it was measured on: when the sources differ, `traffic` is null.
SCAN_TRAFFIC_PER_ALGORITHMIC_BYTE = 1.006
SCAN_TRAFFIC_SOURCES = ("paper_2402_14160_b200/csrc/rsd_scan.cuh", "paper_2402_14160_b200/csrc/rsd_device.cuh")
SCAN_TRAFFIC_SOURCE_SHA256 = "574f6d40fefe2ebb6d1b18716b7cae63a2fc958d6c5241f54ac24a9a039aaa7a"


def _scan_sources_sha256():
    import hashlib
    h = hashlib.sha256()
    for rel in SCAN_TRAFFIC_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


METRIC = "verified tree nodes/sec"
UNIT = "nodes/s"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    return 6650.0, "fallback (profiling recipe)"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, device_index: int):
        self.samples, self.reasons, self.max_mhz, self.ok = [], set(), None, False
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            self._nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:  # NVML missing: report that, never fail the run
            self.error = repr(e)

    def _loop(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.001)

    def __enter__(self):
        if self.ok:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                    "note": getattr(self, "error", "no samples")}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def _oracle_sample_step(w, draft_h, target_h, seed, step, seq_base):
    """One draft + verify step of the oracle over a block of sequences (host arrays).  Returns the walk's outputs
    plus `draft_margin` [b]: the smallest gap of any drafting decision of the sequence."""
    import oracle
    if w.mode == "rsd_c":
        k, nodes = workloads.rsdc_rows(w.branching)
        d = oracle.gumbel_topk(draft_h, k, nodes, seed, step, seq_base=seq_base)
        parent = workloads.rsdc_parent_array(w.branching)
        token = workloads.rsdc_tokens_from_rows(w.branching, d["token"])
        v = oracle.verify_tree(draft_h, target_h, parent, token, w.num_levels, seed, step, seq_base=seq_base)
        v["draft_margin"] = d["margin"].min(axis=1)
        v["tree_token"] = token
        return v
    W, L = w.beam_width, w.depth
    nb = draft_h.shape[0]
    parent = np.full((nb, 1 + W * L), -1, np.int32)
    token = np.full((nb, 1 + W * L), -1, np.int32)
    margin = np.full(nb, np.inf)
    prev = None
    for l in range(L):
        first = 0 if l == 0 else 1 + (l - 1) * W
        n_par = 1 if l == 0 else W
        o = oracle.sbs_step(draft_h[:, first:first + n_par], W, first, None if l == 0 else prev["sum_logprob"],
                            None if l == 0 else prev["trunc_gumbel"], seed, step, is_logprob=w.draft_is_logprob,
                            seq_base=seq_base)
        sl = slice(1 + l * W, 1 + (l + 1) * W)
        token[:, sl] = o["token"]
        parent[:, sl] = np.where(o["parent"] >= 0, first + o["parent"], -1)
        margin = np.minimum(margin, o["margin"])
        prev = o
    v = oracle.verify_tree(draft_h, target_h, parent, token, L, seed, step, seq_base=seq_base)
    v["draft_margin"] = margin
    v["tree_token"] = token
    return v


def _time_oracle(w, n_seq, steps, warmup, threads=None, rows=None):
    """Oracle on the host cores over the first n_seq sequences of the workload (generated on the host, or the given
    (draft, target) tensors); returns (nodes/s, seconds/step, threads used, outputs of the last step)."""
    import oracle
    oracle.build()
    if threads is not None:
        oracle.set_num_threads(threads)
    if rows is None:
        draft, target = workloads.make_logits(w, step=0, device="cpu", seq_begin=0, seq_end=n_seq)
    else:
        draft, target = rows[0][:n_seq], rows[1][:n_seq]
    dh, th = workloads.as_oracle_rows(draft), workloads.as_oracle_rows(target)
    for s in range(warmup):
        _oracle_sample_step(w, dh, th, 0, s, 0)
    t0 = time.perf_counter()
    out = None
    for s in range(steps):
        out = _oracle_sample_step(w, dh, th, 0, warmup + s, 0)
    dt = (time.perf_counter() - t0) / max(steps, 1)
    used = threads if threads is not None else oracle.num_threads()
    if threads is not None:
        oracle.set_num_threads(oracle.num_threads())
    return n_seq * w.num_nodes / dt, dt, used, out


def _parity_sample(gpu, tree_token, ora, margin=1e-5):
    """Sequences of the sample whose GPU step differs from the oracle's, split by the oracle's smallest margin."""
    n = len(ora["accepted_len"])
    differ = borderline = 0
    for b in range(n):
        same = (np.array_equal(tree_token[b], ora["tree_token"][b]) and gpu["accepted_len"][b] == ora["accepted_len"][b]
                and np.array_equal(gpu["accepted_node"][b], ora["accepted_node"][b])
                and gpu["last_token"][b] == ora["last_token"][b])
        if same:
            continue
        differ += 1
        m = min(float(ora["draft_margin"][b]), float(np.nanmin(np.append(ora["margin"][b], np.inf))),
                float(ora["final_margin"][b]))
        borderline += 1 if m <= margin else 0
    return {"sequences": n, "differ": differ, "of_which_borderline": borderline,
            "note": "one step (seed 0, step 0) of the GPU path against the oracle on the cpu_baseline sample; a "
                    "sequence differs if its tree, accepted path or last token does; borderline = the oracle's smallest "
                    "decision margin of that sequence is <= 1e-5"}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_seq = min(w.batch, args.ref_sequences)
    value, dt, cores, _ = _time_oracle(w, n_seq, args.steps, args.warmup)
    sample = "%d of %d sequences of workload %d per step, whole draft+verify step" % (n_seq, w.batch, w.config_id)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "workload_id": w.config_id, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", type=int, default=5, choices=sorted(workloads.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--ref-sequences", type=int, default=16)
    ap.add_argument("--cpu-baseline-sequences", type=int, default=256)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--sequences", type=int, default=0, help="sequences per GPU (default: the workload's batch)")
    ap.add_argument("--top-p", type=float, default=1.0, help="nucleus filtering of the draft and target rows in every step (1: off)")
    ap.add_argument("--top-k", type=int, default=0, help="top-k filtering of the draft and target rows in every step (0: off)")
    ap.add_argument("--per-level", action="store_true",
                    help="Stochastic Beam Search: one rsd_sbs_step call per level instead of rsd_sbs_draft_tree")
    args = ap.parse_args()
    w = workloads.WORKLOADS[args.workload]
    if args.sequences > 0:
        w = workloads.scaled(w, batch=args.sequences)

    if args.impl == "reference":
        if args.steps > 20:
            args.steps = 20
        run_reference(args, w)
        return

    from paper_2402_14160_b200 import api, step as rsd_step

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the hot path has no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    api.lib()

    # weak scaling: every rank owns a full per-GPU batch; its global sequence indices start at rank * B
    B = w.batch
    seq_base = rank * B
    draft, target = workloads.make_logits(w, step=0, device=str(dev), seq_begin=0, seq_end=B)
    stepper = rsd_step.make_step(w, device=dev, rows_ready=not args.per_level)
    is_sbs = w.mode == "rsd_s"
    L = w.num_levels
    resident_bytes = draft.numel() * draft.element_size() + target.numel() * target.element_size()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # optional logit warping: the rows of every step go through rsd_filter_rows first (two more launches per step)
    warp_rows = args.top_p < 1.0 or args.top_k > 0
    raw_draft, raw_target = draft, target
    filt = None
    if warp_rows:
        filt = [api.rsd_filter_rows(raw_draft, args.top_k, args.top_p), api.rsd_filter_rows(raw_target, args.top_k, args.top_p)]
        draft, target = filt[0]["rows"], filt[1]["rows"]
        filter_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]

    def warp_step(s=None):
        if warp_rows:
            if s is not None:
                filter_ev[s][0].record()
            api.rsd_filter_rows(raw_draft, args.top_k, args.top_p, out=filt[0])
            api.rsd_filter_rows(raw_target, args.top_k, args.top_p, out=filt[1])
            if s is not None:
                filter_ev[s][1].record()

    for s in range(max(args.warmup, 3)):
        warp_step()
        stepper.run(draft, target, 0, s, seq_base)
    barrier()

    # ---- timed region: K steps, events on the launching stream -------------------------------------------
    K = args.steps
    per_level = is_sbs and args.per_level
    n_scan = (L if per_level else 1)

    def ev():
        e = torch.cuda.Event(enable_timing=True)
        e.record()          # creates the handle
        return e

    scan_ev = [[(ev(), ev()) for _ in range(n_scan)] for _ in range(K)]
    ver_ev = [(ev(), ev()) for _ in range(K)]
    step_ev = [ev() for _ in range(K + 1)]
    barrier()
    with ClockSampler(local) as clocks:
        step_ev[0].record()
        for s in range(K):
            warp_step(s)
            if per_level:
                W = stepper.W
                for l in range(L):
                    first = 0 if l == 0 else 1 + (l - 1) * W
                    n_par = 1 if l == 0 else W
                    prev, cur = stepper.state[(l + 1) % 2], stepper.state[l % 2]
                    sl = stepper.level_slice(l)
                    out = dict(token=stepper.token[:, sl], parent=stepper.parent[:, sl],
                               sum_logprob=cur["sum_logprob"], trunc_gumbel=cur["trunc_gumbel"],
                               count=stepper.count[l], status=stepper.status[l])
                    api.rsd_profile_next_scan(*scan_ev[s][l])
                    api.rsd_sbs_step(draft[:, first:first + n_par], W, first,
                                     None if l == 0 else prev["sum_logprob"], None if l == 0 else prev["trunc_gumbel"],
                                     0, 1000 + s, is_logprob=w.draft_is_logprob, seq_base=seq_base,
                                     workspace=stepper.workspace, out=out, parent_base=first)
            elif is_sbs:
                api.rsd_profile_next_scan(*scan_ev[s][0])
                stepper.draft_tree(draft, 0, 1000 + s, seq_base)
            else:
                api.rsd_profile_next_scan(*scan_ev[s][0])
                api.rsd_gumbel_topk_draft(draft, stepper.k_per_row, stepper.rng_node, 0, 1000 + s, seq_base=seq_base,
                                          max_k=stepper.max_k, child_base=stepper.child_base,
                                          node_token=stepper.token, out=stepper.draft_out)
            ver_ev[s][0].record()
            stepper.verify_out = api.rsd_verify_tree(draft, target, stepper.parent, stepper.token, L, 0, 1000 + s,
                                                     seq_base=seq_base, out=stepper.verify_out)
            ver_ev[s][1].record()
            step_ev[s + 1].record()
        torch.cuda.synchronize()
    elapsed_ms = step_ev[0].elapsed_time(step_ev[K])
    per_step_ms = [step_ev[i].elapsed_time(step_ev[i + 1]) for i in range(K)]
    barrier()
    if dist is not None:
        t = torch.tensor([elapsed_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed_ms = float(t.item())

    nodes_per_step = world * B * w.num_nodes
    value = nodes_per_step * K / (elapsed_ms * 1e-3)

    # ---- roofline of the dominant kernel: the row scan of the drafting calls ---------------------------------
    scan_ms = sum(a.elapsed_time(b) for row in scan_ev for a, b in row)
    ver_ms = sum(a.elapsed_time(b) for a, b in ver_ev)
    rows_scanned = B * w.num_parents               # every parent row is read once per step
    scan_bytes_per_step = rows_scanned * w.vocab * w.elem_bytes
    peak, peak_kind = _peaks()
    scan_gbs = scan_bytes_per_step * K / (scan_ms * 1e-3) / 1e9
    out = stepper.verify_out
    acc = out["accepted_len"].cpu().numpy()
    reason = out["stop_reason"].cpu().numpy()
    # rows the walk had to read: two per visited node with children, one for the final target row otherwise
    rows_walk = int(np.sum(np.where(reason == 0, 2 * acc + 2, 2 * acc + 1)))
    ver_bytes = rows_walk * w.vocab * w.elem_bytes
    ver_gbs = ver_bytes / (ver_ms / K * 1e-3) / 1e9
    roofline = {"kernel": "scan_topk_kernel (Gumbel-Top-k / SBS parent-row scan)", "bound": "hbm",
                "achieved": scan_gbs, "peak": peak, "unit": "GB/s", "frac": scan_gbs / peak, "peak_kind": peak_kind,
                "traffic": (SCAN_TRAFFIC_PER_ALGORITHMIC_BYTE * scan_bytes_per_step / n_scan
                            if _scan_sources_sha256() == SCAN_TRAFFIC_SOURCE_SHA256 else None),
                "traffic_note": "DRAM bytes per scan launch (average over the step's launches), scaled by rows from a "
                                "256-sequence ncu capture (14,592 rows in one launch); null when the kernel sources "
                                "changed since that capture",
                "algorithmic_bytes_per_step": scan_bytes_per_step,
                "launches_per_step": n_scan, "avg_launch_ms": scan_ms / (K * n_scan),
                "launch_ms_by_level": [sum(scan_ev[s][l][0].elapsed_time(scan_ev[s][l][1]) for s in range(K)) / K
                                       for l in range(n_scan)],
                "share_of_step": scan_ms / elapsed_ms,
                "frac_of_nominal_8000_gbs": scan_gbs / 8000.0,
                "verify_walk": {"achieved": ver_gbs, "frac": ver_gbs / peak, "frac_of_nominal_8000_gbs": ver_gbs / 8000.0,
                                "algorithmic_bytes_last_step": ver_bytes,
                                "avg_launch_ms": ver_ms / K, "share_of_step": ver_ms / elapsed_ms}}
    # the same nodes counted against the drafting launches alone (scans; SBS epilogues excluded) and the walk alone,
    # timed on this rank
    phases = {"draft_scan_only_nodes_per_s": nodes_per_step * K / (scan_ms * 1e-3),
              "verify_only_nodes_per_s": nodes_per_step * K / (ver_ms * 1e-3)}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3),
            "ms_per_step": elapsed_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "workload_id": w.config_id, "mode": w.mode, "sequences_per_gpu": B,
                       "nodes_per_sequence": w.num_nodes, "vocab": w.vocab, "storage": w.dtype,
                       "tree": ({"beam_width": w.beam_width, "depth": w.depth} if is_sbs
                                else {"branching": list(w.branching)}),
                       "l2": "inputs larger than L2 (%.2f GB resident per GPU)" % (resident_bytes / 1e9)
                       if resident_bytes > 256e6 else "inputs smaller than L2: timings are cache-assisted",
                       "drafting": ("rsd_sbs_step per level" if per_level else
                                    "rsd_sbs_draft_tree (all levels, rows ready)" if is_sbs else "rsd_gumbel_topk_draft"),
                       "logit_warping": ({"top_k": args.top_k, "top_p": args.top_p,
                                          "filter_ms_per_step": sum(a.elapsed_time(b) for a, b in filter_ev) / K,
                                          "rows_filtered_per_step": B * (w.num_parents + w.num_nodes + 1)}
                                         if warp_rows else None),
                       "mean_accepted_len": float(acc.mean())},
            "clocks": clocks.summary(), "gpu_launches": (stepper.kernel_launches + (2 if warp_rows else 0)) * K, "roofline": roofline,
            "phases": phases,
            "step_ms": {"mean": elapsed_ms / K, "median": float(np.median(per_step_ms)), "best": float(np.min(per_step_ms)),
                        "note": "per-step CUDA-event times on this rank; `value` uses the mean (max over ranks)"},
            "accepted_len_histogram": np.bincount(acc, minlength=L + 1).tolist(),
            "block_efficiency": float(acc.mean()) + 1.0}

    # ---- two batches in flight (not the headline): the same steps, alternating between two streams -----------------
    # A serving engine that decodes two batches at once lets one batch's row scan fill the SMs that the other batch's
    # last, longest walks leave idle.  Both batches read the same resident rows here; trees, seeds and results are
    # their own.
    if world == 1 and not per_level and not warp_rows:
        streams = [torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)]
        steppers = [stepper, rsd_step.make_step(w, device=dev, rows_ready=True)]
        for s in range(4):
            with torch.cuda.stream(streams[s % 2]):
                steppers[s % 2].run(draft, target, 0, 500 + s, seq_base)
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for st in streams:
            st.wait_event(t0)
        for s in range(K):
            with torch.cuda.stream(streams[s % 2]):
                steppers[s % 2].run(draft, target, 0, 2000 + s, seq_base)
        for st in streams:
            torch.cuda.current_stream().wait_stream(st)
        t1.record()
        torch.cuda.synchronize()
        two_ms = t0.elapsed_time(t1)
        line["two_batches_in_flight"] = {
            "value": nodes_per_step * K / (two_ms * 1e-3), "unit": UNIT, "ms_per_step": two_ms / K,
            "note": "the same K steps issued alternately on two streams (two independent batches over the same resident "
                    "rows): one batch's scan overlaps the other's walk; `value` above is one batch at a time"}

    # ---- end to end: pinned host logits -> device -> step -> results on the host ---------------------------
    if not args.no_e2e:
        h_draft = torch.empty(draft.shape, dtype=draft.dtype, pin_memory=True)
        h_target = torch.empty(target.shape, dtype=target.dtype, pin_memory=True)
        h_draft.copy_(raw_draft)
        h_target.copy_(raw_target)
        res_host = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True)
                    for k, v in stepper.verify_out.items() if v is not None}
        Ke = max(1, args.e2e_steps)

        def e2e_step(s):
            raw_draft.copy_(h_draft, non_blocking=True)
            raw_target.copy_(h_target, non_blocking=True)
            warp_step()
            o = stepper.run(draft, target, 0, 2000 + s, seq_base)
            for k2, v in res_host.items():
                v.copy_(o[k2], non_blocking=True)

        e2e_step(0)
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for s in range(Ke):
            e2e_step(1 + s)
        b.record()
        torch.cuda.synchronize()
        e2e_ms = a.elapsed_time(b)
        if dist is not None:
            t = torch.tensor([e2e_ms], device=dev, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e2e_ms = float(t.item())
        line["e2e"] = {"value": nodes_per_step * Ke / (e2e_ms * 1e-3), "unit": UNIT,
                       "h2d_bytes_per_step": int(resident_bytes),
                       "d2h_bytes_per_step": int(sum(v.numel() * v.element_size() for v in res_host.values())),
                       "steps": Ke, "ms_per_step": e2e_ms / Ke}
        del h_draft, h_target

    # ---- the oracle on the host cores, bounded sample (rank 0, one GPU only) ----------------------------------
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n_seq = min(B, args.cpu_baseline_sequences)
        v, dt, cores, ora = _time_oracle(w, n_seq, 1, 0, rows=(draft, target))   # the rows the GPU holds
        n_one = max(1, min(n_seq, args.cpu_baseline_sequences // 32))
        v1, dt1, _, _ = _time_oracle(w, n_one, 1, 0, threads=1)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": "%d of %d sequences, one whole draft+verify step (%.1f s)" % (n_seq, B, dt),
                                "single_thread": {"value": v1, "unit": UNIT,
                                                  "sample": "%d sequences, one step (%.1f s)" % (n_one, dt1)}}
        # the same step on the GPU, compared with what the oracle just computed
        gv = stepper.run(draft, target, 0, 0, 0)
        torch.cuda.synchronize()
        g = {k2: v2[:n_seq].cpu().numpy() for k2, v2 in gv.items() if v2 is not None}
        line["parity_sample"] = _parity_sample(g, stepper.token[:n_seq].cpu().numpy(), ora)
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
