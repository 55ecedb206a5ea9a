"""Comparison rules for GPU-vs-oracle parity.

A decision (a pick of the sorted top-k, an accept/reject test, the final draw) must agree with the oracle unless
the oracle's margin for it is at most MARGIN; such borderline disagreements are counted, and what follows them in
the same sequence is skipped because it legitimately differs.
"""
import numpy as np

MARGIN = 1e-5
REL_TOL = 1e-5


class Tally:
    def __init__(self):
        self.decisions = 0
        self.borderline = 0
        self.failures = []
        self.final_draws = 0
        self.final_mismatch = 0

    def check(self):
        assert not self.failures, "hard mismatches: %s" % self.failures[:5]
        assert self.borderline <= max(1e-4 * self.decisions, 0 if self.decisions >= 10000 else 1), \
            "borderline %d of %d decisions" % (self.borderline, self.decisions)

    def __repr__(self):
        return "decisions=%d borderline=%d failures=%d final=%d/%d" % (
            self.decisions, self.borderline, len(self.failures), self.final_mismatch, self.final_draws)


def close(gpu, ref, rel=REL_TOL, abs_tol=1e-6):
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    both_inf = np.isinf(gpu) & np.isinf(ref) & (np.sign(gpu) == np.sign(ref))
    both_nan = np.isnan(gpu) & np.isnan(ref)
    ok = both_inf | both_nan | (np.abs(gpu - ref) <= abs_tol + rel * np.abs(ref))
    return ok


def compare_topk(tally, gpu_token, ora, k_per_row, gpu_perturbed=None, gpu_logprob=None, skip_seq=None,
                 logprob_abs_tol=1e-6):
    """Row-wise: picks must match in order; a mismatching row is borderline iff the oracle's smallest gap <= MARGIN.

    logprob_abs_tol: a log-probability (and a perturbed one) is value / T - LSE in fp32; when those two terms are large
    (low temperature) each carries half an ulp of its own size, which the caller passes here."""
    B, R, _ = gpu_token.shape
    bad_seq = set()
    for b in range(B):
        if skip_seq is not None and b in skip_seq:
            continue
        for r in range(R):
            k = int(k_per_row[r])
            tally.decisions += k
            if np.array_equal(gpu_token[b, r], ora["token"][b, r]):
                if gpu_perturbed is not None:
                    ok = close(gpu_perturbed[b, r, :k], ora["perturbed"][b, r, :k], abs_tol=logprob_abs_tol)
                    if not ok.all():
                        tally.failures.append(("perturbed", b, r, gpu_perturbed[b, r, :k], ora["perturbed"][b, r, :k]))
                if gpu_logprob is not None:
                    ok = close(gpu_logprob[b, r, :k], ora["logprob"][b, r, :k], abs_tol=logprob_abs_tol)
                    if not ok.all():
                        tally.failures.append(("logprob", b, r, gpu_logprob[b, r, :k], ora["logprob"][b, r, :k]))
                continue
            bad_seq.add(b)
            if ora["margin"][b, r] <= MARGIN:
                tally.borderline += 1
            else:
                tally.failures.append(("topk", b, r, gpu_token[b, r].tolist(), ora["token"][b, r].tolist(),
                                       float(ora["margin"][b, r])))
    return bad_seq


def compare_sbs_level(tally, gpu, ora, W, skip_seq):
    """One SBS level; returns the sequences that diverged here (to be skipped at later levels)."""
    B = gpu["token"].shape[0]
    bad = set()
    for b in range(B):
        if b in skip_seq:
            continue
        tally.decisions += W
        same = (np.array_equal(gpu["token"][b], ora["token"][b]) and np.array_equal(gpu["parent"][b], ora["parent"][b])
                and gpu["count"][b] == ora["count"][b])
        if same:
            ok = close(gpu["sum_logprob"][b], ora["sum_logprob"][b]) & close(gpu["trunc_gumbel"][b], ora["trunc_gumbel"][b])
            if not ok.all():
                tally.failures.append(("sbs values", b, gpu["sum_logprob"][b], ora["sum_logprob"][b],
                                       gpu["trunc_gumbel"][b], ora["trunc_gumbel"][b]))
            continue
        bad.add(b)
        if ora["margin"][b] <= MARGIN:
            tally.borderline += 1
        else:
            tally.failures.append(("sbs", b, gpu["token"][b].tolist(), ora["token"][b].tolist(),
                                   gpu["parent"][b].tolist(), ora["parent"][b].tolist(), float(ora["margin"][b])))
    return bad


def compare_verify(tally, gpu, ora, parent, skip_seq=None):
    """Walk comparison.  gpu/ora: dicts of numpy arrays; parent: [N+1] or [B, N+1] flat parent indices."""
    B = len(ora["accepted_len"])
    for b in range(B):
        if skip_seq is not None and b in skip_seq:
            continue
        par = parent if parent.ndim == 1 else parent[b]
        tested = ~np.isnan(ora["margin"][b])
        tally.decisions += int(tested.sum()) + 1
        tally.final_draws += 1
        gl, ol = int(gpu["accepted_len"][b]), int(ora["accepted_len"][b])
        gp, op = gpu["accepted_node"][b, :gl].tolist(), ora["accepted_node"][b, :ol].tolist()
        if gp == op:
            if gpu.get("theta") is not None:
                ok = close(gpu["theta"][b][tested], ora["theta"][b][tested], abs_tol=1e-6)
                if not ok.all():
                    tally.failures.append(("theta", b, gpu["theta"][b][tested], ora["theta"][b][tested]))
            if not np.array_equal(gpu["accepted_token"][b], ora["accepted_token"][b]):
                tally.failures.append(("accepted_token", b))
            if gpu["stop_reason"][b] != ora["stop_reason"][b]:
                tally.failures.append(("stop_reason", b, int(gpu["stop_reason"][b]), int(ora["stop_reason"][b])))
            if gpu["last_token"][b] != ora["last_token"][b]:
                tally.final_mismatch += 1
                if ora["final_margin"][b] <= MARGIN:
                    tally.borderline += 1
                else:
                    tally.failures.append(("last_token", b, int(gpu["last_token"][b]), int(ora["last_token"][b]),
                                           float(ora["final_margin"][b])))
            continue
        # first level where the paths part: its parent node is common to both walks
        i = 0
        while i < min(gl, ol) and gp[i] == op[i]:
            i += 1
        node = 0 if i == 0 else op[i - 1]
        sibs = [c for c in range(1, len(par)) if par[c] == node and tested[c]]
        m = min([ora["margin"][b, c] for c in sibs], default=np.inf)
        if m <= MARGIN:
            tally.borderline += 1
        else:
            tally.failures.append(("path", b, gp, op, float(m)))
