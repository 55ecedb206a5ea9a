"""One draft + verify step over resident logits, as a fixed sequence of librsd calls.

These classes only own buffers and issue the C-ABI calls in order (Algorithm 2 for constant branching factors,
Algorithm 7 for Stochastic Beam Search, with the language-model calls replaced by rows that already sit in device
memory).  The drafting calls write the tree's token/parent arrays in place, so no tensor work happens between the
library's kernels.
"""
from __future__ import annotations

from typing import Sequence

import torch

from . import api


class RsdCStep:
    """RSD with constant branching factors b = (b_0, ..., b_{L-1}) for a batch of B sequences."""

    def __init__(self, B: int, V: int, branching: Sequence[int], device="cuda"):
        self.B, self.V, self.branching = B, V, tuple(int(b) for b in branching)
        self.L = len(self.branching)
        sizes = [1]
        for b in self.branching:
            sizes.append(sizes[-1] * b)
        off = [0]
        for n in sizes:
            off.append(off[-1] + n)
        self.level_offsets = off
        self.P, self.n_nodes = off[-2], off[-1]
        k, child_base, parent = [], [], [-1] * self.n_nodes
        for l, b in enumerate(self.branching):
            for i in range(sizes[l]):
                k.append(b)
                child_base.append(off[l + 1] + i * b)
                for j in range(b):
                    parent[off[l + 1] + i * b + j] = off[l] + i
        self.k_per_row, self.child_base = k, child_base
        self.rng_node = list(range(self.P))
        self.max_k = max(k)
        self.parent = torch.tensor(parent, dtype=torch.int32, device=device)
        self.token = api._new((B, self.n_nodes), torch.int32, device).fill_(-1)
        self.draft_out = dict(token=api._new((B, self.P, self.max_k), torch.int32, device),
                              status=api._new((B,), torch.int32, device), perturbed=None, logprob=None)
        self.verify_out = None
        self.kernel_launches = 2  # one scan, one walk

    def run(self, draft: torch.Tensor, target: torch.Tensor, seed: int, step: int, seq_base: int = 0):
        api.rsd_gumbel_topk_draft(draft, self.k_per_row, self.rng_node, seed, step, seq_base=seq_base,
                                  max_k=self.max_k, child_base=self.child_base, node_token=self.token,
                                  out=self.draft_out)
        self.verify_out = api.rsd_verify_tree(draft, target, self.parent, self.token, self.L, seed, step,
                                              seq_base=seq_base, out=self.verify_out)
        return self.verify_out


class RsdSStep:
    """RSD with Stochastic Beam Search of width W and depth L for a batch of B sequences.

    rows_ready=True: the draft rows of every level exist before drafting starts (rows attached to tree slots), so the
    whole tree is drafted by rsd_sbs_draft_tree in two launches; otherwise one rsd_sbs_step call per level."""

    def __init__(self, B: int, V: int, W: int, L: int, draft_is_logprob: bool = False, device="cuda",
                 rows_ready: bool = True):
        self.B, self.V, self.W, self.L, self.is_logprob = B, V, W, L, draft_is_logprob
        self.rows_ready = rows_ready
        self.n_nodes = 1 + W * L
        self.P = 1 + W * (L - 1)
        self.parent = api._new((B, self.n_nodes), torch.int32, device).fill_(-1)
        self.token = api._new((B, self.n_nodes), torch.int32, device).fill_(-1)
        self.state = [dict(sum_logprob=api._new((B, W), torch.float32, device),
                           trunc_gumbel=api._new((B, W), torch.float32, device)) for _ in range(2)]
        self.count = api._new((L, B), torch.int32, device)
        self.status = api._new((L, B), torch.int32, device)
        self.workspace = api._new((max(api.rsd_sbs_workspace_bytes(B, W, W), api.rsd_sbs_tree_workspace_bytes(B, W, L)),),
                                  torch.uint8, device)
        self.tree_out = dict(sum_logprob=self.state[0]["sum_logprob"], trunc_gumbel=self.state[0]["trunc_gumbel"],
                             count=self.count, status=api._new((B,), torch.int32, device))
        self.verify_out = None
        # one scan over all rows, one launch for the levels, one walk; or per level one scan and one epilogue
        self.kernel_launches = 3 if rows_ready else 2 * L + 1

    def level_slice(self, l: int):
        return slice(1 + l * self.W, 1 + (l + 1) * self.W)

    def draft_tree(self, draft: torch.Tensor, seed: int, step: int, seq_base: int = 0):
        """All levels at once (rows_ready)."""
        return api.rsd_sbs_draft_tree(draft, self.W, self.L, seed, step, self.token, self.parent,
                                      is_logprob=self.is_logprob, seq_base=seq_base, workspace=self.workspace,
                                      out=self.tree_out)

    def run(self, draft: torch.Tensor, target: torch.Tensor, seed: int, step: int, seq_base: int = 0):
        W = self.W
        if self.rows_ready:
            self.draft_tree(draft, seed, step, seq_base)
            self.verify_out = api.rsd_verify_tree(draft, target, self.parent, self.token, self.L, seed, step,
                                                  seq_base=seq_base, out=self.verify_out)
            return self.verify_out
        for l in range(self.L):
            first = 0 if l == 0 else 1 + (l - 1) * W
            n_par = 1 if l == 0 else W
            prev, cur = self.state[(l + 1) % 2], self.state[l % 2]
            sl = self.level_slice(l)
            out = dict(token=self.token[:, sl], parent=self.parent[:, sl], sum_logprob=cur["sum_logprob"],
                       trunc_gumbel=cur["trunc_gumbel"], count=self.count[l], status=self.status[l])
            api.rsd_sbs_step(draft[:, first:first + n_par], W, first, None if l == 0 else prev["sum_logprob"],
                             None if l == 0 else prev["trunc_gumbel"], seed, step, is_logprob=self.is_logprob,
                             seq_base=seq_base, workspace=self.workspace, out=out, parent_base=first)
        self.verify_out = api.rsd_verify_tree(draft, target, self.parent, self.token, self.L, seed, step,
                                              seq_base=seq_base, out=self.verify_out)
        return self.verify_out


def make_step(w, batch=None, device="cuda", rows_ready=True):
    """Step object for a workloads.Workload description."""
    B = w.batch if batch is None else batch
    if w.mode == "rsd_c":
        return RsdCStep(B, w.vocab, w.branching, device=device)
    return RsdSStep(B, w.vocab, w.beam_width, w.depth, draft_is_logprob=w.draft_is_logprob, device=device,
                    rows_ready=rows_ready)
