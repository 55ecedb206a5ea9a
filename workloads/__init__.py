"""Seeded synthetic workloads for the RSD hot path.

Holds only input generation and tree-shape bookkeeping: no sampling, no
softmax-based decision, no rejection test.  Both the CUDA parity tests and the
CPU oracle read the tensors produced here, so the stored bytes are the single
source of truth for the two sides.

The five workloads stand in for the paper's Llama 2 (vocabulary 32000) and OPT
(vocabulary 50272) runs: draft logits are i.i.d. Gaussian, target logits are
the draft logits plus Gaussian noise, computed in fp32 and rounded once to the
storage dtype.  Tree shapes follow Appendix C.3 (constant branching factors,
or beam width and depth for Stochastic Beam Search).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    mode: str                      # "rsd_c" (constant branching) or "rsd_s" (stochastic beam search)
    batch: int                     # sequences per step
    vocab: int
    dtype: str                     # "f32" or "bf16" storage
    branching: Tuple[int, ...] = ()  # rsd_c: b_0 .. b_{L-1}
    beam_width: int = 0            # rsd_s: W
    depth: int = 0                 # rsd_s: L
    draft_sigma: float = 2.0
    noise_sigma: float = 0.5
    draft_is_logprob: bool = False
    peaked_fraction: float = 0.0   # fraction of target rows with one token raised by peaked_boost
    peaked_boost: float = 8.0
    steps: int = 1
    config_id: int = 0

    @property
    def num_levels(self) -> int:
        return len(self.branching) if self.mode == "rsd_c" else self.depth

    @property
    def level_sizes(self) -> List[int]:
        """N_0 = 1, N_1, ..., N_L."""
        if self.mode == "rsd_c":
            sizes = [1]
            for b in self.branching:
                sizes.append(sizes[-1] * b)
            return sizes
        return [1] + [self.beam_width] * self.depth

    @property
    def level_offsets(self) -> List[int]:
        """off_0 = 0 (root), off_1 = 1, ..., off_{L+1} = N + 1 (flat, level-major)."""
        off = [0]
        for n in self.level_sizes:
            off.append(off[-1] + n)
        return off

    @property
    def num_nodes(self) -> int:
        """N: non-root nodes."""
        return self.level_offsets[-1] - 1

    @property
    def num_parents(self) -> int:
        """P: nodes above the last level (root included); these need a draft row."""
        return self.level_offsets[-2]

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2


WORKLOADS = {
    1: Workload("rsd_c_tiny", "rsd_c", 1, 32000, "f32", branching=(2, 2, 2), draft_sigma=2.0, noise_sigma=0.5,
                steps=1, config_id=1),
    2: Workload("rsd_c_batch", "rsd_c", 64, 32000, "f32", branching=(3, 2, 2, 1), draft_sigma=2.0, noise_sigma=1.0,
                steps=100, config_id=2),
    3: Workload("rsd_s", "rsd_s", 32, 32000, "f32", beam_width=6, depth=6, draft_sigma=2.0, noise_sigma=0.7,
                draft_is_logprob=True, peaked_fraction=0.05, steps=1, config_id=3),
    4: Workload("opt_vocab_rsd_c", "rsd_c", 256, 50272, "bf16", branching=(4, 2, 2, 1, 1), draft_sigma=3.0,
                noise_sigma=0.5, steps=1, config_id=4),
    5: Workload("serving_rsd_s", "rsd_s", 1024, 32000, "bf16", beam_width=8, depth=8, draft_sigma=2.0,
                noise_sigma=0.8, steps=1, config_id=5),
}


def scaled(w: Workload, *, batch: Optional[int] = None, vocab: Optional[int] = None) -> Workload:
    """Same recipe at another batch size or vocabulary (for small parity cases)."""
    from dataclasses import replace
    return replace(w, batch=batch if batch is not None else w.batch, vocab=vocab if vocab is not None else w.vocab)


def _storage(t: torch.Tensor, dtype: str) -> torch.Tensor:
    return t.to(torch.bfloat16) if dtype == "bf16" else t.to(torch.float32)


def make_logits(w: Workload, step: int = 0, device: str = "cpu", seq_begin: int = 0, seq_end: Optional[int] = None,
                out_draft: Optional[torch.Tensor] = None, out_target: Optional[torch.Tensor] = None):
    """Draft rows [b, P, V] and target rows [b, N+1, V] for sequences seq_begin..seq_end of the workload.

    Every sequence has its own generator seed (1000003 * config + 1009 * step + sequence), so any subset of
    sequences can be produced alone and equals the same slice of the full batch on the same device type.
    """
    seq_end = w.batch if seq_end is None else seq_end
    nb = seq_end - seq_begin
    P, N1, V = w.num_parents, w.num_nodes + 1, w.vocab
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    draft = out_draft if out_draft is not None else torch.empty((nb, P, V), dtype=tdt, device=device)
    target = out_target if out_target is not None else torch.empty((nb, N1, V), dtype=tdt, device=device)
    gen = torch.Generator(device=device)
    for i in range(nb):
        b = seq_begin + i
        gen.manual_seed(1000003 * w.config_id + 1009 * step + b)
        base = torch.randn((N1, V), generator=gen, device=device, dtype=torch.float32) * w.draft_sigma
        if w.draft_is_logprob:
            base = torch.log_softmax(base, dim=-1)
        noise = torch.randn((N1, V), generator=gen, device=device, dtype=torch.float32) * w.noise_sigma
        tgt = base + noise
        if w.peaked_fraction > 0.0:
            pick = torch.rand((N1,), generator=gen, device=device) < w.peaked_fraction
            where = torch.randint(0, V, (N1,), generator=gen, device=device)
            rows = torch.nonzero(pick).flatten()
            tgt[rows, where[rows]] += w.peaked_boost
        draft[i].copy_(_storage(base[:P], w.dtype))
        target[i].copy_(_storage(tgt, w.dtype))
    return draft, target


def as_oracle_rows(t: torch.Tensor) -> np.ndarray:
    """Host view the oracle reads: fp32 arrays as they are, bf16 as their 16-bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


# ---------------------------------------------------------------------------
# tree-shape bookkeeping (Algorithm 3's lists, flattened)
# ---------------------------------------------------------------------------
def rsdc_parent_array(branching) -> np.ndarray:
    """Flat parent index of every node of a constant-branching tree (root: -1)."""
    sizes = [1]
    for b in branching:
        sizes.append(sizes[-1] * b)
    off = np.concatenate([[0], np.cumsum(sizes)])
    parent = np.full(off[-1], -1, dtype=np.int32)
    for l, b in enumerate(branching):
        for i in range(sizes[l + 1]):
            parent[off[l + 1] + i] = off[l] + i // b
    return parent


def rsdc_rows(branching):
    """(k_per_row, rng_node) for the P parent rows of a constant-branching tree: row r is flat node r."""
    sizes = [1]
    for b in branching:
        sizes.append(sizes[-1] * b)
    k = []
    for l, b in enumerate(branching):
        k += [b] * sizes[l]
    return np.asarray(k, dtype=np.int32), np.arange(len(k), dtype=np.int32)


def rsdc_tokens_from_rows(branching, row_tokens: np.ndarray) -> np.ndarray:
    """Scatter per-row picks [B, P, max_k] into the per-node token array [B, N+1] (root: -1).

    The children of parent row r at level l are the flat nodes off_{l+1} + (r - off_l) * b_l + j.
    """
    sizes = [1]
    for b in branching:
        sizes.append(sizes[-1] * b)
    off = np.concatenate([[0], np.cumsum(sizes)])
    B = row_tokens.shape[0]
    token = np.full((B, off[-1]), -1, dtype=np.int32)
    for l, b in enumerate(branching):
        for i in range(sizes[l]):
            r = off[l] + i
            for j in range(b):
                token[:, off[l + 1] + i * b + j] = row_tokens[:, r, j]
    return token


def shard_range(batch: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous block of sequences owned by `rank` (sizes differ by at most one)."""
    base, rem = divmod(batch, world)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)
