"""Thin binding over librsd's C ABI (include/rsd.h): argument marshalling only.

Every function takes torch CUDA tensors, passes their device pointers and the current CUDA stream to the entry
point of the same name, and returns freshly allocated output tensors.  Nothing is computed here.  The library is
loaded on first use and a missing or unbuilt library raises: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("RSD_LIB_PATH") or os.path.join(_HERE, "librsd.so")  # override: a variant build

RSD_F32, RSD_BF16 = 0, 1
ST_NAN_INPUT, ST_FEWER_THAN_K, ST_ZERO_RESIDUAL, ST_ZERO_DRAFT_PROB, ST_DRAFT_EXHAUSTED, ST_TIMEOUT = 1, 2, 4, 8, 16, 32
STOP_ALL_REJECTED, STOP_NO_CHILDREN, STOP_LEAF = 0, 1, 2
RULE_RRS, RULE_MULTIROUND, RULE_KSEQ = 0, 1, 2
FINAL_INVERSE_CDF, FINAL_GUMBEL_TOP1 = 0, 1
MAX_K = 32

EXPORTS = ["rsd_version", "rsd_rng_layout", "rsd_last_error", "rsd_profile_next_scan", "rsd_filter_rows", "rsd_gumbel_topk_draft", "rsd_sbs_workspace_bytes",
           "rsd_sbs_step", "rsd_sbs_step_static", "rsd_sbs_tree_workspace_bytes", "rsd_sbs_draft_tree", "rsd_verify_tree", "rsd_verify_tree_rule", "rsd_resample_residual"]


class RsdRows(C.Structure):
    _fields_ = [("data", C.c_void_p), ("dtype", C.c_int32), ("is_logprob", C.c_int32),
                ("seq_stride", C.c_int64), ("row_stride", C.c_int64), ("temperature", C.c_float)]


class RsdTree(C.Structure):
    _fields_ = [("num_levels", C.c_int32), ("num_nodes", C.c_int32), ("parent", C.c_void_p),
                ("token", C.c_void_p), ("topology_is_shared", C.c_int32)]


class RsdError(RuntimeError):
    pass


_lib = None


def lib():
    """The loaded library.  Raises if it has not been built (python -m paper_2402_14160_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RsdError("librsd.so is missing at %s: build it with `python -m paper_2402_14160_b200.build` "
                           "(there is no fallback path)" % LIB_PATH)
        l = C.CDLL(LIB_PATH)
        l.rsd_last_error.restype = C.c_char_p
        l.rsd_profile_next_scan.argtypes = [C.c_void_p, C.c_void_p]
        l.rsd_sbs_workspace_bytes.restype = C.c_size_t
        l.rsd_sbs_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int]
        l.rsd_gumbel_topk_draft.argtypes = [C.POINTER(RsdRows), C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                            C.c_int, C.c_uint64, C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        l.rsd_sbs_step.argtypes = [C.POINTER(RsdRows), C.c_int, C.c_int, C.c_int, C.c_int, C.c_int32, C.c_void_p,
                                   C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p,
                                   C.c_int64, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                   C.c_void_p, C.c_size_t, C.c_void_p]
        l.rsd_filter_rows.argtypes = [C.POINTER(RsdRows), C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, C.c_void_p,
                                      C.c_void_p, C.c_void_p, C.c_void_p]
        l.rsd_sbs_tree_workspace_bytes.restype = C.c_size_t
        l.rsd_sbs_tree_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int]
        l.rsd_sbs_draft_tree.argtypes = [C.POINTER(RsdRows), C.c_int, C.c_int, C.c_int, C.c_int, C.c_uint64, C.c_uint32,
                                         C.c_uint32, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        l.rsd_sbs_step_static.argtypes = [C.POINTER(RsdRows), C.c_int, C.c_int, C.c_int, C.c_int, C.c_int32,
                                          C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint32, C.c_void_p,
                                          C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_void_p]
        l.rsd_verify_tree.argtypes = [C.POINTER(RsdRows), C.POINTER(RsdRows), C.POINTER(RsdTree), C.c_int, C.c_int,
                                      C.c_uint64, C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        l.rsd_verify_tree_rule.argtypes = [C.POINTER(RsdRows), C.POINTER(RsdRows), C.POINTER(RsdTree), C.c_int, C.c_int,
                                           C.c_int, C.c_float, C.c_int, C.c_uint64, C.c_uint32, C.c_uint32, C.c_void_p,
                                           C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.c_void_p]
        l.rsd_resample_residual.argtypes = [C.POINTER(RsdRows), C.POINTER(RsdRows), C.c_int, C.c_int, C.c_void_p,
                                            C.c_int, C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint32, C.c_void_p,
                                            C.c_void_p, C.c_void_p, C.c_void_p]
        _lib = l
    return _lib


def _check(code: int):
    if code != 0:
        raise RsdError("librsd error %d: %s" % (code, lib().rsd_last_error().decode()))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def rows_of(t: torch.Tensor, is_logprob: bool = False, temperature: float = 1.0) -> RsdRows:
    """Describe a [B, R, V] (or [B, V]) CUDA tensor of fp32 or bf16 rows; the last dimension must be dense."""
    if not t.is_cuda:
        raise RsdError("rows must live on a CUDA device")
    if t.dtype == torch.float32:
        dt = RSD_F32
    elif t.dtype == torch.bfloat16:
        dt = RSD_BF16
    else:
        raise RsdError("rows must be float32 or bfloat16")
    if t.stride(-1) != 1:
        raise RsdError("rows must be dense along the vocabulary")
    if t.dim() == 3:
        return RsdRows(t.data_ptr(), dt, int(is_logprob), t.stride(0), t.stride(1), float(temperature))
    if t.dim() == 2:
        return RsdRows(t.data_ptr(), dt, int(is_logprob), t.stride(0), t.shape[1], float(temperature))
    raise RsdError("rows must be [B, R, V] or [B, V]")


def _new(shape, dtype, device):
    """Every output tensor this package allocates comes from here (one place, so that the tests can surround each of
    them with guard words and check that no kernel writes outside its outputs)."""
    return torch.empty(shape, dtype=dtype, device=device)


def _host_i32(values: Sequence[int]):
    arr = (C.c_int32 * len(values))(*[int(v) for v in values])
    return arr


def rsd_filter_rows(rows: torch.Tensor, top_k: int = 0, top_p: float = 1.0, *, temperature: float = 1.0,
                    out: Optional[dict] = None):
    """rows [B, R, V] -> dict(rows [B, R, V] with -inf at the entries that top-k / nucleus filtering removes, kept [B, R],
    status [B]).  Pass the result to the drafting and verification calls in place of the rows, with the same temperature."""
    B, R, V = rows.shape
    dev = rows.device
    if out is None:
        out = dict(rows=_new((B, R, V), rows.dtype, dev), kept=_new((B, R), torch.int32, dev),
                   status=_new((B,), torch.int32, dev))
    if not out["rows"].is_contiguous() or out["rows"].dtype != rows.dtype:
        raise RsdError("out rows must be contiguous and of the rows' dtype")
    r = rows_of(rows, False, temperature)
    _check(lib().rsd_filter_rows(C.byref(r), B, R, V, int(top_k), float(top_p), _ptr(out["rows"]), _ptr(out["kept"]),
                                 _ptr(out["status"]), _stream()))
    return out


def rsd_gumbel_topk_draft(draft: torch.Tensor, k_per_row: Sequence[int], rng_node: Sequence[int], seed: int,
                          step: int, *, is_logprob: bool = False, seq_base: int = 0, max_k: Optional[int] = None,
                          want_values: bool = False, child_base: Optional[Sequence[int]] = None,
                          node_token: Optional[torch.Tensor] = None, out: Optional[dict] = None,
                          temperature: float = 1.0):
    """draft [B, R, V] -> dict(token [B, R, max_k], status [B], and perturbed/logprob when want_values).

    With child_base [R] and node_token [B, N+1] (int32) the picks also land in the tree's per-node token array.
    """
    B, R, V = draft.shape
    max_k = int(max_k or max(k_per_row))
    dev = draft.device
    if out is None:
        out = dict(token=_new((B, R, max_k), torch.int32, dev),
                   status=_new((B,), torch.int32, dev),
                   perturbed=_new((B, R, max_k), torch.float32, dev) if want_values else None,
                   logprob=_new((B, R, max_k), torch.float32, dev) if want_values else None)
    rows = rows_of(draft, is_logprob, temperature)
    if node_token is not None and (node_token.dtype != torch.int32 or not node_token.is_contiguous()):
        raise RsdError("node_token must be contiguous int32")
    _check(lib().rsd_gumbel_topk_draft(C.byref(rows), B, R, V, _host_i32(k_per_row), _host_i32(rng_node), max_k,
                                       seed, step, seq_base, _ptr(out["token"]), _ptr(out.get("perturbed")),
                                       _ptr(out.get("logprob")), None if child_base is None else _host_i32(child_base),
                                       _ptr(node_token), 0 if node_token is None else node_token.shape[1],
                                       _ptr(out["status"]), _stream()))
    return out


def rsd_profile_next_scan(before: Optional[torch.cuda.Event], after: Optional[torch.cuda.Event]):
    """Have the next drafting call record these (timing-enabled, already created) events around its scan kernel."""
    _check(lib().rsd_profile_next_scan(None if before is None else before.cuda_event,
                                       None if after is None else after.cuda_event))


def rsd_sbs_workspace_bytes(B: int, n_par: int, W: int) -> int:
    return int(lib().rsd_sbs_workspace_bytes(B, n_par, W))


def rsd_sbs_step(draft_level: torch.Tensor, W: int, first_parent_node: int, sum_logprob_in: Optional[torch.Tensor],
                 trunc_gumbel_in: Optional[torch.Tensor], seed: int, step: int, *, is_logprob: bool = False,
                 seq_base: int = 0, workspace: Optional[torch.Tensor] = None, out: Optional[dict] = None,
                 parent_base: int = 0, temperature: float = 1.0):
    """draft_level [B, n_par, V] -> dict(token, parent, sum_logprob, trunc_gumbel [B, W], count [B], status [B]).

    out["token"] / out["parent"] may be [B, W] views into wider [B, N+1] tree arrays (row stride kept); parent_base
    is added to every parent index.
    """
    B, n_par, V = draft_level.shape
    dev = draft_level.device
    need = rsd_sbs_workspace_bytes(B, n_par, W)
    if workspace is None:
        workspace = _new((need,), torch.uint8, dev)
    if out is None:
        out = dict(token=_new((B, W), torch.int32, dev),
                   parent=_new((B, W), torch.int32, dev),
                   sum_logprob=_new((B, W), torch.float32, dev),
                   trunc_gumbel=_new((B, W), torch.float32, dev),
                   count=_new((B,), torch.int32, dev),
                   status=_new((B,), torch.int32, dev))
    rows = rows_of(draft_level, is_logprob, temperature)
    if out["token"].stride(0) != out["parent"].stride(0) or out["token"].stride(1) != 1 or out["parent"].stride(1) != 1:
        raise RsdError("out token/parent must share a row stride and be dense along the picks")
    _check(lib().rsd_sbs_step(C.byref(rows), B, n_par, V, W, first_parent_node, _ptr(sum_logprob_in),
                              _ptr(trunc_gumbel_in), seed, step, seq_base, _ptr(out["token"]), _ptr(out["parent"]),
                              out["token"].stride(0), parent_base, _ptr(out["sum_logprob"]), _ptr(out["trunc_gumbel"]), _ptr(out["count"]),
                              _ptr(out["status"]), _ptr(workspace), workspace.numel(), _stream()))
    return out


def rsd_sbs_tree_workspace_bytes(B: int, W: int, L: int) -> int:
    return int(lib().rsd_sbs_tree_workspace_bytes(B, W, L))


def rsd_sbs_draft_tree(draft: torch.Tensor, W: int, L: int, seed: int, step: int, node_token: torch.Tensor,
                       node_parent: torch.Tensor, *, is_logprob: bool = False, seq_base: int = 0,
                       temperature: float = 1.0, workspace: Optional[torch.Tensor] = None, out: Optional[dict] = None):
    """draft [B, 1 + (L - 1) W, V]: every level of one Stochastic Beam Search tree in two launches.  Fills
    node_token / node_parent [B, >= 1 + L W] (the tree arrays rsd_verify_tree reads) and returns
    dict(sum_logprob, trunc_gumbel [B, W] of the last level, count [L, B], status [B])."""
    B, P, V = draft.shape
    dev = draft.device
    if P != 1 + (L - 1) * W:
        raise RsdError("draft must hold 1 + (L - 1) W = %d rows per sequence, got %d" % (1 + (L - 1) * W, P))
    if node_token.stride(0) != node_parent.stride(0) or node_token.stride(1) != 1 or node_parent.stride(1) != 1:
        raise RsdError("node_token / node_parent must share a row stride and be dense along the nodes")
    if workspace is None:
        workspace = _new((rsd_sbs_tree_workspace_bytes(B, W, L),), torch.uint8, dev)
    if out is None:
        out = dict(sum_logprob=_new((B, W), torch.float32, dev),
                   trunc_gumbel=_new((B, W), torch.float32, dev),
                   count=_new((L, B), torch.int32, dev),
                   status=_new((B,), torch.int32, dev))
    rows = rows_of(draft, is_logprob, temperature)
    _check(lib().rsd_sbs_draft_tree(C.byref(rows), B, V, W, L, seed, step, seq_base, _ptr(node_token),
                                    _ptr(node_parent), node_token.stride(0), _ptr(out["sum_logprob"]),
                                    _ptr(out["trunc_gumbel"]), _ptr(out["count"]), _ptr(out["status"]),
                                    _ptr(workspace), workspace.numel(), _stream()))
    return out


SBS_STATIC_SCRATCH_BYTES = 1 << 20


def rsd_sbs_step_static(draft_level: torch.Tensor, W: int, first_parent_node: int,
                        sum_logprob_in: Optional[torch.Tensor], trunc_gumbel_in: Optional[torch.Tensor], seed: int,
                        step: int, out: dict, *, is_logprob: bool = False, seq_base: int = 0, parent_base: int = 0,
                        temperature: float = 1.0):
    """rsd_sbs_step with the library's built-in scratch, for callers that may not allocate device memory.

    `out` must hold the caller's own tensors (token, parent, sum_logprob, trunc_gumbel [B, W]; count, status [B]):
    this wrapper allocates nothing either.  Raises RsdError when B * n_par * W is too large for the built-in
    scratch.  Calls that overlap on one GPU share that scratch and race.
    """
    B, n_par, V = draft_level.shape
    rows = rows_of(draft_level, is_logprob, temperature)
    if out["token"].stride(0) != out["parent"].stride(0) or out["token"].stride(1) != 1 or out["parent"].stride(1) != 1:
        raise RsdError("out token/parent must share a row stride and be dense along the picks")
    _check(lib().rsd_sbs_step_static(C.byref(rows), B, n_par, V, W, first_parent_node, _ptr(sum_logprob_in),
                                     _ptr(trunc_gumbel_in), seed, step, seq_base, _ptr(out["token"]),
                                     _ptr(out["parent"]), out["token"].stride(0), parent_base,
                                     _ptr(out["sum_logprob"]), _ptr(out["trunc_gumbel"]), _ptr(out["count"]),
                                     _ptr(out["status"]), _stream()))
    return out


def rsd_verify_tree(draft: torch.Tensor, target: torch.Tensor, parent: torch.Tensor, token: torch.Tensor,
                    num_levels: int, seed: int, step: int, *, seq_base: int = 0, want_theta: bool = False,
                    out: Optional[dict] = None, draft_temperature: float = 1.0, target_temperature: float = 1.0,
                    rule: int = 0, gamma: float = 1.0, final_sampler: int = 0, _force_rule_entry: bool = False):
    """draft [B, P, V], target [B, N+1, V], parent [N+1] or [B, N+1] int32, token [B, N+1] int32.
    rule = RULE_RRS with final_sampler = FINAL_INVERSE_CDF calls rsd_verify_tree; anything else calls
    rsd_verify_tree_rule."""
    B, _, V = target.shape
    dev = target.device
    n_nodes = token.shape[1]
    L = int(num_levels)
    if parent.dtype != torch.int32 or token.dtype != torch.int32:
        raise RsdError("parent and token must be int32")
    if not (parent.is_contiguous() and token.is_contiguous()):
        raise RsdError("parent and token must be contiguous")
    if out is None:
        out = dict(accepted_len=_new((B,), torch.int32, dev),
                   accepted_node=_new((B, max(L, 1)), torch.int32, dev)[:, :L],
                   accepted_token=_new((B, max(L, 1)), torch.int32, dev)[:, :L],
                   last_token=_new((B,), torch.int32, dev),
                   stop_reason=_new((B,), torch.int32, dev),
                   status=_new((B,), torch.int32, dev))
        out["theta"] = _new((B, n_nodes), torch.float32, dev) if want_theta else None
    tree = RsdTree(L, n_nodes, parent.data_ptr(), token.data_ptr(), 1 if parent.dim() == 1 else 0)
    d, t = rows_of(draft, False, draft_temperature), rows_of(target, False, target_temperature)
    outs = (_ptr(out["accepted_len"]), _ptr(out["accepted_node"]), _ptr(out["accepted_token"]),
            _ptr(out["last_token"]), _ptr(out["stop_reason"]), _ptr(out.get("theta")), _ptr(out["status"]), _stream())
    if rule == RULE_RRS and final_sampler == FINAL_INVERSE_CDF and not _force_rule_entry:
        _check(lib().rsd_verify_tree(C.byref(d), C.byref(t), C.byref(tree), B, V, seed, step, seq_base, *outs))
    else:
        _check(lib().rsd_verify_tree_rule(C.byref(d), C.byref(t), C.byref(tree), B, V, int(rule), float(gamma),
                                          int(final_sampler), seed, step, seq_base, *outs))
    return out


def rsd_verify_tree_rule(draft: torch.Tensor, target: torch.Tensor, parent: torch.Tensor, token: torch.Tensor,
                         num_levels: int, rule: int, gamma: float, final_sampler: int, seed: int, step: int, **kw):
    """rsd_verify_tree with a verification rule (RULE_RRS, RULE_MULTIROUND, RULE_KSEQ with its gamma) and a sampler
    of the last token (FINAL_INVERSE_CDF, FINAL_GUMBEL_TOP1)."""
    return rsd_verify_tree(draft, target, parent, token, num_levels, seed, step, rule=rule, gamma=gamma,
                           final_sampler=final_sampler, _force_rule_entry=True, **kw)


def rsd_resample_residual(draft_row: Optional[torch.Tensor], target_row: torch.Tensor,
                          rejected: Optional[torch.Tensor], rng_node: torch.Tensor, seed: int, step: int, *,
                          seq_base: int = 0, want_residual: bool = False, draft_temperature: float = 1.0,
                          target_temperature: float = 1.0):
    """draft_row/target_row [B, V]; rejected [B, max_k] int32 (-1 padded) or None; rng_node [B] int32."""
    B, V = target_row.shape
    dev = target_row.device
    token = _new((B,), torch.int32, dev)
    status = _new((B,), torch.int32, dev)
    residual = _new((B, V), torch.float32, dev) if want_residual else None
    t = rows_of(target_row, False, target_temperature)
    d = rows_of(draft_row, False, draft_temperature) if draft_row is not None else t
    max_k = 0 if rejected is None else rejected.shape[1]
    if rejected is not None and (rejected.dtype != torch.int32 or not rejected.is_contiguous()):
        raise RsdError("rejected must be contiguous int32")
    _check(lib().rsd_resample_residual(C.byref(d), C.byref(t), B, V, _ptr(rejected), max_k, _ptr(rng_node), seed,
                                       step, seq_base, _ptr(token), _ptr(residual), _ptr(status), _stream()))
    return dict(token=token, residual=residual, status=status)
