"""CPU oracle for the RSD hot path (test infrastructure, never a product path).

A ctypes front end to ``rsd_oracle.c``: plain double-precision restatements of
Gumbel-Top-k drafting (Algorithm 4), the Stochastic Beam Search step
(Algorithm 9), recursive rejection sampling (Algorithm 1, Eqs. 1-4) and the
tree verification walk (Algorithm 6).  Only tests, the smoke check and the
CPU-baseline leg of the benchmark may import this package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rsd_oracle.c")
_LIB = os.path.join(_HERE, "librsd_oracle.so")

F32, BF16 = 0, 1
ST_NAN_INPUT, ST_FEWER_THAN_K, ST_ZERO_RESIDUAL, ST_ZERO_DRAFT_PROB, ST_DRAFT_EXHAUSTED = 1, 2, 4, 8, 16
STOP_ALL_REJECTED, STOP_NO_CHILDREN, STOP_LEAF = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over independent rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.rsd_oracle_gumbel.restype = C.c_double
        _lib.rsd_oracle_gumbel.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32]
        _lib.rsd_oracle_gumbel_parts.restype = None
        _lib.rsd_oracle_gumbel_parts.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32,
                                                 C.POINTER(C.c_double), C.POINTER(C.c_int32), C.POINTER(C.c_double)]
        _lib.rsd_oracle_accept_uniform.restype = C.c_double
        _lib.rsd_oracle_accept_uniform.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32]
        _lib.rsd_oracle_resample_uniform.restype = C.c_double
        _lib.rsd_oracle_resample_uniform.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32]
        _lib.rsd_oracle_truncated_gumbel.restype = C.c_double
        _lib.rsd_oracle_truncated_gumbel.argtypes = [C.c_double, C.c_double, C.c_double]
        _lib.rsd_oracle_inverse_cdf.restype = C.c_int
        _lib.rsd_oracle_rng_layout.restype = C.c_int
    return _lib


def num_threads() -> int:
    """Threads the OpenMP loops use (OMP_NUM_THREADS or the visible cores)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def set_num_threads(n: int) -> None:
    """Threads of the OpenMP loops from now on (the benchmark's single-thread figure)."""
    lib()
    C.CDLL("libgomp.so.1").omp_set_num_threads(int(n))


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _rows(a: np.ndarray):
    """(array, dtype code): float32 arrays are fp32 rows, uint16 arrays are bf16 bit patterns."""
    if a.dtype == np.float32:
        return a, F32
    if a.dtype == np.uint16:
        return a, BF16
    raise TypeError("rows must be float32 or uint16 (bf16 bits), got %s" % a.dtype)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


# ---------------------------------------------------------------------------
def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().rsd_oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def gumbel(seed, step, seq, node, e):
    return lib().rsd_oracle_gumbel(seed, step, seq, node, e)


def gumbel_parts(seed, step, seq, node, e):
    """(t of the group's uniform, position of the group's largest noise, t of the element's uniform)."""
    tg, a, te = C.c_double(), C.c_int32(), C.c_double()
    lib().rsd_oracle_gumbel_parts(seed, step, seq, node, e, C.byref(tg), C.byref(a), C.byref(te))
    return tg.value, a.value, te.value


def accept_uniform(seed, step, seq, node, j):
    return lib().rsd_oracle_accept_uniform(seed, step, seq, node, j)


def resample_uniform(seed, step, seq, node):
    return lib().rsd_oracle_resample_uniform(seed, step, seq, node)


def truncated_gumbel(u, phi, z):
    return lib().rsd_oracle_truncated_gumbel(u, phi, z)


def inverse_cdf(w, u):
    w = np.ascontiguousarray(w, dtype=np.float64)
    m = C.c_double(0.0)
    y = lib().rsd_oracle_inverse_cdf(_ptr(w), C.c_int(w.shape[0]), C.c_double(u), C.byref(m))
    return y, m.value


def rrs_chain(p, q, tokens):
    """theta[k] and the final residual q^(K+1) for an ordered draft tuple (Eqs. 2-3)."""
    p = np.ascontiguousarray(p, dtype=np.float64)
    q = np.ascontiguousarray(q, dtype=np.float64)
    t = _i32(tokens)
    theta = np.zeros(len(t), dtype=np.float64)
    res = np.zeros(p.shape[0], dtype=np.float64)
    st = lib().rsd_oracle_rrs_chain(_ptr(p), _ptr(q), C.c_int(p.shape[0]), _ptr(t), C.c_int(len(t)),
                                    _ptr(theta), _ptr(res))
    return theta, res, st


def baseline_chain(rule, p, q, tokens, gamma=1.0):
    """theta[k] and the all-rejected residual of a baseline verifier (RULE_MULTIROUND or RULE_KSEQ) for an
    ordered tuple of independent drafts (Section 2)."""
    p = np.ascontiguousarray(p, dtype=np.float64)
    q = np.ascontiguousarray(q, dtype=np.float64)
    t = _i32(tokens)
    theta = np.zeros(len(t), dtype=np.float64)
    res = np.zeros(p.shape[0], dtype=np.float64)
    st = lib().rsd_oracle_baseline_chain(C.c_int(int(rule)), C.c_double(float(gamma)), _ptr(p), _ptr(q),
                                         C.c_int(p.shape[0]), _ptr(t), C.c_int(len(t)), _ptr(theta), _ptr(res))
    return theta, res, st


def gumbel_topk(rows, k_per_row, rng_node, seed, step, *, is_logprob=False, seq_base=0, max_k=None,
                temperature=1.0):
    """rows [B,R,V]; returns dict(token[B,R,max_k], perturbed, logprob, margin[B,R], status[B])."""
    a, dt = _rows(rows)
    B, R, V = a.shape
    assert a.strides[2] == a.itemsize
    k = _i32(k_per_row)
    nodes = _i32(rng_node)
    max_k = int(max_k or k.max())
    tok = np.zeros((B, R, max_k), np.int32)
    pert = np.zeros((B, R, max_k), np.float64)
    logp = np.zeros((B, R, max_k), np.float64)
    margin = np.zeros((B, R), np.float64)
    status = np.zeros(B, np.int32)
    lib().rsd_oracle_gumbel_topk(_ptr(a), C.c_int(dt), C.c_int(int(is_logprob)), C.c_double(temperature),
                                 C.c_int64(a.strides[0] // a.itemsize), C.c_int64(a.strides[1] // a.itemsize),
                                 C.c_int(B), C.c_int(R), C.c_int(V), _ptr(k), _ptr(nodes), C.c_int(max_k),
                                 C.c_uint64(seed), C.c_uint32(step), C.c_uint32(seq_base),
                                 _ptr(tok), _ptr(pert), _ptr(logp), _ptr(margin), _ptr(status))
    return dict(token=tok, perturbed=pert, logprob=logp, margin=margin, status=status)


def sbs_step(rows, W, first_parent_node, sum_logprob_in, trunc_gumbel_in, seed, step, *, is_logprob=False,
             seq_base=0, temperature=1.0):
    """rows [B,n_par,V]; one Stochastic Beam Search level."""
    a, dt = _rows(rows)
    B, n_par, V = a.shape
    assert a.strides[2] == a.itemsize
    sig = None if sum_logprob_in is None else np.ascontiguousarray(sum_logprob_in, dtype=np.float64)
    gam = None if trunc_gumbel_in is None else np.ascontiguousarray(trunc_gumbel_in, dtype=np.float64)
    tok = np.zeros((B, W), np.int32)
    par = np.zeros((B, W), np.int32)
    so = np.zeros((B, W), np.float64)
    go = np.zeros((B, W), np.float64)
    cnt = np.zeros(B, np.int32)
    margin = np.zeros(B, np.float64)
    status = np.zeros(B, np.int32)
    lib().rsd_oracle_sbs_step(_ptr(a), C.c_int(dt), C.c_int(int(is_logprob)), C.c_double(temperature),
                              C.c_int64(a.strides[0] // a.itemsize), C.c_int64(a.strides[1] // a.itemsize),
                              C.c_int(B), C.c_int(n_par), C.c_int(V), C.c_int(W), C.c_int32(first_parent_node),
                              _ptr(sig), _ptr(gam), C.c_uint64(seed), C.c_uint32(step), C.c_uint32(seq_base),
                              _ptr(tok), _ptr(par), _ptr(so), _ptr(go), _ptr(cnt), _ptr(margin), _ptr(status))
    return dict(token=tok, parent=par, sum_logprob=so, trunc_gumbel=go, count=cnt, margin=margin, status=status)


RULE_RRS, RULE_MULTIROUND, RULE_KSEQ = 0, 1, 2


def verify_tree(draft, target, parent, token, num_levels, seed, step, *, seq_base=0, want_weights=False,
                draft_temperature=1.0, target_temperature=1.0, rule=RULE_RRS, gamma=1.0, final_sampler=0):
    """draft [B,P,V], target [B,N+1,V], parent [N+1] or [B,N+1] (flat, root -1), token [B,N+1].
    rule: recursive rejection sampling (the paper's), or one of the two baselines of Section 2 on the same tree:
    multi-round rejection sampling with one draft model, K-SEQ with parameter gamma.
    final_sampler: 0 = inverse CDF with one uniform, 1 = Gumbel-Top-1 (Algorithm 6's last step)."""
    d, ddt = _rows(draft)
    t, tdt = _rows(target)
    B, _, V = t.shape
    par = _i32(parent)
    tok = _i32(token)
    n_nodes = tok.shape[1]
    shared = 1 if par.ndim == 1 else 0
    L = int(num_levels)
    alen = np.zeros(B, np.int32)
    anode = np.zeros((B, L), np.int32)
    atok = np.zeros((B, L), np.int32)
    last = np.zeros(B, np.int32)
    reason = np.zeros(B, np.int32)
    theta = np.zeros((B, n_nodes), np.float64)
    margin = np.zeros((B, n_nodes), np.float64)
    fmargin = np.zeros(B, np.float64)
    weights = np.zeros((B, V), np.float64) if want_weights else None
    status = np.zeros(B, np.int32)
    lib().rsd_oracle_verify_tree_rule(C.c_int(int(rule)), C.c_double(float(gamma)), C.c_int(int(final_sampler)),
                                 _ptr(d), C.c_int(ddt), C.c_int64(d.strides[0] // d.itemsize),
                                 C.c_int64(d.strides[1] // d.itemsize), C.c_double(draft_temperature),
                                 _ptr(t), C.c_int(tdt), C.c_int64(t.strides[0] // t.itemsize),
                                 C.c_int64(t.strides[1] // t.itemsize), C.c_double(target_temperature),
                                 C.c_int(B), C.c_int(V), C.c_int(n_nodes), C.c_int(L),
                                 _ptr(par), C.c_int(shared), _ptr(tok),
                                 C.c_uint64(seed), C.c_uint32(step), C.c_uint32(seq_base),
                                 _ptr(alen), _ptr(anode), _ptr(atok), _ptr(last), _ptr(reason),
                                 _ptr(theta), _ptr(margin), _ptr(fmargin), _ptr(weights), _ptr(status))
    return dict(accepted_len=alen, accepted_node=anode, accepted_token=atok, last_token=last, stop_reason=reason,
                theta=theta, margin=margin, final_margin=fmargin, final_weights=weights, status=status)


def resample_residual(draft, target, rejected, rng_node, seed, step, *, seq_base=0, draft_temperature=1.0,
                      target_temperature=1.0):
    """draft/target [B,V] (draft may be None when nothing was rejected); rejected [B,max_k] (-1 padded)."""
    t, tdt = _rows(target)
    B, V = t.shape
    if draft is not None:
        d, ddt = _rows(draft)
        dstride = d.strides[0] // d.itemsize
    else:
        d, ddt, dstride = None, F32, 0
    rej = _i32(rejected) if rejected is not None else np.full((B, 1), -1, np.int32)
    nodes = _i32(rng_node)
    out = np.zeros(B, np.int32)
    res = np.zeros((B, V), np.float64)
    margin = np.zeros(B, np.float64)
    status = np.zeros(B, np.int32)
    lib().rsd_oracle_resample_residual(_ptr(d), C.c_int(ddt), C.c_int64(dstride), C.c_double(draft_temperature),
                                       _ptr(t), C.c_int(tdt), C.c_int64(t.strides[0] // t.itemsize),
                                       C.c_double(target_temperature),
                                       C.c_int(B), C.c_int(V), _ptr(rej), C.c_int(rej.shape[1]), _ptr(nodes),
                                       C.c_uint64(seed), C.c_uint32(step), C.c_uint32(seq_base),
                                       _ptr(out), _ptr(res), _ptr(margin), _ptr(status))
    return dict(token=out, residual=res, margin=margin, status=status)


def filter_rows(rows, top_k=0, top_p=1.0, *, temperature=1.0):
    """rows [B,R,V] -> dict(keep [B,R,V] bool, kept [B,R], margin [B,R]): top-k then nucleus filtering of every row
    (after the temperature); a filtered token counts as -inf from then on."""
    a, dt = _rows(rows)
    B, R, V = a.shape
    assert a.strides[2] == a.itemsize
    keep = np.zeros((B, R, V), np.uint8)
    kept = np.zeros((B, R), np.int32)
    margin = np.zeros((B, R), np.float64)
    lib().rsd_oracle_filter_rows(_ptr(a), C.c_int(dt), C.c_double(temperature), C.c_int64(a.strides[0] // a.itemsize),
                                 C.c_int64(a.strides[1] // a.itemsize), C.c_int(B), C.c_int(R), C.c_int(V),
                                 C.c_int(int(top_k)), C.c_double(float(top_p)), _ptr(keep), _ptr(kept), _ptr(margin))
    return dict(keep=keep.astype(bool), kept=kept, margin=margin)


def apply_filter(rows, keep):
    """The rows with -inf at every filtered entry (same storage type: float32, or bf16 bit patterns)."""
    out = np.array(rows, copy=True)
    if out.dtype == np.uint16:
        out[~keep] = 0xFF80
    else:
        out[~keep] = -np.inf
    return out
