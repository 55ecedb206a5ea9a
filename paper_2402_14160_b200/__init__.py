"""B200-native hot path of Recursive Speculative Decoding: Gumbel-Top-k / Stochastic Beam Search drafting and
recursive rejection sampling over the draft tree, as CUDA kernels (sm_100a) behind a C ABI (include/rsd.h).

The functions below are argument-marshalling wrappers with the names of the C entry points.
"""
from . import api  # noqa: F401
from .api import (LIB_PATH, MAX_K, RsdError, lib, rows_of, rsd_filter_rows, rsd_gumbel_topk_draft, rsd_profile_next_scan, rsd_resample_residual,  # noqa: F401
                  rsd_sbs_step, rsd_sbs_step_static, rsd_sbs_workspace_bytes, rsd_sbs_draft_tree,
                  rsd_sbs_tree_workspace_bytes, rsd_verify_tree, rsd_verify_tree_rule)
from .api import (ST_DRAFT_EXHAUSTED, ST_FEWER_THAN_K, ST_NAN_INPUT, ST_ZERO_DRAFT_PROB, ST_ZERO_RESIDUAL, ST_TIMEOUT,  # noqa: F401
                  STOP_ALL_REJECTED, STOP_LEAF, STOP_NO_CHILDREN, RULE_RRS, RULE_MULTIROUND, RULE_KSEQ, FINAL_INVERSE_CDF, FINAL_GUMBEL_TOP1)
