"""Stem sparse causal prefill attention for NVIDIA B200 (sm_100a).

The product is the C-ABI library ``libstem.so`` (see ``include/stem.h``); this package holds its
CUDA sources, the in-tree build, a thin ctypes binding with the same entry-point names, and the
seeded synthetic workloads used by the tests and the benchmark.
"""
from . import workloads  # noqa: F401
from .binding import (  # noqa: F401
    StemConfig, StemError, StemOptions, StemPlan, StemPlanInfo, load, library_path, status_string,
    stem_check_status, stem_pool_kv, stem_prefill, stem_prefill_cached, stem_score, stem_score_select,
    stem_score_select_cached, stem_score_static, stem_select, stem_sparse_prefill, stem_token_attention,
    stem_token_budget, stem_token_check_status, stem_token_select,
)
