"""Thin ctypes binding of libstem (same names as the C ABI in ``include/stem.h``).

Argument marshalling only: every step of the path runs inside the CUDA kernels of the library.
PyTorch tensors are used as device buffers and for the current stream; nothing here computes.
There is no fallback: if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

from . import _build

STEM_OK = 0
STEM_ERR_INVALID_ARG = -1
STEM_ERR_UNSUPPORTED = -2
STEM_ERR_WORKSPACE = -3
STEM_ERR_CUDA = -4
STEM_ERR_DEVICE_TIMEOUT = -5
STEM_ERR_STATIC_SCRATCH = -6
STATIC_SCRATCH_BYTES = 8 * 1024 * 1024

EXPORTS = ("stem_version", "stem_status_string", "stem_plan_create", "stem_plan_create_ex", "stem_plan_destroy", "stem_plan_query",
           "stem_pool_kv", "stem_score_select_cached", "stem_prefill_cached",
           "stem_token_budget", "stem_token_select", "stem_token_attention", "stem_token_check_status",
           "stem_plan_budget", "stem_budget_table", "stem_score", "stem_score_static", "stem_select", "stem_score_select", "stem_sparse_prefill", "stem_prefill",
           "stem_check_status", "stem_selftest_wait_timeout", "stem_last_launch_count")


class StemConfig(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32),
        ("cu_seqlens_host", ctypes.POINTER(ctypes.c_int32)),
        ("num_q_heads", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("block", ctypes.c_int32),
        ("budget_permille", ctypes.c_int32),
        ("k_start_blocks", ctypes.c_int32),
        ("mu_num", ctypes.c_int32),
        ("mu_den", ctypes.c_int32),
        ("stem_blocks", ctypes.c_int32),
        ("local_blocks", ctypes.c_int32),
        ("min_blocks", ctypes.c_int32),
        ("beta", ctypes.c_float),
        ("score_scale", ctypes.c_float),
        ("softmax_scale", ctypes.c_float),
        ("q_stride_tok", ctypes.c_int64),
        ("q_stride_head", ctypes.c_int64),
        ("kv_stride_tok", ctypes.c_int64),
        ("kv_stride_head", ctypes.c_int64),
    ]


class StemPlanInfo(ctypes.Structure):
    _fields_ = [
        ("workspace_bytes", ctypes.c_size_t),
        ("total_tokens", ctypes.c_int32),
        ("total_q_blocks", ctypes.c_int32),
        ("k_max", ctypes.c_int32),
        ("metric_elems", ctypes.c_int64),
        ("selected_blocks", ctypes.c_int64),
        ("causal_blocks", ctypes.c_int64),
        ("selected_pairs", ctypes.c_int64),
        ("causal_pairs", ctypes.c_int64),
        ("total_kv_tokens", ctypes.c_int32),
        ("list_heads", ctypes.c_int32),
        ("kcache_bytes", ctypes.c_size_t),
        ("total_key_blocks", ctypes.c_int32),
        ("new_key_blocks", ctypes.c_int32),
    ]


class StemOptions(ctypes.Structure):
    _fields_ = [
        ("q_start_host", ctypes.POINTER(ctypes.c_int32)),
        ("total_len_host", ctypes.POINTER(ctypes.c_int32)),
        ("kcache_blocks_per_seq", ctypes.c_int32),
        ("share_group", ctypes.c_int32),
        ("score_mode", ctypes.c_int32),
        ("reserved", ctypes.c_int32 * 3),
    ]


class StemError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


_lib = None


def library_path() -> str:
    return _build.LIB


def load(build_if_missing: bool = True) -> ctypes.CDLL:
    """Load libstem.so (building it in-tree first if the sources are newer). Raises if impossible."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing and _build.needs_build():
        _build.build()
    if not os.path.exists(_build.LIB):
        raise RuntimeError(f"{_build.LIB} is missing: build it with `python -m paper_2603_06274_b200._build`")
    lib = ctypes.CDLL(_build.LIB)
    vp, i32p = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32)
    lib.stem_version.restype = ctypes.c_int
    lib.stem_status_string.restype = ctypes.c_char_p
    lib.stem_status_string.argtypes = [ctypes.c_int]
    lib.stem_plan_create.argtypes = [ctypes.POINTER(StemConfig), ctypes.POINTER(vp)]
    lib.stem_plan_create_ex.argtypes = [ctypes.POINTER(StemConfig), ctypes.POINTER(StemOptions), ctypes.POINTER(vp)]
    lib.stem_pool_kv.argtypes = [vp, vp, vp, vp, vp]
    lib.stem_score_select_cached.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.stem_prefill_cached.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_int, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.stem_token_budget.argtypes = [ctypes.c_int32] * 6 + [i32p]
    lib.stem_token_select.argtypes = [vp, ctypes.c_int32, ctypes.c_int32, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, vp, vp]
    lib.stem_token_attention.argtypes = [vp, vp, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int64, ctypes.c_int64,
                                         ctypes.c_int64, ctypes.c_int64, vp, vp, ctypes.c_int32, ctypes.c_float, vp, vp, vp]
    lib.stem_token_check_status.argtypes = [vp, i32p]
    lib.stem_plan_destroy.argtypes = [vp]
    lib.stem_plan_query.argtypes = [vp, ctypes.POINTER(StemPlanInfo)]
    lib.stem_plan_budget.argtypes = [vp, i32p]
    lib.stem_budget_table.argtypes = [ctypes.POINTER(StemConfig), i32p, ctypes.c_int64, i32p]
    lib.stem_score.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.stem_score_static.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.stem_select.argtypes = [vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.stem_score_select.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.stem_sparse_prefill.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.stem_prefill.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.stem_check_status.argtypes = [vp, vp, vp, i32p]
    lib.stem_selftest_wait_timeout.argtypes = [vp, vp, ctypes.c_size_t, vp]
    lib.stem_last_launch_count.argtypes = [vp]
    for name in EXPORTS:
        if name not in ("stem_status_string",):
            getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().stem_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != STEM_OK:
        raise StemError(status, where)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


class StemPlan:
    """Owns a ``stem_plan`` handle and (optionally) a workspace tensor for it."""

    def __init__(self, seqlens: Sequence[int], num_q_heads: int, num_kv_heads: int, block: int = 128,
                 budget_permille: int = 100, k_start_blocks: int = 0, mu=(7, 10), stem_blocks: int = 4,
                 local_blocks: int = 4, min_blocks: int = 0, beta: float = 0.2, score_scale: float = 0.0,
                 softmax_scale: float = 0.0, head_dim: int = 128, q_strides=None, kv_strides=None,
                 q_starts: Optional[Sequence[int]] = None, total_lens: Optional[Sequence[int]] = None,
                 kcache_blocks_per_seq: int = 0, share_group: bool = False, score_mode: int = 0):
        """``seqlens`` are the lengths of K and V.  With ``q_starts`` (chunked prefill) Q and O hold only the
        tokens q_start(b) .. seqlens[b]-1 of every sequence and ``total_lens`` are the full sequence lengths the
        budget schedule is evaluated on; ``kcache_blocks_per_seq`` > 0 puts the pooled K-side tensors into a
        caller-owned cache (``stem_pool_kv`` / ``*_cached``); ``share_group`` selects one list per kv head;
        ``score_mode`` = 1 the anti-diagonal scoring mode."""
        lib = load()
        cu = [0]
        for n in seqlens:
            cu.append(cu[-1] + int(n))
        self._cu = (ctypes.c_int32 * len(cu))(*cu)
        cfg = StemConfig()
        cfg.batch = len(seqlens)
        cfg.cu_seqlens_host = ctypes.cast(self._cu, ctypes.POINTER(ctypes.c_int32))
        cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.block = num_q_heads, num_kv_heads, head_dim, block
        cfg.budget_permille, cfg.k_start_blocks = budget_permille, k_start_blocks
        cfg.mu_num, cfg.mu_den = mu
        cfg.stem_blocks, cfg.local_blocks, cfg.min_blocks = stem_blocks, local_blocks, min_blocks
        cfg.beta, cfg.score_scale, cfg.softmax_scale = beta, score_scale, softmax_scale
        qs = q_strides or (num_q_heads * head_dim, head_dim)
        ks = kv_strides or (num_kv_heads * head_dim, head_dim)
        cfg.q_stride_tok, cfg.q_stride_head = qs
        cfg.kv_stride_tok, cfg.kv_stride_head = ks
        self.config = cfg
        self._h = ctypes.c_void_p()
        opts = StemOptions()
        if q_starts is not None:
            self._qs = (ctypes.c_int32 * len(seqlens))(*[int(x) for x in q_starts])
            opts.q_start_host = ctypes.cast(self._qs, ctypes.POINTER(ctypes.c_int32))
        if total_lens is not None:
            self._tl = (ctypes.c_int32 * len(seqlens))(*[int(x) for x in total_lens])
            opts.total_len_host = ctypes.cast(self._tl, ctypes.POINTER(ctypes.c_int32))
        opts.kcache_blocks_per_seq = int(kcache_blocks_per_seq)
        opts.share_group = 1 if share_group else 0
        opts.score_mode = int(score_mode)
        _check(lib.stem_plan_create_ex(ctypes.byref(cfg), ctypes.byref(opts), ctypes.byref(self._h)), "stem_plan_create_ex")
        info = StemPlanInfo()
        _check(lib.stem_plan_query(self._h, ctypes.byref(info)), "stem_plan_query")
        self.info = info
        self.num_q_heads, self.num_kv_heads, self.head_dim, self.block = num_q_heads, num_kv_heads, head_dim, block
        self._ws: Optional[torch.Tensor] = None

    @classmethod
    def from_workload(cls, w, **overrides) -> "StemPlan":
        kw = dict(seqlens=w.seqlens, num_q_heads=w.num_q_heads, num_kv_heads=w.num_kv_heads, block=w.block,
                  budget_permille=w.budget_permille, k_start_blocks=w.k_start_blocks, mu=(w.mu_num, w.mu_den),
                  stem_blocks=w.stem_blocks, local_blocks=w.local_blocks, min_blocks=w.min_blocks, beta=w.beta,
                  score_scale=w.score_scale)
        kw.update(overrides)
        return cls(**kw)

    @property
    def handle(self):
        return self._h

    def budget(self) -> torch.Tensor:
        out = torch.empty(self.info.total_q_blocks, dtype=torch.int32)
        _check(load().stem_plan_budget(self._h, ctypes.cast(out.data_ptr(), ctypes.POINTER(ctypes.c_int32))),
               "stem_plan_budget")
        return out

    def workspace(self, device="cuda") -> torch.Tensor:
        """A workspace tensor of the size the plan asks for (allocated once, outside the hot path)."""
        if self._ws is None:
            self._ws = torch.zeros(int(self.info.workspace_bytes) + 256, dtype=torch.uint8, device=device)
        return self._ws

    def last_launch_count(self) -> int:
        return int(load().stem_last_launch_count(self._h))

    def close(self) -> None:
        if self._h:
            load().stem_plan_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _ws_args(plan: StemPlan, workspace: Optional[torch.Tensor]):
    ws = plan.workspace() if workspace is None else workspace
    off = (-ws.data_ptr()) % 256
    return ws.data_ptr() + off, ws.numel() * ws.element_size() - off


def stem_score(plan: StemPlan, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, M: Optional[torch.Tensor] = None,
               workspace: Optional[torch.Tensor] = None) -> None:
    p, n = _ws_args(plan, workspace)
    _check(load().stem_score(plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(M), p, n, _stream()), "stem_score")


def stem_score_static(plan: StemPlan, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, M: torch.Tensor) -> None:
    """stem_score without a workspace: the pooled tensors go to a fixed array inside the library, so
    the call allocates nothing.  For callers that may not allocate device memory where they run
    (inside a framework's memory pool, in allocator-free callbacks).  Problems whose pooled
    tensors exceed STATIC_SCRATCH_BYTES raise StemError(STEM_ERR_STATIC_SCRATCH).  Calls share
    the array: do not overlap two of them on the GPU."""
    _check(load().stem_score_static(plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(M), _stream()), "stem_score_static")


def stem_select(plan: StemPlan, M: Optional[torch.Tensor], sel_idx: torch.Tensor, sel_cnt: torch.Tensor,
                workspace: Optional[torch.Tensor] = None) -> None:
    p, n = _ws_args(plan, workspace)
    _check(load().stem_select(plan.handle, _ptr(M), _ptr(sel_idx), _ptr(sel_cnt), p, n, _stream()), "stem_select")


def stem_score_select(plan: StemPlan, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, sel_idx: torch.Tensor,
                      sel_cnt: torch.Tensor, workspace: Optional[torch.Tensor] = None) -> None:
    p, n = _ws_args(plan, workspace)
    _check(load().stem_score_select(plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(sel_idx), _ptr(sel_cnt), p, n,
                                    _stream()), "stem_score_select")


def stem_pool_kv(plan: StemPlan, k: torch.Tensor, v: torch.Tensor, kcache: torch.Tensor) -> None:
    """K side of step 1 for the key blocks the plan's chunk adds, into the caller-owned pooled-K cache."""
    _check(load().stem_pool_kv(plan.handle, _ptr(k), _ptr(v), _ptr(kcache), _stream()), "stem_pool_kv")


def stem_score_select_cached(plan: StemPlan, q: torch.Tensor, kcache: torch.Tensor, sel_idx: torch.Tensor,
                             sel_cnt: torch.Tensor, workspace: Optional[torch.Tensor] = None) -> None:
    p, n = _ws_args(plan, workspace)
    _check(load().stem_score_select_cached(plan.handle, _ptr(q), _ptr(kcache), _ptr(sel_idx), _ptr(sel_cnt), p, n,
                                           _stream()), "stem_score_select_cached")


def stem_prefill_cached(plan: StemPlan, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor,
                        kcache: torch.Tensor, update_cache: bool = True, sel_idx: Optional[torch.Tensor] = None,
                        sel_cnt: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                        workspace: Optional[torch.Tensor] = None) -> None:
    p, n = _ws_args(plan, workspace)
    _check(load().stem_prefill_cached(plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(kcache),
                                      1 if update_cache else 0, _ptr(sel_idx), _ptr(sel_cnt), _ptr(lse), p, n, _stream()),
           "stem_prefill_cached")


def stem_token_budget(n_tokens: int, k_start: int, mu=(7, 10), stem_tokens: int = 0, local_tokens: int = 1) -> torch.Tensor:
    """Eq. 3 at token positions -> int32 [n_tokens] (host tensor)."""
    out = torch.empty(n_tokens, dtype=torch.int32)
    _check(load().stem_token_budget(n_tokens, k_start, mu[0], mu[1], stem_tokens, local_tokens,
                                    ctypes.cast(out.data_ptr(), ctypes.POINTER(ctypes.c_int32))), "stem_token_budget")
    return out


def stem_token_select(scores: torch.Tensor, k_tok: torch.Tensor, sel_idx: torch.Tensor, sel_cnt: torch.Tensor,
                      stem_tokens: int = 0, local_tokens: int = 1) -> None:
    """Token-level top-k(t) from indexer scores [list_heads, N, N]; lists [list_heads, N, k_max]."""
    h, n, _ = scores.shape
    _check(load().stem_token_select(_ptr(scores), n, h, _ptr(k_tok), stem_tokens, local_tokens, sel_idx.shape[2], _ptr(sel_idx),
                                    _ptr(sel_cnt), _stream()), "stem_token_select")


def stem_token_attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, sel_idx: torch.Tensor, sel_cnt: torch.Tensor,
                         out: torch.Tensor, lse: Optional[torch.Tensor] = None, softmax_scale: float = 0.0) -> None:
    """Gather-style attention over per-kv-head token lists; q [N, H_q, 128], k / v [N, H_kv, 128]."""
    n, hq, _ = q.shape
    hkv = k.shape[1]
    _check(load().stem_token_attention(_ptr(q), _ptr(k), _ptr(v), n, hq, hkv, q.stride(0), q.stride(1), k.stride(0), k.stride(1),
                                       _ptr(sel_idx), _ptr(sel_cnt), sel_idx.shape[2], softmax_scale, _ptr(out), _ptr(lse), _stream()),
           "stem_token_attention")


def stem_token_check_status():
    """Synchronise the current stream and return (status, detail[4]) of the gather-attention kernel."""
    detail = (ctypes.c_int32 * 4)()
    st = load().stem_token_check_status(_stream(), ctypes.cast(detail, ctypes.POINTER(ctypes.c_int32)))
    return int(st), [int(x) for x in detail]


def stem_sparse_prefill(plan: StemPlan, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                        sel_idx: Optional[torch.Tensor], sel_cnt: Optional[torch.Tensor], out: torch.Tensor,
                        lse: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None) -> None:
    p, n = _ws_args(plan, workspace)
    _check(load().stem_sparse_prefill(plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(sel_idx), _ptr(sel_cnt), _ptr(out),
                                      _ptr(lse), p, n, _stream()), "stem_sparse_prefill")


def stem_prefill(plan: StemPlan, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor,
                 sel_idx: Optional[torch.Tensor] = None, sel_cnt: Optional[torch.Tensor] = None,
                 lse: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None) -> None:
    p, n = _ws_args(plan, workspace)
    _check(load().stem_prefill(plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(sel_idx), _ptr(sel_cnt),
                               _ptr(lse), p, n, _stream()), "stem_prefill")


def stem_check_status(plan: StemPlan, workspace: Optional[torch.Tensor] = None, static_scratch: bool = False):
    """Synchronise the current stream and return (status, detail[4]).  With ``static_scratch`` the status
    words of the scratch built into the library (stem_score_static) are read instead of a workspace's."""
    p = None if static_scratch else _ws_args(plan, workspace)[0]
    detail = (ctypes.c_int32 * 4)()
    st = load().stem_check_status(plan.handle, p, _stream(), ctypes.cast(detail, ctypes.POINTER(ctypes.c_int32)))
    return int(st), [int(x) for x in detail]


def status_words(plan: StemPlan, workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The eight int32 status words at the start of the (aligned) workspace, as a view."""
    ws = plan.workspace() if workspace is None else workspace
    off = (-ws.data_ptr()) % 256
    return ws[off:off + 32].view(torch.int32)


def stem_selftest_wait_timeout(plan: StemPlan, workspace: Optional[torch.Tensor] = None) -> None:
    """Enqueue the library's time-out self-test: a 1 ms bounded wait that runs out and records it."""
    p, n = _ws_args(plan, workspace)
    _check(load().stem_selftest_wait_timeout(plan.handle, p, n, _stream()), "stem_selftest_wait_timeout")
