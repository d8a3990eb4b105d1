"""ctypes front end of the CPU checker (``stem_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the CPU
baseline leg of the benchmark.  The product never imports this module, and this
module imports nothing from the product.

Each function follows one step of Algorithm 1 of the paper; see the C file for
the per-step statements and citations.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "stem_oracle.c")
_LIB = os.path.join(_HERE, "libstem_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the checker with gcc (OpenMP) next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-shared", "-fPIC", "-std=c11", _SRC, "-o", _LIB, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.so_num_threads.restype = ctypes.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(_load().so_num_threads())


@dataclass
class StemParams:
    """Hyper-parameters of Algorithm 1 plus the forced-block settings of the implementation details."""

    block: int
    budget_permille: int = 100
    k_start_blocks: int = 0
    mu_num: int = 7
    mu_den: int = 10
    stem_blocks: int = 4
    local_blocks: int = 4
    min_blocks: int = 0
    beta: float = 0.2
    score_scale: float = 1.0
    softmax_scale: float = 0.0  # 0 -> 1/sqrt(d)


def n_blocks(seqlens: Sequence[int], block: int) -> np.ndarray:
    return np.array([(int(n) + block - 1) // block for n in seqlens], dtype=np.int32)


def k_start(n_blk: int, p: StemParams) -> int:
    """Initial budget in blocks: an explicit count, else floor(permille * N_blk / 1000)."""
    return int(p.k_start_blocks) if p.k_start_blocks > 0 else (int(p.budget_permille) * int(n_blk)) // 1000


def schedule(n_blk: int, k_s: int, p: StemParams):
    """Eq. 3 in block units -> (k_blk, k_eff), each int32 [n_blk]."""
    kb = np.empty(n_blk, dtype=np.int32)
    ke = np.empty(n_blk, dtype=np.int32)
    _load().so_schedule(ctypes.c_int32(n_blk), ctypes.c_int64(k_s), ctypes.c_int64(p.mu_num), ctypes.c_int64(p.mu_den),
                        ctypes.c_int32(p.stem_blocks), ctypes.c_int32(p.local_blocks), ctypes.c_int32(p.min_blocks),
                        _p(kb), _p(ke))
    return kb, ke


def schedule_batch(seqlens: Sequence[int], p: StemParams) -> np.ndarray:
    """k_eff for every global row, sequence-major."""
    out = []
    for nb in n_blocks(seqlens, p.block):
        out.append(schedule(int(nb), k_start(int(nb), p), p)[1])
    return np.concatenate(out) if out else np.zeros(0, np.int32)


def _strides(x: np.ndarray):
    assert x.dtype == np.uint16 and x.ndim == 3 and x.strides[2] == 2
    return x.strides[0] // 2, x.strides[1] // 2


def pool_mean(x_bits: np.ndarray, cu_seqlens: np.ndarray, block: int) -> np.ndarray:
    """Alg. 1 'Pool': block means of Q or K -> fp32 [H, R_tot, d]."""
    T, H, d = x_bits.shape
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    r_tot = int(n_blocks(np.diff(cu), block).sum())
    out = np.empty((H, r_tot, d), dtype=np.float32)
    st, sh = _strides(x_bits)
    _load().so_pool_mean(_p(x_bits), ctypes.c_int64(st), ctypes.c_int64(sh), ctypes.c_int32(H), ctypes.c_int32(d),
                         ctypes.c_int32(len(cu) - 1), _p(cu), ctypes.c_int32(block), _p(out))
    return out


def value_magnitude(v_bits: np.ndarray, cu_seqlens: np.ndarray, block: int) -> np.ndarray:
    """Alg. 1 'MaxPool(log||V||)' with the max(0, .) of Eq. 7 -> fp32 [H_kv, R_tot]."""
    T, H, d = v_bits.shape
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    r_tot = int(n_blocks(np.diff(cu), block).sum())
    out = np.empty((H, r_tot), dtype=np.float32)
    st, sh = _strides(v_bits)
    _load().so_value_magnitude(_p(v_bits), ctypes.c_int64(st), ctypes.c_int64(sh), ctypes.c_int32(H), ctypes.c_int32(d),
                               ctypes.c_int32(len(cu) - 1), _p(cu), ctypes.c_int32(block), _p(out))
    return out


def metric(qbar: np.ndarray, kbar: np.ndarray, mv: np.ndarray, nblk: np.ndarray, beta: float,
           score_scale: float = 1.0) -> np.ndarray:
    """Eq. 7 on pooled blocks -> fp32 [H_q, sum_b N_blk_b^2] (entries j <= r defined, rest NaN)."""
    hq, r_tot, d = qbar.shape
    hkv = kbar.shape[0]
    nblk = np.ascontiguousarray(nblk, dtype=np.int32)
    m_tot = int((nblk.astype(np.int64) ** 2).sum())
    M = np.full((hq, m_tot), np.nan, dtype=np.float32)
    _load().so_metric(_p(np.ascontiguousarray(qbar)), _p(np.ascontiguousarray(kbar)), _p(np.ascontiguousarray(mv)),
                      ctypes.c_int32(hq), ctypes.c_int32(hkv), ctypes.c_int32(d), ctypes.c_int32(len(nblk)), _p(nblk),
                      ctypes.c_float(beta), ctypes.c_float(score_scale), _p(M))
    return M


def select(M: np.ndarray, nblk: np.ndarray, k_eff: np.ndarray, stem: int, local: int, k_max: Optional[int] = None):
    """Alg. 1 'TopK' with forced stem/local blocks -> (sel_idx [H_q,R_tot,k_max], sel_cnt [H_q,R_tot])."""
    hq = M.shape[0]
    nblk = np.ascontiguousarray(nblk, dtype=np.int32)
    k_eff = np.ascontiguousarray(k_eff, dtype=np.int32)
    r_tot = int(nblk.sum())
    if k_max is None:
        k_max = int(k_eff.max())
    idx = np.empty((hq, r_tot, k_max), dtype=np.int32)
    cnt = np.empty((hq, r_tot), dtype=np.int32)
    _load().so_select(_p(np.ascontiguousarray(M, dtype=np.float32)), ctypes.c_int32(hq), ctypes.c_int32(len(nblk)),
                      _p(nblk), _p(k_eff), ctypes.c_int32(stem), ctypes.c_int32(local), ctypes.c_int32(k_max),
                      _p(idx), _p(cnt))
    return idx, cnt


def attention(q_bits: np.ndarray, k_bits: np.ndarray, v_bits: np.ndarray, cu_seqlens: np.ndarray, block: int,
              sel_idx: np.ndarray, sel_cnt: np.ndarray, softmax_scale: float = 0.0,
              rows: Optional[np.ndarray] = None, want_lse: bool = True):
    """Alg. 1 step d for the (head, global row) pairs in ``rows`` (all rows when None).

    Returns (O fp32 [T,H_q,d], lse fp32 [H_q,T]); entries of rows not requested are NaN.
    """
    T, hq, d = q_bits.shape
    hkv = k_bits.shape[1]
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    if softmax_scale == 0.0:
        softmax_scale = 1.0 / np.sqrt(d)
    r_tot = sel_cnt.shape[1]
    if rows is None:
        hh, rr = np.meshgrid(np.arange(hq, dtype=np.int32), np.arange(r_tot, dtype=np.int32), indexing="ij")
        rows = np.stack([hh.ravel(), rr.ravel()], axis=1)
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    O = np.full((T, hq, d), np.nan, dtype=np.float32)
    lse = np.full((hq, T), np.nan, dtype=np.float32) if want_lse else None
    qs, qh = _strides(q_bits)
    ks, kh = _strides(k_bits)
    assert _strides(v_bits) == (ks, kh)
    sel_idx = np.ascontiguousarray(sel_idx, dtype=np.int32)
    sel_cnt = np.ascontiguousarray(sel_cnt, dtype=np.int32)
    _load().so_attention(_p(q_bits), ctypes.c_int64(qs), ctypes.c_int64(qh), _p(k_bits), _p(v_bits),
                         ctypes.c_int64(ks), ctypes.c_int64(kh), ctypes.c_int32(hq), ctypes.c_int32(hkv),
                         ctypes.c_int32(d), ctypes.c_int32(len(cu) - 1), _p(cu), ctypes.c_int32(block), _p(sel_idx),
                         _p(sel_cnt), ctypes.c_int32(sel_idx.shape[2]), ctypes.c_float(softmax_scale), _p(rows),
                         ctypes.c_int64(len(rows)), _p(O), _p(lse))
    return O, lse


def score(q_bits, k_bits, v_bits, cu_seqlens, p: StemParams):
    """Steps 1 and 3a: pooled tensors and the metric. Returns (M, qbar, kbar, mv)."""
    qbar = pool_mean(q_bits, cu_seqlens, p.block)
    kbar = pool_mean(k_bits, cu_seqlens, p.block)
    mv = value_magnitude(v_bits, cu_seqlens, p.block)
    nblk = n_blocks(np.diff(cu_seqlens), p.block)
    return metric(qbar, kbar, mv, nblk, p.beta, p.score_scale), qbar, kbar, mv


def prefill(q_bits, k_bits, v_bits, cu_seqlens, p: StemParams, rows: Optional[np.ndarray] = None):
    """All of Algorithm 1. Returns dict with M, sel_idx, sel_cnt, k_eff, O, lse."""
    M, qbar, kbar, mv = score(q_bits, k_bits, v_bits, cu_seqlens, p)
    seqlens = np.diff(cu_seqlens)
    nblk = n_blocks(seqlens, p.block)
    k_eff = schedule_batch(seqlens, p)
    idx, cnt = select(M, nblk, k_eff, p.stem_blocks, p.local_blocks)
    O, lse = attention(q_bits, k_bits, v_bits, cu_seqlens, p.block, idx, cnt, p.softmax_scale, rows)
    return {"M": M, "qbar": qbar, "kbar": kbar, "mv": mv, "k_eff": k_eff, "sel_idx": idx, "sel_cnt": cnt,
            "O": O, "lse": lse}


def dense_lists(seqlens: Sequence[int], block: int, hq: int):
    """Index lists naming every causal block (the full-budget case)."""
    nblk = n_blocks(seqlens, block)
    r_tot, k_max = int(nblk.sum()), int(nblk.max())
    idx = np.full((hq, r_tot, k_max), -1, dtype=np.int32)
    cnt = np.empty((hq, r_tot), dtype=np.int32)
    off = 0
    for nb in nblk:
        for r in range(int(nb)):
            idx[:, off + r, : r + 1] = np.arange(r + 1, dtype=np.int32)
            cnt[:, off + r] = r + 1
        off += int(nb)
    return idx, cnt


# ----------------------------------------------------------------------------------------------
# Chunked prefill with global token offsets (Conclusion, "Limitations and future work")
# ----------------------------------------------------------------------------------------------

def chunk_geometry(kv_lens: Sequence[int], q_starts: Sequence[int], block: int):
    """(n_kv_blk, r0) per sequence: blocks of the K/V prefix, first global block row of the chunk."""
    nkb = n_blocks(kv_lens, block)
    r0 = np.array([int(s) // block for s in q_starts], dtype=np.int32)
    for s, n in zip(q_starts, kv_lens):
        assert int(s) % block == 0 and 0 <= int(s) < int(n), "a chunk starts on a block boundary inside the prefix"
    return nkb, r0


def schedule_chunk(kv_lens: Sequence[int], q_starts: Sequence[int], total_lens: Sequence[int], p: StemParams) -> np.ndarray:
    """k_eff of the chunk's rows: Eq. 3 evaluated at the GLOBAL row of a sequence of ceil(total_len / B)
    blocks (k_start from that block count too), sliced to the rows r0 .. n_kv_blk - 1."""
    nkb, r0 = chunk_geometry(kv_lens, q_starts, p.block)
    out = []
    for b, n_tot in enumerate(n_blocks(total_lens, p.block)):
        assert int(n_tot) >= int(nkb[b])
        ke = schedule(int(n_tot), k_start(int(n_tot), p), p)[1]
        out.append(ke[int(r0[b]):int(nkb[b])])
    return np.concatenate(out).astype(np.int32)


def metric_chunk(qbar: np.ndarray, kbar: np.ndarray, mv: np.ndarray, nkb: np.ndarray, r0: np.ndarray, beta: float,
                 score_scale: float = 1.0) -> np.ndarray:
    hq, hkv, d = qbar.shape[0], kbar.shape[0], qbar.shape[2]
    nkb = np.ascontiguousarray(nkb, dtype=np.int32)
    r0 = np.ascontiguousarray(r0, dtype=np.int32)
    m_tot = int(((nkb - r0).astype(np.int64) * nkb).sum())
    M = np.full((hq, m_tot), np.nan, dtype=np.float32)
    _load().so_metric_chunk(_p(np.ascontiguousarray(qbar)), _p(np.ascontiguousarray(kbar)), _p(np.ascontiguousarray(mv)),
                            ctypes.c_int32(hq), ctypes.c_int32(hkv), ctypes.c_int32(d), ctypes.c_int32(len(nkb)),
                            _p(nkb), _p(r0), ctypes.c_float(beta), ctypes.c_float(score_scale), _p(M))
    return M


def select_chunk(M: np.ndarray, nkb: np.ndarray, r0: np.ndarray, k_eff: np.ndarray, stem: int, local: int,
                 k_max: Optional[int] = None):
    hq = M.shape[0]
    nkb = np.ascontiguousarray(nkb, dtype=np.int32)
    r0 = np.ascontiguousarray(r0, dtype=np.int32)
    k_eff = np.ascontiguousarray(k_eff, dtype=np.int32)
    rq_tot = int((nkb - r0).sum())
    if k_max is None:
        k_max = int(k_eff.max())
    idx = np.empty((hq, rq_tot, k_max), dtype=np.int32)
    cnt = np.empty((hq, rq_tot), dtype=np.int32)
    _load().so_select_chunk(_p(np.ascontiguousarray(M, dtype=np.float32)), ctypes.c_int32(hq), ctypes.c_int32(len(nkb)),
                            _p(nkb), _p(r0), _p(k_eff), ctypes.c_int32(stem), ctypes.c_int32(local), ctypes.c_int32(k_max),
                            _p(idx), _p(cnt))
    return idx, cnt


def attention_chunk(q_bits: np.ndarray, k_bits: np.ndarray, v_bits: np.ndarray, cu_q: np.ndarray, cu_kv: np.ndarray,
                    q_starts: Sequence[int], block: int, sel_idx: np.ndarray, sel_cnt: np.ndarray,
                    softmax_scale: float = 0.0, rows: Optional[np.ndarray] = None, want_lse: bool = True):
    Tq, hq, d = q_bits.shape
    hkv = k_bits.shape[1]
    cu_q = np.ascontiguousarray(cu_q, dtype=np.int32)
    cu_kv = np.ascontiguousarray(cu_kv, dtype=np.int32)
    qs = np.ascontiguousarray(q_starts, dtype=np.int32)
    if softmax_scale == 0.0:
        softmax_scale = 1.0 / np.sqrt(d)
    rq_tot = sel_cnt.shape[1]
    if rows is None:
        hh, rr = np.meshgrid(np.arange(hq, dtype=np.int32), np.arange(rq_tot, dtype=np.int32), indexing="ij")
        rows = np.stack([hh.ravel(), rr.ravel()], axis=1)
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    O = np.full((Tq, hq, d), np.nan, dtype=np.float32)
    lse = np.full((hq, Tq), np.nan, dtype=np.float32) if want_lse else None
    qst, qsh = _strides(q_bits)
    kst, ksh = _strides(k_bits)
    assert _strides(v_bits) == (kst, ksh)
    sel_idx = np.ascontiguousarray(sel_idx, dtype=np.int32)
    sel_cnt = np.ascontiguousarray(sel_cnt, dtype=np.int32)
    _load().so_attention_chunk(_p(q_bits), ctypes.c_int64(qst), ctypes.c_int64(qsh), _p(k_bits), _p(v_bits),
                               ctypes.c_int64(kst), ctypes.c_int64(ksh), ctypes.c_int32(hq), ctypes.c_int32(hkv),
                               ctypes.c_int32(d), ctypes.c_int32(len(cu_q) - 1), _p(cu_q), _p(cu_kv), _p(qs),
                               ctypes.c_int32(block), _p(sel_idx), _p(sel_cnt), ctypes.c_int32(sel_idx.shape[2]),
                               ctypes.c_float(softmax_scale), _p(rows), ctypes.c_int64(len(rows)), _p(O), _p(lse))
    return O, lse


def prefill_chunk(q_bits, k_bits, v_bits, cu_q, cu_kv, q_starts, total_lens, p: StemParams,
                  rows: Optional[np.ndarray] = None):
    """All of Algorithm 1 for one chunk of every sequence: Q holds the chunk's tokens, K / V the prefix
    up to the chunk's end.  Returns dict with M, sel_idx, sel_cnt, k_eff, O, lse (chunk rows / tokens)."""
    kv_lens = np.diff(cu_kv)
    nkb, r0 = chunk_geometry(kv_lens, q_starts, p.block)
    qbar = pool_mean(q_bits, cu_q, p.block)
    kbar = pool_mean(k_bits, cu_kv, p.block)
    mv = value_magnitude(v_bits, cu_kv, p.block)
    assert qbar.shape[1] == int((nkb - r0).sum()), "the chunk must end where the prefix ends"
    M = metric_chunk(qbar, kbar, mv, nkb, r0, p.beta, p.score_scale)
    k_eff = schedule_chunk(kv_lens, q_starts, total_lens, p)
    idx, cnt = select_chunk(M, nkb, r0, k_eff, p.stem_blocks, p.local_blocks)
    O, lse = attention_chunk(q_bits, k_bits, v_bits, cu_q, cu_kv, q_starts, p.block, idx, cnt, p.softmax_scale, rows)
    return {"M": M, "k_eff": k_eff, "sel_idx": idx, "sel_cnt": cnt, "O": O, "lse": lse}


def merge_partitions(o_parts, lse_parts):
    """Exact combination of attention over disjoint key partitions from the partial outputs and their
    log-sum-exps: O = sum_p exp(lse_p - lse) O_p with lse = log sum_p exp(lse_p).  o_parts [P][T,H,d],
    lse_parts [P][H,T]; a partition without keys has lse = -inf and contributes nothing."""
    lse_all = np.stack([np.asarray(x, dtype=np.float64) for x in lse_parts])      # [P, H, T]
    mx = lse_all.max(axis=0)
    w = np.exp(lse_all - mx)                                                        # exp(-inf) = 0
    tot = w.sum(axis=0)
    out = np.zeros(np.asarray(o_parts[0]).shape, dtype=np.float64)
    for o, wp in zip(o_parts, w):
        out += np.nan_to_num(np.asarray(o, dtype=np.float64)) * (wp / tot).T[:, :, None]
    return out, mx + np.log(tot)


# ----------------------------------------------------------------------------------------------
# Group-shared selection (Main Results: integration with a block-level top-k shared per GQA group)
# ----------------------------------------------------------------------------------------------

def metric_shared(qbar: np.ndarray, kbar: np.ndarray, mv: np.ndarray, nblk: np.ndarray, beta: float,
                  score_scale: float = 1.0) -> np.ndarray:
    """The group's metric: mean over the group's query heads of Eq. 7 -> fp32 [H_kv, sum_b N_blk_b^2]."""
    hq, r_tot, d = qbar.shape
    hkv = kbar.shape[0]
    nblk = np.ascontiguousarray(nblk, dtype=np.int32)
    m_tot = int((nblk.astype(np.int64) ** 2).sum())
    M = np.full((hkv, m_tot), np.nan, dtype=np.float32)
    _load().so_metric_shared(_p(np.ascontiguousarray(qbar)), _p(np.ascontiguousarray(kbar)), _p(np.ascontiguousarray(mv)),
                             ctypes.c_int32(hq), ctypes.c_int32(hkv), ctypes.c_int32(d), ctypes.c_int32(len(nblk)), _p(nblk),
                             ctypes.c_float(beta), ctypes.c_float(score_scale), _p(M))
    return M


def expand_group_lists(idx_g: np.ndarray, cnt_g: np.ndarray, g: int):
    """Per-kv-head lists [H_kv, R, k] -> per-query-head lists [H_kv * g, R, k] (every head of a group gets its list)."""
    return np.repeat(idx_g, g, axis=0), np.repeat(cnt_g, g, axis=0)


# ----------------------------------------------------------------------------------------------
# Anti-diagonal scoring mode (Overall Algorithm; Alg. 1 step 1 comment)
# ----------------------------------------------------------------------------------------------

def metric_antidiag(q_bits: np.ndarray, k_bits: np.ndarray, mv: np.ndarray, cu_seqlens: np.ndarray, block: int,
                    beta: float, score_scale: float = 1.0) -> np.ndarray:
    """Metric with the routing term taken as the mean of the token scores along the main anti-diagonal of every
    B x B score block -> fp32 [H_q, sum_b N_blk_b^2] (entries j <= r defined, rest NaN)."""
    T, hq, d = q_bits.shape
    hkv = k_bits.shape[1]
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    nblk = n_blocks(np.diff(cu), block)
    m_tot = int((nblk.astype(np.int64) ** 2).sum())
    M = np.full((hq, m_tot), np.nan, dtype=np.float32)
    qs, qh = _strides(q_bits)
    ks, kh = _strides(k_bits)
    _load().so_metric_antidiag(_p(q_bits), ctypes.c_int64(qs), ctypes.c_int64(qh), _p(k_bits), ctypes.c_int64(ks),
                               ctypes.c_int64(kh), _p(np.ascontiguousarray(mv, dtype=np.float32)), ctypes.c_int32(hq),
                               ctypes.c_int32(hkv), ctypes.c_int32(d), ctypes.c_int32(len(cu) - 1), _p(cu),
                               ctypes.c_int32(block), ctypes.c_float(beta), ctypes.c_float(score_scale), _p(M))
    return M


def score_antidiag(q_bits, k_bits, v_bits, cu_seqlens, p: StemParams):
    """Steps 1 and 3a in the anti-diagonal scoring mode. Returns (M, mv)."""
    mv = value_magnitude(v_bits, cu_seqlens, p.block)
    return metric_antidiag(q_bits, k_bits, mv, cu_seqlens, p.block, p.beta, p.score_scale), mv
