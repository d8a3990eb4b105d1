"""Seeded synthetic workloads for the Stem prefill path.

This module holds only shapes, hyper-parameter values and random tensor
recipes.  None of the method's arithmetic (pooling, metric, schedule,
selection, attention) lives here, so both the CUDA path and the CPU checker
may draw their inputs from it.

Tensors are returned as numpy ``uint16`` arrays holding bf16 bit patterns in
the packed layout ``[T, H, d]`` (token-major, ``d`` contiguous); the same bytes
are handed to the GPU and to the checker.

The recipes stand in for the *shapes* of long-context prefill attention layers
(4K-128K tokens, Llama-3-8B / Qwen2.5-7B / Llama-3-70B head layouts, bf16,
block size 128; Section 3.1 and the implementation details of Section 3 of the
paper).  No benchmark items are involved.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np

HEAD_DIM = 128
BASE_SEED = 20260306


@dataclass(frozen=True)
class Workload:
    """One synthetic attention-layer workload and its Stem hyper-parameters."""

    name: str
    seqlens: Tuple[int, ...]
    num_q_heads: int
    num_kv_heads: int
    block: int
    budget_permille: int
    mu_num: int = 7
    mu_den: int = 10
    stem_blocks: int = 4
    local_blocks: int = 4
    min_blocks: int = 0
    beta: float = 0.2
    score_scale: float = 1.0
    k_start_blocks: int = 0
    head_dim: int = HEAD_DIM
    # input recipe switches
    heavy_mode: str = "bernoulli"   # "bernoulli": K row 0 + 2% of rows x4; "window": 8 rows per 4096-token window x4
    sink: bool = False              # add a shared direction to the first 4 K rows and to every Q row
    v_recipe: str = "norm_lognormal"  # "norm_lognormal": ||V_t|| itself is log-normal(0, 0.5) (elements ~ 0.1);
                                      # "gain_lognormal": V_t = g_t z_t with z_t ~ N(0, I), elements O(1)
    seed: int = BASE_SEED
    layers: int = 1

    @property
    def total_tokens(self) -> int:
        return int(sum(self.seqlens))

    @property
    def cu_seqlens(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.seqlens)]).astype(np.int32)

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def _cfg(idx: int, **kw) -> Workload:
    return Workload(seed=BASE_SEED + 1000 * idx, **kw)


# The five configurations of the build's baseline file.
CFG1 = _cfg(1, name="cfg1_tiny_4k_mha2_b64", seqlens=(4096,), num_q_heads=2, num_kv_heads=2,
            block=64, budget_permille=250)
CFG2 = _cfg(2, name="cfg2_llama3_8b_32k", seqlens=(32768,), num_q_heads=32, num_kv_heads=8,
            block=128, budget_permille=100, sink=True)
CFG3 = _cfg(3, name="cfg3_llama3_8b_128k", seqlens=(131072,), num_q_heads=32, num_kv_heads=8,
            block=128, budget_permille=50, local_blocks=2, sink=True)
CFG4 = _cfg(4, name="cfg4_qwen25_7b_varlen", seqlens=(65536, 40960), num_q_heads=28, num_kv_heads=4,
            block=128, budget_permille=50, heavy_mode="window")
CFG5 = _cfg(5, name="cfg5_llama3_70b_128k", seqlens=(131072,), num_q_heads=64, num_kv_heads=8,
            block=128, budget_permille=50, sink=True, layers=4)

CONFIGS: Dict[str, Workload] = {c.name.split("_")[0]: c for c in (CFG1, CFG2, CFG3, CFG4, CFG5)}

CFG4_BUDGET_SWEEP = (30, 50, 100, 200)
CFG5_DECAY_SWEEP = {"none": (1, 1), "linear": (1, 2), "paper": (7, 10)}


def small(name: str = "small", seqlens=(1024,), hq=4, hkv=2, block=128, permille=250, **kw) -> Workload:
    """A reduced workload for parity tests: same recipe, smaller shape."""
    return Workload(name=name, seqlens=tuple(seqlens), num_q_heads=hq, num_kv_heads=hkv, block=block,
                    budget_permille=permille, **kw)


# ----------------------------------------------------------------------------------------------
# bf16 helpers (bit-level; no arithmetic of the method)
# ----------------------------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even) and return the uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    out = ((u + rounding) >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) exactly to float32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------------------------
# generators
# ----------------------------------------------------------------------------------------------

_CHUNK = 8192  # tokens generated per step (bounds host memory)


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([seed, stream]))


def make_qkv(w: Workload, layer: int = 0) -> Dict[str, np.ndarray]:
    """Draw Q, K, V for one layer of workload ``w``.

    Returns a dict with ``q`` [T,Hq,d], ``k`` and ``v`` [T,Hkv,d] (uint16 bf16 bits) and
    ``cu_seqlens`` (int32 [batch+1]).

    Recipe: Q, K i.i.d. N(0,1).  V_t = g_t * z_t / ||z_t|| with z_t ~ N(0, I) and
    g_t = exp(0.5 n_t), n_t ~ N(0,1), per token and kv head, i.e. the per-token value norm is
    log-normal(0, 0.5): about half of the tokens have ||V_t|| < 1, so the max(0, .) clamp of the
    magnitude term is exercised, and block maxima of ln ||V|| are O(1).  With
    ``v_recipe = "gain_lognormal"`` the normalisation is left out (V_t = g_t z_t: elements of
    order one, norms about sqrt(d) times larger, outputs about sqrt(d) times larger).  A sparse set of K
    rows per kv head is scaled by 4 ("heavy" keys): either row 0 of each sequence plus a
    Bernoulli(0.02) subset, or 8 uniformly placed rows in every 4096-token window.  With
    ``sink`` a unit direction u per kv head is added (x8) to the first 4 K rows of each
    sequence and to every Q row of the heads that share that kv head, which creates an
    attention sink on the first block.
    """
    seed = w.seed + layer
    T, hq, hkv, d = w.total_tokens, w.num_q_heads, w.num_kv_heads, w.head_dim
    g = hq // hkv
    q = np.empty((T, hq, d), dtype=np.uint16)
    k = np.empty((T, hkv, d), dtype=np.uint16)
    v = np.empty((T, hkv, d), dtype=np.uint16)
    cu = w.cu_seqlens

    u = None
    if w.sink:
        u = _rng(seed, 7).standard_normal((hkv, d), dtype=np.float32)
        u /= np.linalg.norm(u, axis=1, keepdims=True)

    rq, rk, rv, rn, rh = (_rng(seed, s) for s in (1, 2, 3, 4, 5))
    seq_start = {int(s) for s in cu[:-1]}
    for t0 in range(0, T, _CHUNK):
        t1 = min(T, t0 + _CHUNK)
        n = t1 - t0
        qc = rq.standard_normal((n, hq, d), dtype=np.float32)
        kc = rk.standard_normal((n, hkv, d), dtype=np.float32)
        vc = rv.standard_normal((n, hkv, d), dtype=np.float32)
        gain = np.exp(0.5 * rn.standard_normal((n, hkv, 1), dtype=np.float32))
        if w.v_recipe == "norm_lognormal":
            vc *= gain / np.linalg.norm(vc, axis=2, keepdims=True)
        elif w.v_recipe == "gain_lognormal":
            vc *= gain
        else:
            raise ValueError(w.v_recipe)
        # heavy keys
        if w.heavy_mode == "bernoulli":
            heavy = rh.random((n, hkv)) < 0.02
        elif w.heavy_mode == "window":
            heavy = np.zeros((n, hkv), dtype=bool)
            for wnd in range(0, n, 4096):
                wl = min(4096, n - wnd)
                for h in range(hkv):
                    pos = rh.integers(0, wl, size=8)
                    heavy[wnd + pos, h] = True
        else:
            raise ValueError(w.heavy_mode)
        tok = np.arange(t0, t1)
        if w.heavy_mode == "bernoulli":
            for s in seq_start:
                if t0 <= s < t1:
                    heavy[s - t0, :] = True
        kc[heavy] *= 4.0
        if u is not None:
            # position of each token inside its own sequence
            seq_id = np.searchsorted(cu, tok, side="right") - 1
            local = tok - cu[seq_id]
            first4 = local < 4
            kc[first4] += 8.0 * u[None, :, :]
            qc += 8.0 * np.repeat(u, g, axis=0)[None, :, :]
        q[t0:t1] = f32_to_bf16_bits(qc)
        k[t0:t1] = f32_to_bf16_bits(kc)
        v[t0:t1] = f32_to_bf16_bits(vc)
    return {"q": q, "k": k, "v": v, "cu_seqlens": cu}


def make_scores(seed: int, heads: int, n_blk: int, ties: bool = False) -> np.ndarray:
    """A random lower-triangular metric tensor [heads, n_blk, n_blk] (float32) for selection tests.

    With ``ties`` the values are quantised so that equal scores occur often (tie-break coverage).
    """
    r = _rng(seed, 11)
    m = r.standard_normal((heads, n_blk, n_blk), dtype=np.float32)
    if ties:
        m = np.round(m * 4.0) / 4.0
        m[m == 0.0] = np.where(r.random(int((m == 0.0).sum())) < 0.5, np.float32(0.0), np.float32(-0.0))
    return m.astype(np.float32)
