"""Shared helpers for the GPU parity tests (device upload, oracle parameter mapping, comparisons)."""
from __future__ import annotations

import numpy as np
import torch

from oracle import stem_oracle as so
from paper_2603_06274_b200 import workloads as wl

# Tolerances of the attention output against the fp64 checker for bf16 inputs, same index set.
ATTN_MAX_ABS = 2e-2
ATTN_MEAN_ABS = 2e-3
# A selection mismatch is tolerated only where the k-th / (k+1)-th metric values are this close.
TIE_REL = 1e-3


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> CUDA bfloat16 tensor with the same bytes."""
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def from_dev_bf16(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy()


def oracle_params(w: wl.Workload) -> so.StemParams:
    return so.StemParams(block=w.block, budget_permille=w.budget_permille, k_start_blocks=w.k_start_blocks,
                         mu_num=w.mu_num, mu_den=w.mu_den, stem_blocks=w.stem_blocks, local_blocks=w.local_blocks,
                         min_blocks=w.min_blocks, beta=w.beta, score_scale=w.score_scale)


def metric_views(M_flat: np.ndarray, nblk: np.ndarray):
    """Split [H, sum nb^2] into per-sequence [H, nb, nb] views."""
    out, off = [], 0
    for nb in nblk:
        nb = int(nb)
        out.append(M_flat[:, off:off + nb * nb].reshape(M_flat.shape[0], nb, nb))
        off += nb * nb
    return out


def compare_selection(idx_gpu, cnt_gpu, idx_ref, cnt_ref, M_ref, nblk, w: wl.Workload):
    """Bit-exact comparison of index lists; rows that differ must be near-ties of the reference
    metric at the top-k boundary (relative gap <= TIE_REL).  Returns the list of logged near-ties."""
    assert np.array_equal(cnt_gpu, cnt_ref), "list lengths must equal the budget table"
    diff_rows = np.argwhere((idx_gpu != idx_ref).any(axis=2))
    logged = []
    if len(diff_rows) == 0:
        return logged
    views = metric_views(M_ref, nblk)
    row_off = np.concatenate([[0], np.cumsum(nblk)])
    for h, R in diff_rows:
        b = int(np.searchsorted(row_off, R, side="right") - 1)
        r = int(R - row_off[b])
        got = set(idx_gpu[h, R, :cnt_gpu[h, R]].tolist())
        want = set(idx_ref[h, R, :cnt_ref[h, R]].tolist())
        only_gpu, only_ref = got - want, want - got
        assert len(only_gpu) == len(only_ref) and all(0 <= j <= r for j in got)
        mrow = views[b][h, r]
        # every swapped pair must straddle the boundary within the tie tolerance
        top = max(float(mrow[j]) for j in only_ref)     # best block the GPU dropped
        bottom = min(float(mrow[j]) for j in only_gpu)  # worst block the GPU took instead
        gap = abs(top - bottom)
        scale = max(abs(top), abs(bottom), 1e-30)
        assert gap <= TIE_REL * scale, f"selection differs beyond a near-tie at head {h} row {R}: gap {gap}"
        logged.append((int(h), int(R), gap / scale))
    return logged


# The outputs of these workloads are small (|O| ~ 0.05 with unit-scale value norms), so the absolute
# bounds alone would accept errors of tens of per cent.  Scale-aware bounds beside them: the mean
# error against the mean magnitude of the reference and the largest error against its largest
# magnitude, over the compared elements.  bf16 rounding of the output alone is 2^-9 = 0.2 % relative.
ATTN_MEAN_REL = 1e-2
ATTN_MAX_REL = 5e-2
# The output is stored as bf16: rounding it moves an element by up to 2^-8 of its magnitude, which exceeds the
# absolute bound once |O| > 5 (value elements of order one give such outputs).  An element may therefore
# differ by the absolute bound or by two bf16 rounding steps of the reference value (one for the stored output,
# one for the probabilities, which enter the P V product as bf16), whichever is larger.
ATTN_BF16_STEPS = 2.0 * 2.0 ** -8


def check_attention(o_gpu: np.ndarray, o_ref: np.ndarray, mask=None, label: str = ""):
    if mask is None:
        mask = ~np.isnan(o_ref)
    ref = o_ref[mask].astype(np.float64)
    d = np.abs(o_gpu[mask].astype(np.float64) - ref)
    assert d.size > 0
    assert np.isfinite(o_gpu[mask]).all()
    mean_ref, max_ref = float(np.abs(ref).mean()), float(np.abs(ref).max())
    rel_mean = float(d.mean()) / max(mean_ref, 1e-30)
    rel_max = float(d.max()) / max(max_ref, 1e-30)
    print(f"{label or 'attention'}: {d.size // 128} rows, max abs {d.max():.3e} ({100 * rel_max:.3f} % of max |O| = "
          f"{max_ref:.3e}), mean abs {d.mean():.3e} ({100 * rel_mean:.3f} % of mean |O| = {mean_ref:.3e})")
    over = d - np.maximum(ATTN_MAX_ABS, ATTN_BF16_STEPS * np.abs(ref))
    assert over.max() <= 0.0, f"max abs {d.max()} (worst excess over the element-wise bound {over.max()})"
    assert d.mean() <= ATTN_MEAN_ABS, f"mean abs {d.mean()}"
    assert rel_mean <= ATTN_MEAN_REL, f"mean abs error is {100 * rel_mean:.2f} % of the mean output magnitude"
    assert rel_max <= ATTN_MAX_REL, f"max abs error is {100 * rel_max:.2f} % of the largest output magnitude"
    return float(d.max()), float(d.mean())


def sample_rows(hq: int, nblk: np.ndarray, k_s_rows, n_random: int, seed: int, full_heads=()):
    """(head, global row) pairs: structural rows of every head plus seeded random rows."""
    rng = np.random.default_rng(seed)
    rows = set()
    row_off = np.concatenate([[0], np.cumsum(nblk)])
    for b, nb in enumerate(nblk):
        nb = int(nb)
        special = {0, nb // 2, nb - 1} | {min(nb - 1, max(0, int(x))) for x in k_s_rows}
        for h in range(hq):
            for r in special:
                rows.add((h, int(row_off[b] + r)))
        for h in full_heads:
            for r in range(nb):
                rows.add((h, int(row_off[b] + r)))
    r_tot = int(row_off[-1])
    for _ in range(n_random):
        rows.add((int(rng.integers(hq)), int(rng.integers(r_tot))))
    return np.array(sorted(rows), dtype=np.int32)


def check_full_path(w: wl.Workload, data, q, k, v, n_random: int = 24, tie_budget=None, all_rows: bool = False):
    """Runs stem_prefill on the GPU for workload w and compares it with the checker: selection on
    every (head, row) (bit-exact except logged near-ties), attention on sampled lists computed on
    the index lists the GPU used.  Returns (idx_gpu, cnt_gpu, out)."""
    from paper_2603_06274_b200 import binding
    from paper_2603_06274_b200.binding import StemPlan
    plan = StemPlan.from_workload(w)
    info = plan.info
    idx = torch.full((w.num_q_heads, info.total_q_blocks, info.k_max), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((w.num_q_heads, info.total_q_blocks), -7, dtype=torch.int32, device="cuda")
    out = torch.full((w.total_tokens, w.num_q_heads, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    binding.stem_prefill(plan, q, k, v, out, idx, cnt)
    st, detail = binding.stem_check_status(plan)
    assert st == 0, f"device status {st} detail {detail}"
    idx_g, cnt_g = idx.cpu().numpy(), cnt.cpu().numpy()
    p = oracle_params(w)
    M_ref, *_ = so.score(data["q"], data["k"], data["v"], data["cu_seqlens"], p)
    nblk = so.n_blocks(w.seqlens, w.block)
    k_eff = so.schedule_batch(w.seqlens, p)
    assert np.array_equal(plan.budget().numpy(), k_eff)
    idx_ref, cnt_ref = so.select(M_ref, nblk, k_eff, w.stem_blocks, w.local_blocks)
    ties = compare_selection(idx_g, cnt_g, idx_ref, cnt_ref, M_ref, nblk, w)
    for t in ties[:20]:
        print(f"near-tie at head {t[0]} row {t[1]}: relative gap {t[2]:.2e}")
    n_lists = idx_g.shape[0] * idx_g.shape[1]
    print(f"{w.name}: {len(ties)} of {n_lists} lists differ from the checker at near-ties")
    assert len(ties) <= (max(2, n_lists // 200) if tie_budget is None else tie_budget)
    k_s = [so.k_start(int(nb), p) for nb in nblk]
    rows = None if all_rows else sample_rows(w.num_q_heads, nblk, [k_s[0] - 1, k_s[0]], n_random=n_random, seed=w.seed)
    O_ref, _ = so.attention(data["q"], data["k"], data["v"], data["cu_seqlens"], w.block, idx_g, cnt_g,
                            softmax_scale=0.0, rows=rows, want_lse=False)
    mask = ~np.isnan(O_ref)
    assert mask.any()
    check_attention(from_dev_bf16(out), O_ref, mask, label=f"{w.name} ({'every list' if all_rows else f'{len(rows)} sampled lists'})")
    assert torch.isfinite(out.float()).all()
    plan.close()
    return idx_g, cnt_g, out
