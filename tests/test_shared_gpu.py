"""GPU parity of group-shared selection: one index list per (kv head, row), decided on the mean over the group's
query heads of the Output-Aware Metric; every query head of the group attends over its group's list."""
import numpy as np
import pytest
import torch

from oracle import stem_oracle as so
from paper_2603_06274_b200 import binding, workloads as wl
from paper_2603_06274_b200.binding import StemPlan
from tests._util import check_attention, compare_selection, from_dev_bf16, oracle_params, sample_rows, to_dev

pytestmark = pytest.mark.gpu


def _reference(w, data):
    p = oracle_params(w)
    _, qbar, kbar, mv = so.score(data["q"], data["k"], data["v"], data["cu_seqlens"], p)
    nblk = so.n_blocks(w.seqlens, w.block)
    Mg = so.metric_shared(qbar, kbar, mv, nblk, p.beta, p.score_scale)
    k_eff = so.schedule_batch(w.seqlens, p)
    idx, cnt = so.select(Mg, nblk, k_eff, w.stem_blocks, w.local_blocks)
    return Mg, nblk, k_eff, idx, cnt


@pytest.mark.parametrize("w", [
    wl.small("shared_g3", seqlens=(1300, 260), hq=6, hkv=2, block=128, permille=300, sink=True),
    wl.small("shared_g7_b64", seqlens=(2100,), hq=7, hkv=1, block=64, permille=200, heavy_mode="window"),
])
def test_group_shared_selection_matches_checker(w):
    data = wl.make_qkv(w)
    g = w.num_q_heads // w.num_kv_heads
    Mg_ref, nblk, k_eff, idx_ref, cnt_ref = _reference(w, data)
    q, k, v = to_dev(data["q"]), to_dev(data["k"]), to_dev(data["v"])
    plan = StemPlan.from_workload(w, share_group=True)
    info = plan.info
    assert info.list_heads == w.num_kv_heads
    assert info.selected_blocks == int(k_eff.sum()) * w.num_q_heads     # every query head still attends over k_eff blocks
    # the group's metric
    M = torch.full((w.num_kv_heads, info.metric_elems), float("nan"), dtype=torch.float32, device="cuda")
    binding.stem_score(plan, q, k, v, M)
    torch.cuda.synchronize()
    M_g = M.cpu().numpy()
    defined = ~np.isnan(Mg_ref)
    assert np.array_equal(np.isnan(M_g), ~defined)
    assert np.all(np.abs(M_g[defined] - Mg_ref[defined]) <= 2e-6 * np.maximum(1.0, np.abs(Mg_ref[defined])) + 1e-6)
    # selection from the checker's group metric: bit-exact
    idx = torch.full((w.num_kv_heads, info.total_q_blocks, info.k_max), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((w.num_kv_heads, info.total_q_blocks), -7, dtype=torch.int32, device="cuda")
    binding.stem_select(plan, torch.from_numpy(np.nan_to_num(Mg_ref, nan=0.0)).cuda(), idx, cnt)
    torch.cuda.synchronize()
    assert np.array_equal(cnt.cpu().numpy(), cnt_ref) and np.array_equal(idx.cpu().numpy(), idx_ref)
    # the whole path
    out = torch.full((w.total_tokens, w.num_q_heads, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    binding.stem_prefill(plan, q, k, v, out, idx, cnt)
    assert binding.stem_check_status(plan)[0] == 0
    idx_g, cnt_g = idx.cpu().numpy(), cnt.cpu().numpy()
    ties = compare_selection(idx_g, cnt_g, idx_ref, cnt_ref, Mg_ref, nblk, w)
    assert len(ties) <= 2
    ei, ec = so.expand_group_lists(idx_g, cnt_g, g)
    O_ref, _ = so.attention(data["q"], data["k"], data["v"], data["cu_seqlens"], w.block, ei, ec)
    check_attention(from_dev_bf16(out), O_ref, label=w.name)
    plan.close()


def test_32k_layer_with_group_shared_lists():
    w = wl.CONFIGS["cfg2"]
    data = wl.make_qkv(w)
    g = w.num_q_heads // w.num_kv_heads
    Mg_ref, nblk, k_eff, idx_ref, cnt_ref = _reference(w, data)
    q, k, v = to_dev(data["q"]), to_dev(data["k"]), to_dev(data["v"])
    plan = StemPlan.from_workload(w, share_group=True)
    info = plan.info
    idx = torch.empty((w.num_kv_heads, info.total_q_blocks, info.k_max), dtype=torch.int32, device="cuda")
    cnt = torch.empty((w.num_kv_heads, info.total_q_blocks), dtype=torch.int32, device="cuda")
    out = torch.full((w.total_tokens, w.num_q_heads, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    binding.stem_prefill(plan, q, k, v, out, idx, cnt)
    assert binding.stem_check_status(plan)[0] == 0
    idx_g, cnt_g = idx.cpu().numpy(), cnt.cpu().numpy()
    ties = compare_selection(idx_g, cnt_g, idx_ref, cnt_ref, Mg_ref, nblk, w)
    print(f"{len(ties)} of {idx_g.shape[0] * idx_g.shape[1]} group lists differ from the checker at near-ties")
    assert len(ties) <= max(2, idx_g.shape[0] * idx_g.shape[1] // 200)
    ei, ec = so.expand_group_lists(idx_g, cnt_g, g)
    rows = sample_rows(w.num_q_heads, nblk, [10, 24, 25], n_random=100, seed=5, full_heads=(0, 1))
    O_ref, _ = so.attention(data["q"], data["k"], data["v"], data["cu_seqlens"], w.block, ei, ec, rows=rows, want_lse=False)
    mask = ~np.isnan(O_ref)
    check_attention(from_dev_bf16(out), O_ref, mask, label=f"{w.name} shared lists ({len(rows)} lists)")
    assert torch.isfinite(out.float()).all()
    plan.close()
