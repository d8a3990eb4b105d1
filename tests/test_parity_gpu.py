"""GPU parity: every stage of the CUDA path, called through the C ABI, against the CPU checker on
the same seeded inputs.  Integer work (budget, index lists) is compared bit for bit; the metric
and the attention output within the tolerances written in tests/_util.py."""
import numpy as np
import pytest
import torch

from oracle import stem_oracle as so
from paper_2603_06274_b200 import binding, workloads as wl
from paper_2603_06274_b200.binding import StemPlan
from tests._util import (check_attention, compare_selection, from_dev_bf16, metric_views, oracle_params,
                         sample_rows, to_dev)

pytestmark = pytest.mark.gpu

SMALL = {
    # several tiles, ragged tail (1000 = 7 full blocks + 104 tokens), GQA 2
    "ragged_b128": wl.small("ragged_b128", seqlens=(1000,), hq=4, hkv=2, block=128, permille=400),
    # block 64, MHA, more rows than one score/select tile
    "b64_mha": wl.small("b64_mha", seqlens=(2304,), hq=2, hkv=2, block=64, permille=250),
    # varlen batch with a sequence shorter than one block and a ragged one, GQA 7 (Qwen-like grouping)
    "varlen_g7": wl.small("varlen_g7", seqlens=(50, 1500, 641), hq=7, hkv=1, block=128, permille=300,
                          heavy_mode="window"),
    # sink recipe, longer rows, local 2
    "sink_4k": wl.small("sink_4k", seqlens=(4096,), hq=8, hkv=2, block=128, permille=200, sink=True, local_blocks=2),
    # no decay, forced blocks dominate (tiny budget)
    "forced_only": wl.small("forced_only", seqlens=(2048,), hq=2, hkv=1, block=128, permille=10, mu_num=1, mu_den=1),
    # value elements of order one (V_t = g_t z_t): outputs about sqrt(d) times larger, the scale the absolute
    # attention tolerances were stated for
    "gain_v_b128": wl.small("gain_v_b128", seqlens=(3000, 1100), hq=4, hkv=2, block=128, permille=300, sink=True,
                            v_recipe="gain_lognormal"),
    "gain_v_b64": wl.small("gain_v_b64", seqlens=(2500,), hq=3, hkv=1, block=64, permille=200,
                           v_recipe="gain_lognormal"),
}


def _setup(w: wl.Workload):
    data = wl.make_qkv(w)
    plan = StemPlan.from_workload(w)
    q, k, v = to_dev(data["q"]), to_dev(data["k"]), to_dev(data["v"])
    return data, plan, q, k, v


def _alloc_lists(plan: StemPlan):
    info = plan.info
    idx = torch.full((plan.num_q_heads, info.total_q_blocks, info.k_max), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((plan.num_q_heads, info.total_q_blocks), -7, dtype=torch.int32, device="cuda")
    return idx, cnt


def _ok(plan):
    st, detail = binding.stem_check_status(plan)
    assert st == 0, f"device status {st} detail {detail}"


@pytest.mark.parametrize("name", list(SMALL))
def test_plan_tables_match_checker(name):
    w = SMALL[name]
    plan = StemPlan.from_workload(w)
    k_eff = so.schedule_batch(w.seqlens, oracle_params(w))
    assert np.array_equal(plan.budget().numpy(), k_eff)
    nblk = so.n_blocks(w.seqlens, w.block)
    assert plan.info.total_q_blocks == int(nblk.sum())
    assert plan.info.k_max == int(k_eff.max())
    assert plan.info.metric_elems == int((nblk.astype(np.int64) ** 2).sum())
    assert plan.info.selected_blocks == int(k_eff.sum()) * w.num_q_heads
    assert plan.info.causal_blocks == sum(int(nb) * (int(nb) + 1) // 2 for nb in nblk) * w.num_q_heads
    # unmasked pairs of dense causal attention: n(n+1)/2 per sequence and head
    assert plan.info.causal_pairs == sum(n * (n + 1) // 2 for n in w.seqlens) * w.num_q_heads


@pytest.mark.parametrize("name", list(SMALL))
def test_score_matches_checker(name):
    w = SMALL[name]
    data, plan, q, k, v = _setup(w)
    M = torch.full((w.num_q_heads, plan.info.metric_elems), float("nan"), dtype=torch.float32, device="cuda")
    binding.stem_score(plan, q, k, v, M)
    torch.cuda.synchronize()
    M_ref, *_ = so.score(data["q"], data["k"], data["v"], data["cu_seqlens"], oracle_params(w))
    M_gpu = M.cpu().numpy()
    defined = ~np.isnan(M_ref)
    assert np.array_equal(np.isnan(M_gpu), ~defined), "exactly the causal blocks j <= r are written"
    err = np.abs(M_gpu[defined] - M_ref[defined])
    tol = 2e-6 * np.maximum(1.0, np.abs(M_ref[defined])) + 1e-6
    assert np.all(err <= tol), f"metric max err {err.max()}"


@pytest.mark.parametrize("name", list(SMALL))
def test_select_bit_exact_from_checker_scores(name):
    w = SMALL[name]
    data, plan, q, k, v = _setup(w)
    p = oracle_params(w)
    M_ref, *_ = so.score(data["q"], data["k"], data["v"], data["cu_seqlens"], p)
    nblk = so.n_blocks(w.seqlens, w.block)
    k_eff = so.schedule_batch(w.seqlens, p)
    idx_ref, cnt_ref = so.select(M_ref, nblk, k_eff, w.stem_blocks, w.local_blocks)
    idx, cnt = _alloc_lists(plan)
    binding.stem_select(plan, torch.from_numpy(np.nan_to_num(M_ref, nan=0.0)).cuda(), idx, cnt)
    torch.cuda.synchronize()
    assert np.array_equal(cnt.cpu().numpy(), cnt_ref)
    assert np.array_equal(idx.cpu().numpy(), idx_ref)


@pytest.mark.parametrize("ties", [False, True])
def test_select_bit_exact_on_random_scores_with_ties(ties):
    nb, heads = 200, 4
    w = wl.small("scores", seqlens=(nb * 128,), hq=heads, hkv=2, block=128, permille=150, stem_blocks=3,
                 local_blocks=2)
    M = wl.make_scores(99, heads, nb, ties=ties)
    if ties:
        M[1, 150, 17] = np.nan
        M[2, 190, 60:70] = np.inf
        M[3, 180, 30:40] = -np.inf
    plan = StemPlan.from_workload(w)
    p = oracle_params(w)
    k_eff = so.schedule_batch(w.seqlens, p)
    idx_ref, cnt_ref = so.select(M.reshape(heads, -1), np.array([nb]), k_eff, 3, 2)
    idx, cnt = _alloc_lists(plan)
    binding.stem_select(plan, torch.from_numpy(M.reshape(heads, -1)).cuda(), idx, cnt)
    torch.cuda.synchronize()
    assert np.array_equal(cnt.cpu().numpy(), cnt_ref)
    assert np.array_equal(idx.cpu().numpy(), idx_ref)


def test_select_from_caller_metric_with_more_than_1024_blocks():
    """stem_select on a caller's M for a sequence of 1025..2048 blocks (two key sets per lane)."""
    nb, heads = 1500, 2
    w = wl.small("scores_long", seqlens=(nb * 64 - 17,), hq=heads, hkv=1, block=64, permille=60, stem_blocks=2,
                 local_blocks=3)
    M = wl.make_scores(123, heads, nb, ties=True)
    M[0, 1400, 900:910] = np.nan
    M[1, 1499, 5:1200:7] = np.inf
    plan = StemPlan.from_workload(w)
    assert plan.info.total_q_blocks == nb
    p = oracle_params(w)
    k_eff = so.schedule_batch(w.seqlens, p)
    idx_ref, cnt_ref = so.select(M.reshape(heads, -1), np.array([nb]), k_eff, 2, 3)
    idx, cnt = _alloc_lists(plan)
    binding.stem_select(plan, torch.from_numpy(M.reshape(heads, -1)).cuda(), idx, cnt)
    torch.cuda.synchronize()
    assert np.array_equal(cnt.cpu().numpy(), cnt_ref)
    assert np.array_equal(idx.cpu().numpy(), idx_ref)


@pytest.mark.parametrize("name", list(SMALL))
def test_sparse_attention_matches_checker_on_checker_lists(name):
    w = SMALL[name]
    data, plan, q, k, v = _setup(w)
    ref = so.prefill(data["q"], data["k"], data["v"], data["cu_seqlens"], oracle_params(w))
    idx = torch.from_numpy(ref["sel_idx"]).cuda()
    cnt = torch.from_numpy(ref["sel_cnt"]).cuda()
    out = torch.full((w.total_tokens, w.num_q_heads, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((w.num_q_heads, w.total_tokens), float("nan"), dtype=torch.float32, device="cuda")
    binding.stem_sparse_prefill(plan, q, k, v, idx, cnt, out, lse)
    _ok(plan)
    check_attention(from_dev_bf16(out), ref["O"], label=name)
    assert np.abs(lse.cpu().numpy() - ref["lse"]).max() < 1e-3
    # a second run must reproduce the first bit for bit (barrier / TMEM protocol check)
    out2 = torch.empty_like(out)
    binding.stem_sparse_prefill(plan, q, k, v, idx, cnt, out2, None)
    _ok(plan)
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))


@pytest.mark.parametrize("name", ["ragged_b128", "b64_mha", "varlen_g7"])
def test_dense_mode_matches_dense_causal_attention(name):
    w = SMALL[name]
    data, plan, q, k, v = _setup(w)
    idx, cnt = so.dense_lists(w.seqlens, w.block, w.num_q_heads)
    O_ref, _ = so.attention(data["q"], data["k"], data["v"], data["cu_seqlens"], w.block, idx, cnt)
    out = torch.full((w.total_tokens, w.num_q_heads, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    binding.stem_sparse_prefill(plan, q, k, v, None, None, out, None)
    _ok(plan)
    check_attention(from_dev_bf16(out), O_ref)


@pytest.mark.parametrize("name", list(SMALL))
def test_fused_prefill_matches_checker(name):
    w = SMALL[name]
    data, plan, q, k, v = _setup(w)
    p = oracle_params(w)
    ref = so.prefill(data["q"], data["k"], data["v"], data["cu_seqlens"], p, rows=np.zeros((0, 2), np.int32))
    idx, cnt = _alloc_lists(plan)
    out = torch.full((w.total_tokens, w.num_q_heads, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    binding.stem_prefill(plan, q, k, v, out, idx, cnt)
    _ok(plan)
    assert plan.last_launch_count() >= 3  # pooling phases, score/select phases, attention
    idx_g, cnt_g = idx.cpu().numpy(), cnt.cpu().numpy()
    nblk = so.n_blocks(w.seqlens, w.block)
    ties = compare_selection(idx_g, cnt_g, ref["sel_idx"], ref["sel_cnt"], ref["M"], nblk, w)
    for t in ties:
        print(f"near-tie at head {t[0]} row {t[1]}: relative gap {t[2]:.2e}")
    assert len(ties) <= max(2, idx_g.shape[0] * idx_g.shape[1] // 100)
    # attention is compared on the index set the GPU actually used
    O_ref, _ = so.attention(data["q"], data["k"], data["v"], data["cu_seqlens"], w.block, idx_g, cnt_g)
    check_attention(from_dev_bf16(out), O_ref)
    # lists may stay inside the workspace
    out2 = torch.empty_like(out)
    binding.stem_prefill(plan, q, k, v, out2)
    _ok(plan)
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))


def test_strided_inputs():
    """Q/K/V as slices of one fused QKV projection output (token stride larger than heads * d)."""
    w = wl.small("strided", seqlens=(1200,), hq=4, hkv=2, block=128, permille=300)
    data = wl.make_qkv(w)
    T = w.total_tokens
    fused = torch.zeros((T, 4 + 2 + 2, 128), dtype=torch.bfloat16, device="cuda")
    fused[:, :4] = to_dev(data["q"])
    fused[:, 4:6] = to_dev(data["k"])
    fused[:, 6:8] = to_dev(data["v"])
    q, k, v = fused[:, :4], fused[:, 4:6], fused[:, 6:8]
    plan = StemPlan.from_workload(w, q_strides=(8 * 128, 128), kv_strides=(8 * 128, 128))
    out = torch.empty((T, 4, 128), dtype=torch.bfloat16, device="cuda")
    idx, cnt = _alloc_lists(plan)
    binding.stem_prefill(plan, q, k, v, out, idx, cnt)
    _ok(plan)
    plan_c = StemPlan.from_workload(w)
    out_c = torch.empty_like(out)
    idx_c, cnt_c = _alloc_lists(plan_c)
    binding.stem_prefill(plan_c, q.contiguous(), k.contiguous(), v.contiguous(), out_c, idx_c, cnt_c)
    _ok(plan_c)
    assert torch.equal(idx, idx_c) and torch.equal(out.view(torch.int16), out_c.view(torch.int16))


def test_argument_errors_enqueue_nothing():
    w = SMALL["ragged_b128"]
    data, plan, q, k, v = _setup(w)
    out = torch.empty((w.total_tokens, w.num_q_heads, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.StemError) as e:
        binding.stem_prefill(plan, q, k, v, out, workspace=torch.zeros(1024, dtype=torch.uint8, device="cuda"))
    assert e.value.status == binding.STEM_ERR_WORKSPACE
    with pytest.raises(binding.StemError) as e:
        binding.stem_prefill(plan, q, k, v, None)
    assert e.value.status == binding.STEM_ERR_INVALID_ARG
    idx, cnt = _alloc_lists(plan)
    with pytest.raises(binding.StemError) as e:
        binding.stem_sparse_prefill(plan, q, k, v, idx, None, out)
    assert e.value.status == binding.STEM_ERR_INVALID_ARG
    with pytest.raises(binding.StemError) as e:
        binding.stem_prefill(plan, q.view(-1)[1:-7].view(-1), k, v, out)  # 2-byte offset: misaligned
    assert e.value.status == binding.STEM_ERR_INVALID_ARG
