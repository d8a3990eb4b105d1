"""GPU parity of the anti-diagonal scoring mode (Overall Algorithm, "anti-diagonal scoring"; Alg. 1 step 1
comment, stride = B): the metric from the tensor-core contraction of Q with K against the CPU checker's
plain anti-diagonal means, then selection and attention through the fused path."""
import numpy as np
import pytest
import torch

from oracle import stem_oracle as so
from paper_2603_06274_b200 import binding, workloads as wl
from paper_2603_06274_b200.binding import StemPlan
from tests._util import check_attention, compare_selection, from_dev_bf16, oracle_params, sample_rows, to_dev

pytestmark = pytest.mark.gpu

# The contraction adds B * d = 16384 exact bf16 products into one fp32 tensor-memory accumulator over 1024 MMAs, and
# the tensor core's accumulation truncates: a running sum of a few hundred picks up about 1e-2 before the division
# by B, i.e. about 1e-4 on metric values of order 1 (measured 1.4e-4).  The checker sums in fp64.  Lists may then
# differ from the checker's only at near-ties of 1e-3 relative, like on the block-mean path.
METRIC_ABS, METRIC_REL = 3e-4, 1e-4

CASES = {
    # full blocks only, two column tiles
    "full_b128": wl.small("ad_full_b128", seqlens=(130 * 128,), hq=2, hkv=1, block=128, permille=100, sink=True),
    # ragged last block (its metric row comes from the plain-FMA kernel), GQA 3, varlen batch with a tiny sequence
    "ragged_varlen": wl.small("ad_ragged", seqlens=(1000, 50, 1664), hq=6, hkv=2, block=128, permille=300),
    # block 64
    "b64": wl.small("ad_b64", seqlens=(2500,), hq=2, hkv=2, block=64, permille=250),
}


@pytest.mark.parametrize("name", list(CASES))
def test_antidiagonal_metric_and_fused_path_match_checker(name):
    w = CASES[name]
    data = wl.make_qkv(w)
    p = oracle_params(w)
    M_ref, _ = so.score_antidiag(data["q"], data["k"], data["v"], data["cu_seqlens"], p)
    q, k, v = to_dev(data["q"]), to_dev(data["k"]), to_dev(data["v"])
    plan = StemPlan.from_workload(w, score_mode=1)
    info = plan.info
    M = torch.full((w.num_q_heads, info.metric_elems), float("nan"), dtype=torch.float32, device="cuda")
    binding.stem_score(plan, q, k, v, M)
    assert binding.stem_check_status(plan)[0] == 0
    M_g = M.cpu().numpy()
    defined = ~np.isnan(M_ref)
    assert np.array_equal(np.isnan(M_g), ~defined), "exactly the causal blocks j <= r are written"
    err = np.abs(M_g[defined] - M_ref[defined])
    assert np.all(err <= METRIC_ABS + METRIC_REL * np.abs(M_ref[defined])), f"metric max err {err.max()}"
    # fused path
    nblk = so.n_blocks(w.seqlens, w.block)
    k_eff = so.schedule_batch(w.seqlens, p)
    idx_ref, cnt_ref = so.select(M_ref, nblk, k_eff, w.stem_blocks, w.local_blocks)
    idx = torch.full((w.num_q_heads, info.total_q_blocks, info.k_max), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((w.num_q_heads, info.total_q_blocks), -7, dtype=torch.int32, device="cuda")
    out = torch.full((w.total_tokens, w.num_q_heads, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    binding.stem_prefill(plan, q, k, v, out, idx, cnt)
    assert binding.stem_check_status(plan)[0] == 0
    idx_g, cnt_g = idx.cpu().numpy(), cnt.cpu().numpy()
    ties = compare_selection(idx_g, cnt_g, idx_ref, cnt_ref, M_ref, nblk, w)
    assert len(ties) <= max(2, idx_g.shape[0] * idx_g.shape[1] // 100)
    O_ref, _ = so.attention(data["q"], data["k"], data["v"], data["cu_seqlens"], w.block, idx_g, cnt_g)
    check_attention(from_dev_bf16(out), O_ref, label=w.name)
    # the lists differ from the block-mean mode's (another scoring rule), so the mode switch is live
    plan0 = StemPlan.from_workload(w)
    idx0, cnt0 = torch.empty_like(idx), torch.empty_like(cnt)
    binding.stem_score_select(plan0, q, k, v, idx0, cnt0)
    torch.cuda.synchronize()
    assert torch.equal(cnt0, cnt)
    if name != "ragged_varlen":     # (its sequences are so short that every causal block is kept in either mode)
        assert not torch.equal(idx0, idx)
    plan.close(); plan0.close()


def test_antidiagonal_mode_limits():
    w = CASES["b64"]
    for kw in (dict(share_group=True), dict(kcache_blocks_per_seq=64)):
        with pytest.raises(binding.StemError) as e:
            StemPlan.from_workload(w, score_mode=1, **kw)
        assert e.value.status == binding.STEM_ERR_UNSUPPORTED


def test_32k_layer_in_antidiagonal_mode():
    w = wl.CONFIGS["cfg2"]
    data = wl.make_qkv(w)
    p = oracle_params(w)
    # the checker's anti-diagonal metric of two query heads (heads 0 and 9) in full: 33 k block pairs x 128 dots each
    sub = {"q": np.ascontiguousarray(data["q"][:, [0, 9]]), "k": np.ascontiguousarray(data["k"][:, [0, 2]]),
           "v": np.ascontiguousarray(data["v"][:, [0, 2]])}
    M_ref, _ = so.score_antidiag(sub["q"], sub["k"], sub["v"], data["cu_seqlens"], p)
    q, k, v = to_dev(data["q"]), to_dev(data["k"]), to_dev(data["v"])
    plan = StemPlan.from_workload(w, score_mode=1)
    info = plan.info
    M = torch.full((w.num_q_heads, info.metric_elems), float("nan"), dtype=torch.float32, device="cuda")
    binding.stem_score(plan, q, k, v, M)
    assert binding.stem_check_status(plan)[0] == 0
    M_g = M[[0, 9]].cpu().numpy()
    defined = ~np.isnan(M_ref)
    assert np.array_equal(np.isnan(M_g), ~defined)
    err = np.abs(M_g[defined] - M_ref[defined])
    print(f"anti-diagonal metric at 32K: max abs err {err.max():.2e}")
    assert np.all(err <= METRIC_ABS + METRIC_REL * np.abs(M_ref[defined]))
    # fused path: lists of those heads against the checker, attention on sampled lists
    nblk = so.n_blocks(w.seqlens, w.block)
    k_eff = so.schedule_batch(w.seqlens, p)
    idx_ref, cnt_ref = so.select(M_ref, nblk, k_eff, w.stem_blocks, w.local_blocks)
    idx = torch.empty((w.num_q_heads, info.total_q_blocks, info.k_max), dtype=torch.int32, device="cuda")
    cnt = torch.empty((w.num_q_heads, info.total_q_blocks), dtype=torch.int32, device="cuda")
    out = torch.full((w.total_tokens, w.num_q_heads, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    binding.stem_prefill(plan, q, k, v, out, idx, cnt)
    assert binding.stem_check_status(plan)[0] == 0
    idx_g, cnt_g = idx.cpu().numpy(), cnt.cpu().numpy()
    ties = compare_selection(idx_g[[0, 9]], cnt_g[[0, 9]], idx_ref, cnt_ref, M_ref, nblk, w)
    print(f"{len(ties)} of {2 * info.total_q_blocks} lists differ from the checker at near-ties")
    assert len(ties) <= 4
    rows = sample_rows(w.num_q_heads, nblk, [24, 25], n_random=60, seed=11)
    O_ref, _ = so.attention(data["q"], data["k"], data["v"], data["cu_seqlens"], w.block, idx_g, cnt_g, rows=rows, want_lse=False)
    mask = ~np.isnan(O_ref)
    check_attention(from_dev_bf16(out), O_ref, mask, label=f"{w.name} anti-diagonal mode ({len(rows)} lists)")
    assert torch.isfinite(out.float()).all()
    plan.close()
