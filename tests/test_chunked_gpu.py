"""GPU parity of chunked prefill with global token offsets (the paper's Conclusion) and of the pooled-K cache.

A chunk call sees Q for the chunk's tokens and K / V for the prefix up to the chunk's end.  Its lists must equal
the CPU checker's chunk lists (and so the rows of the one-shot result), its outputs the checker's attention on
those lists; the cached path (K-side pooled tensors kept in caller memory across chunks, only the new blocks
pooled per chunk) must reproduce the workspace path bit for bit."""
import numpy as np
import pytest
import torch

from oracle import stem_oracle as so
from paper_2603_06274_b200 import binding, workloads as wl
from paper_2603_06274_b200.binding import StemPlan
from tests._util import check_attention, from_dev_bf16, oracle_params, to_dev

pytestmark = pytest.mark.gpu


def _chunk_inputs(data, cu, splits, c):
    nseq = len(splits)
    q_starts = [s[c] for s in splits]
    kv_lens = [s[c + 1] for s in splits]
    q = np.concatenate([data["q"][cu[b] + q_starts[b]:cu[b] + kv_lens[b]] for b in range(nseq)])
    k = np.concatenate([data["k"][cu[b]:cu[b] + kv_lens[b]] for b in range(nseq)])
    v = np.concatenate([data["v"][cu[b]:cu[b] + kv_lens[b]] for b in range(nseq)])
    cu_q = np.concatenate([[0], np.cumsum([kv_lens[b] - q_starts[b] for b in range(nseq)])]).astype(np.int32)
    cu_kv = np.concatenate([[0], np.cumsum(kv_lens)]).astype(np.int32)
    return q_starts, kv_lens, q, k, v, cu_q, cu_kv


def _plan(w, kv_lens, q_starts, **kw):
    return StemPlan.from_workload(w, seqlens=kv_lens, q_starts=q_starts, total_lens=w.seqlens, **kw)


@pytest.mark.parametrize("w,splits", [
    (wl.small("chunks_b128", seqlens=(1500, 900), hq=4, hkv=2, block=128, permille=400, sink=True),
     [(0, 512, 1024, 1500), (0, 256, 640, 900)]),
    (wl.small("chunks_b64", seqlens=(1000,), hq=2, hkv=1, block=64, permille=250, stem_blocks=2, local_blocks=3,
              mu_num=1, mu_den=2),
     [(0, 64, 704, 1000)]),
])
def test_chunk_calls_match_checker_and_cached_path_matches_workspace_path(w, splits):
    data = wl.make_qkv(w)
    cu = data["cu_seqlens"]
    p = oracle_params(w)
    cap = int(so.n_blocks(w.seqlens, w.block).max())
    cache = None
    for c in range(len(splits[0]) - 1):
        q_starts, kv_lens, q, k, v, cu_q, cu_kv = _chunk_inputs(data, cu, splits, c)
        ref = so.prefill_chunk(q, k, v, cu_q, cu_kv, q_starts, w.seqlens, p)
        qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
        plan = _plan(w, kv_lens, q_starts)
        info = plan.info
        assert info.total_tokens == q.shape[0] and info.total_kv_tokens == k.shape[0]
        assert np.array_equal(plan.budget().numpy(), ref["k_eff"])
        idx = torch.full((w.num_q_heads, info.total_q_blocks, info.k_max), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((w.num_q_heads, info.total_q_blocks), -7, dtype=torch.int32, device="cuda")
        out = torch.full((q.shape[0], w.num_q_heads, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((w.num_q_heads, q.shape[0]), float("nan"), dtype=torch.float32, device="cuda")
        binding.stem_prefill(plan, qd, kd, vd, out, idx, cnt, lse)
        assert binding.stem_check_status(plan)[0] == 0
        idx_g, cnt_g = idx.cpu().numpy(), cnt.cpu().numpy()
        assert np.array_equal(cnt_g, ref["sel_cnt"])
        n_diff = int((idx_g != ref["sel_idx"]).any(axis=2).sum())
        assert n_diff <= 1, f"{n_diff} chunk lists differ from the checker"
        O_ref, lse_ref = so.attention_chunk(q, k, v, cu_q, cu_kv, q_starts, w.block, idx_g, cnt_g)
        check_attention(from_dev_bf16(out), O_ref, label=f"{w.name} chunk {c}")
        assert np.abs(lse.cpu().numpy() - lse_ref).max() < 1e-3
        # the metric of the chunk's rows (rectangular: chunk rows x prefix blocks)
        M = torch.full((w.num_q_heads, info.metric_elems), float("nan"), dtype=torch.float32, device="cuda")
        binding.stem_score(plan, qd, kd, vd, M)
        torch.cuda.synchronize()
        M_g, M_ref = M.cpu().numpy(), ref["M"]
        defined = ~np.isnan(M_ref)
        assert np.array_equal(np.isnan(M_g), ~defined)
        assert np.all(np.abs(M_g[defined] - M_ref[defined]) <= 2e-6 * np.maximum(1.0, np.abs(M_ref[defined])) + 1e-6)
        # the same chunk through the pooled-K cache: only the chunk's new key blocks are pooled
        cplan = _plan(w, kv_lens, q_starts, kcache_blocks_per_seq=cap)
        if cache is None:
            cache = torch.full((int(cplan.info.kcache_bytes),), 0xff, dtype=torch.uint8, device="cuda")   # NaN patterns
        assert cplan.info.new_key_blocks == info.total_q_blocks
        idx2, cnt2, out2 = torch.empty_like(idx), torch.empty_like(cnt), torch.empty_like(out)
        binding.stem_prefill_cached(cplan, qd, kd, vd, out2, cache, True, idx2, cnt2)
        assert binding.stem_check_status(cplan)[0] == 0
        assert torch.equal(idx2, idx) and torch.equal(cnt2, cnt)
        assert torch.equal(out2.view(torch.int16), out.view(torch.int16))
        # scoring alone, reading only Q (the cache already holds this chunk's blocks)
        idx3, cnt3 = torch.empty_like(idx), torch.empty_like(cnt)
        binding.stem_score_select_cached(cplan, qd, cache, idx3, cnt3)
        torch.cuda.synchronize()
        assert torch.equal(idx3, idx) and torch.equal(cnt3, cnt)
        with pytest.raises(binding.StemError):
            binding.stem_prefill(cplan, qd, kd, vd, out2)       # a cache plan has no K side in its workspace
        plan.close(); cplan.close()


def test_chunk_plan_validation():
    w = wl.small("chunk_bad", seqlens=(1024,), hq=2, hkv=1, block=128, permille=300)
    for kw in (dict(q_starts=[100]), dict(q_starts=[1024]), dict(q_starts=[0], total_lens=[512]),
               dict(kcache_blocks_per_seq=4)):
        with pytest.raises(binding.StemError) as e:
            StemPlan.from_workload(w, **kw)
        assert e.value.status == binding.STEM_ERR_INVALID_ARG


def test_128k_layer_in_four_chunks_equals_the_one_shot_call():
    w = wl.CONFIGS["cfg3"]
    data = wl.make_qkv(w)
    q, k, v = to_dev(data["q"]), to_dev(data["k"]), to_dev(data["v"])
    N = w.seqlens[0]
    plan = StemPlan.from_workload(w)
    info = plan.info
    idx = torch.empty((w.num_q_heads, info.total_q_blocks, info.k_max), dtype=torch.int32, device="cuda")
    cnt = torch.empty((w.num_q_heads, info.total_q_blocks), dtype=torch.int32, device="cuda")
    out = torch.empty((N, w.num_q_heads, 128), dtype=torch.bfloat16, device="cuda")
    binding.stem_prefill(plan, q, k, v, out, idx, cnt)
    assert binding.stem_check_status(plan)[0] == 0
    cap = info.total_q_blocks
    cache = None
    step = N // 4
    for c in range(4):
        lo, hi = c * step, (c + 1) * step
        cplan = StemPlan.from_workload(w, seqlens=(hi,), q_starts=[lo], total_lens=[N], kcache_blocks_per_seq=cap)
        ci = cplan.info
        if cache is None:
            cache = torch.zeros(int(ci.kcache_bytes), dtype=torch.uint8, device="cuda")
        # the chunk's lists hold at most max k_eff over its rows entries; the one-shot lists are padded to their own k_max
        cidx = torch.empty((w.num_q_heads, ci.total_q_blocks, ci.k_max), dtype=torch.int32, device="cuda")
        ccnt = torch.empty((w.num_q_heads, ci.total_q_blocks), dtype=torch.int32, device="cuda")
        cout = torch.empty((hi - lo, w.num_q_heads, 128), dtype=torch.bfloat16, device="cuda")
        binding.stem_prefill_cached(cplan, q[lo:hi], k[:hi], v[:hi], cout, cache, True, cidx, ccnt)
        assert binding.stem_check_status(cplan)[0] == 0
        r_lo, r_hi = lo // w.block, hi // w.block
        assert torch.equal(ccnt, cnt[:, r_lo:r_hi])
        assert torch.equal(cidx, idx[:, r_lo:r_hi, :ci.k_max])
        assert torch.equal(cout.view(torch.int16), out[lo:hi].view(torch.int16))
        cplan.close()
    plan.close()
