"""GPU parity of the token-level path (Main Results: Token Position-Decay on a selector that keeps the top 2048
tokens per query, k_start = 2048, mu = 0.7): the budget k(t) of Eq. 3 at token positions, exact top-k(t) selection
from caller-supplied indexer scores, and gather-style attention over the token lists.  The CPU checker is
Algorithm 1's own code with a block size of one token."""
import numpy as np
import pytest
import torch

from oracle import stem_oracle as so
from paper_2603_06274_b200 import binding, workloads as wl
from tests._util import check_attention, from_dev_bf16, to_dev

pytestmark = pytest.mark.gpu


def _scores(seed, heads, n, ties):
    r = np.random.Generator(np.random.PCG64([seed, 31]))
    m = r.standard_normal((heads, n, n), dtype=np.float32)
    if ties:
        m = np.round(m * 3.0) / 3.0
        m[0, n - 1, 5:40] = np.nan
        m[heads - 1, n // 2, 0:n // 4:3] = np.inf
        m[0, n // 3, 10:20] = -np.inf
        m[m == 0.0] = -0.0
    return m


def _case(n, hq, hkv, k_start, stem, local, seed, ties, sample=None):
    w = wl.small(f"token_{n}", seqlens=(n,), hq=hq, hkv=hkv, block=64, permille=100, sink=True, seed=seed)
    data = wl.make_qkv(w)
    g = hq // hkv
    p = so.StemParams(block=1, k_start_blocks=k_start, mu_num=7, mu_den=10, stem_blocks=stem, local_blocks=local)
    k_ref = so.schedule(n, k_start, p)[1]
    k_tok = binding.stem_token_budget(n, k_start, (7, 10), stem, local)
    assert np.array_equal(k_tok.numpy(), k_ref)
    k_max = int(k_ref.max())
    sc = _scores(seed, hkv, n, ties)
    idx_ref, cnt_ref = so.select(sc.reshape(hkv, -1), np.array([n], np.int32), k_ref, stem, local)
    idx = torch.full((hkv, n, k_max), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((hkv, n), -7, dtype=torch.int32, device="cuda")
    binding.stem_token_select(torch.from_numpy(sc).cuda(), k_tok.cuda(), idx, cnt, stem, local)
    torch.cuda.synchronize()
    assert np.array_equal(cnt.cpu().numpy(), cnt_ref)
    assert np.array_equal(idx.cpu().numpy(), idx_ref)
    # gather attention on those lists; the checker runs Algorithm 1 step d with one token per block
    q, k, v = to_dev(data["q"]), to_dev(data["k"]), to_dev(data["v"])
    out = torch.full((n, hq, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((hq, n), float("nan"), dtype=torch.float32, device="cuda")
    binding.stem_token_attention(q, k, v, idx, cnt, out, lse)
    st, detail = binding.stem_token_check_status()
    assert st == 0, detail
    ei, ec = so.expand_group_lists(idx_ref, cnt_ref, g)
    rows = None
    if sample is not None:
        r = np.random.default_rng(seed)
        toks = np.unique(np.concatenate([[0, 1, k_start - 1, k_start, n // 2, n - 1], r.integers(0, n, sample)]))
        rows = np.array([(h, t) for h in range(hq) for t in toks], dtype=np.int32)
    O_ref, lse_ref = so.attention(data["q"], data["k"], data["v"], data["cu_seqlens"], 1, ei, ec, rows=rows)
    mask = ~np.isnan(O_ref)
    check_attention(from_dev_bf16(out), O_ref, mask, label=f"token-level n={n} k_start={k_start}")
    lm = ~np.isnan(lse_ref)
    assert np.abs(lse.cpu().numpy()[lm] - lse_ref[lm]).max() < 1e-3
    assert torch.isfinite(out.float()).all()


def test_token_level_selection_and_gather_attention_small():
    _case(n=700, hq=4, hkv=2, k_start=200, stem=4, local=8, seed=7, ties=True)
    _case(n=333, hq=3, hkv=3, k_start=64, stem=0, local=1, seed=8, ties=False)
    _case(n=520, hq=8, hkv=1, k_start=300, stem=2, local=3, seed=10, ties=False)   # 8 query heads on one kv head


def test_token_level_top_2048_selector():
    # the paper's setting for that integration: k_start = 2048, mu = 0.7; 4096 tokens, GQA 4
    _case(n=4096, hq=8, hkv=2, k_start=2048, stem=0, local=1, seed=9, ties=True, sample=40)


def test_token_level_rows_of_9000_tokens():
    # lists longer than one 2048-token budget window, rows that span several passes of every thread over the keys
    _case(n=9000, hq=2, hkv=1, k_start=2048, stem=2, local=4, seed=11, ties=True, sample=12)


def test_gather_attention_on_hand_made_lists_with_strided_tensors():
    # 16 query heads on one kv head (the widest group), lists of any length from 0 to 140 tokens (a list need not come
    # from the selector; empty lists give a zero row and lse = -inf), Q / K / V as slices of wider tensors
    n, hq, hkv = 300, 16, 1
    w = wl.small("token_lists", seqlens=(n,), hq=hq, hkv=hkv, block=64, permille=100, sink=False, seed=21)
    data = wl.make_qkv(w)
    r = np.random.default_rng(21)
    k_max = 140
    idx_ref = np.full((hkv, n, k_max), -1, np.int32)
    cnt_ref = np.zeros((hkv, n), np.int32)
    for t in range(n):
        m = 0 if r.random() < 0.1 else int(r.integers(1, min(t + 1, k_max) + 1))
        idx_ref[0, t, :m] = np.sort(r.choice(t + 1, size=m, replace=False))
        cnt_ref[0, t] = m
    q_wide = torch.zeros((n, hq + 4, 128), dtype=torch.bfloat16, device="cuda")
    k_wide = torch.zeros((n, 3, 128), dtype=torch.bfloat16, device="cuda")
    v_wide = torch.zeros((n, 3, 128), dtype=torch.bfloat16, device="cuda")
    q, k, v = q_wide[:, 2:2 + hq], k_wide[:, 1:2], v_wide[:, 1:2]
    q.copy_(to_dev(data["q"])); k.copy_(to_dev(data["k"])); v.copy_(to_dev(data["v"]))
    out = torch.full((n, hq, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((hq, n), float("nan"), dtype=torch.float32, device="cuda")
    binding.stem_token_attention(q, k, v, torch.from_numpy(idx_ref).cuda(), torch.from_numpy(cnt_ref).cuda(), out, lse)
    st, detail = binding.stem_token_check_status()
    assert st == 0, detail
    ei, ec = so.expand_group_lists(idx_ref, cnt_ref, hq // hkv)
    O_ref, lse_ref = so.attention(data["q"], data["k"], data["v"], data["cu_seqlens"], 1, ei, ec)
    check_attention(from_dev_bf16(out), O_ref, label="hand-made token lists, 16 heads per kv head")
    empty = cnt_ref[0] == 0
    assert empty.any()
    assert (from_dev_bf16(out)[empty] == 0).all()
    got_lse = lse.cpu().numpy()
    assert np.isneginf(got_lse[:, empty]).all() and np.isneginf(lse_ref[:, empty]).all()
    assert np.abs(got_lse[:, ~empty] - lse_ref[:, ~empty]).max() < 1e-3


@pytest.mark.parametrize("seed", [31, 32, 33, 34, 35, 36])
def test_gather_attention_on_random_shapes_and_list_lengths(seed):
    # item boundaries in every phase of the pipeline: lists of 0 .. 3 tiles in random order, any group size; the
    # result must also be the same bits on a second run
    r = np.random.default_rng(seed)
    hkv = int(r.integers(1, 4))
    g = int(r.choice([1, 2, 3, 4, 5, 8, 12, 16]))
    hq = hkv * g
    n = int(r.integers(130, 420))
    w = wl.small(f"token_fuzz_{seed}", seqlens=(n,), hq=hq, hkv=hkv, block=64, permille=100, sink=bool(seed & 1), seed=seed)
    data = wl.make_qkv(w)
    k_max = int(r.integers(1, n + 1))
    idx_ref = np.full((hkv, n, k_max), -1, np.int32)
    cnt_ref = np.zeros((hkv, n), np.int32)
    for h in range(hkv):
        for t in range(n):
            top = min(t + 1, k_max)
            m = int(r.choice([0, 1, min(top, 127), min(top, 128), min(top, 129), top, int(r.integers(0, top + 1))]))
            idx_ref[h, t, :m] = np.sort(r.choice(t + 1, size=m, replace=False))
            cnt_ref[h, t] = m
    q, k, v = to_dev(data["q"]), to_dev(data["k"]), to_dev(data["v"])
    idx, cnt = torch.from_numpy(idx_ref).cuda(), torch.from_numpy(cnt_ref).cuda()
    outs = []
    for _ in range(2):
        out = torch.full((n, hq, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((hq, n), float("nan"), dtype=torch.float32, device="cuda")
        binding.stem_token_attention(q, k, v, idx, cnt, out, lse)
        st, detail = binding.stem_token_check_status()
        assert st == 0, detail
        outs.append((out, lse))
    assert torch.equal(outs[0][0].view(torch.int16), outs[1][0].view(torch.int16))
    assert torch.equal(outs[0][1].view(torch.int32), outs[1][1].view(torch.int32))
    ei, ec = so.expand_group_lists(idx_ref, cnt_ref, g)
    O_ref, lse_ref = so.attention(data["q"], data["k"], data["v"], data["cu_seqlens"], 1, ei, ec)
    check_attention(from_dev_bf16(outs[0][0]), O_ref, label=f"random token lists, n={n}, {hq}/{hkv} heads, k_max={k_max}")
    got = outs[0][1].cpu().numpy()
    empty = np.repeat(cnt_ref == 0, g, axis=0)
    assert np.isneginf(got[empty]).all()
    assert np.abs(got[~empty] - lse_ref[~empty]).max() < 1e-3


def test_token_level_argument_errors():
    with pytest.raises(binding.StemError):
        binding.stem_token_budget(100, 10, (11, 10))
    q = torch.zeros((64, 34, 128), dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros((64, 2, 128), dtype=torch.bfloat16, device="cuda")
    idx = torch.zeros((2, 64, 4), dtype=torch.int32, device="cuda")
    cnt = torch.zeros((2, 64), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.StemError) as e:
        binding.stem_token_attention(q, kv, kv, idx, cnt, torch.empty_like(q))     # 17 query heads per kv head
    assert e.value.status == binding.STEM_ERR_UNSUPPORTED
