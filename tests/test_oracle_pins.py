"""Pins for the CPU checker: each step of Algorithm 1 is compared with something it does not
itself compute - a closed form from the paper, a library routine (numpy / torch in fp64),
brute force on tiny inputs, or an invariant of the definition."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import stem_oracle as so
from paper_2603_06274_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def _golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split()
                out[k] = float(v)
    return out


def _bits(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _rand_bits(rng, shape, scale=1.0):
    return _bits(rng.standard_normal(shape).astype(np.float32) * scale)


# ------------------------------------------------------------------------------------------------
# schedule (Eq. 3, Eq. 2, Eq. 4, ablation identity)
# ------------------------------------------------------------------------------------------------

def test_schedule_endpoints_and_monotone():
    g = _golden()
    mu = g["mu_default"]
    p = so.StemParams(block=128, mu_num=7, mu_den=10, stem_blocks=0, local_blocks=1, min_blocks=0)
    assert abs(p.mu_num / p.mu_den - mu) < 1e-12
    for n_blk, k_s in [(1024, 51), (256, 25), (64, 16), (1000, 333), (7, 3)]:
        kb, ke = so.schedule(n_blk, k_s, p)
        assert np.all(np.diff(kb) <= 0), "budget must not increase with position"
        assert kb[-1] == (7 * k_s) // 10, "k(N) = floor(mu k_start)"
        # first row: k_start minus less than one decay step, floored
        assert kb[0] in (k_s, k_s - 1)
        # independent evaluation of Eq. 3 with exact fractions
        from fractions import Fraction
        for i in (1, 2, n_blk // 3, n_blk // 2, n_blk - 1, n_blk):
            if i < 1:
                continue
            exact = Fraction(k_s) - Fraction(k_s) * (1 - Fraction(7, 10)) / n_blk * i
            assert kb[i - 1] == math.floor(exact)
        assert np.all(ke <= np.arange(1, n_blk + 1))


def test_schedule_no_decay_is_constant():
    p = so.StemParams(block=128, mu_num=1, mu_den=1, stem_blocks=0, local_blocks=1)
    kb, ke = so.schedule(512, 40, p)
    assert np.all(kb == 40)
    assert np.all(ke == np.minimum(np.arange(1, 513), 40))


def test_schedule_token_level_cost_closed_forms():
    """Eq. 2 and Eq. 4: total cost sum_i min(i, k(i)) at token granularity (B = 1)."""
    g = _golden()
    N, k_s = 8192, 2048
    uni = so.StemParams(block=1, mu_num=1, mu_den=1, stem_blocks=0, local_blocks=1)
    _, ke = so.schedule(N, k_s, uni)
    c_uni = int(ke.astype(np.int64).sum())
    eq2 = N * k_s - 0.5 * k_s ** 2
    assert abs(c_uni - eq2) <= N + k_s

    dec = so.StemParams(block=1, mu_num=7, mu_den=10, stem_blocks=0, local_blocks=1)
    kb, ke = so.schedule(N, k_s, dec)
    c_dec = int(ke.astype(np.int64).sum())
    mu = 0.7
    eq4 = N * k_s - 0.5 * k_s ** 2 - 0.5 * k_s * (1 - mu) * (N - k_s)
    # Eq. 4 is stated as an approximation: it ignores the decay inside the causal triangle.
    assert abs(c_dec - eq4) <= 0.5 * k_s ** 2 * (1 - mu) + 2 * N
    # exact continuous form: area under min(i, k(i)), crossing point i* = k_s / (1 + (1-mu) k_s / N)
    i_star = k_s / (1 + (1 - mu) * k_s / N)
    exact = N * k_s * (1 + mu) / 2 - 0.5 * k_s * i_star
    assert abs(c_dec - exact) / exact < 2e-3
    # average budget ratio printed in the ablation section
    assert abs(kb.astype(np.float64).sum() / (N * k_s) - g["k_uni_over_k_start"]) < 1e-3


def test_schedule_forced_and_min_blocks():
    g = _golden()
    p = so.StemParams(block=128, stem_blocks=int(g["stem_blocks"]), local_blocks=int(g["local_blocks"]),
                      min_blocks=int(g["min_blocks"]))
    n_blk = 1024
    k_s = int(g["k_start_frac_long"] * n_blk)
    kb, ke = so.schedule(n_blk, k_s, p)
    i = np.arange(1, n_blk + 1)
    assert np.all(ke == np.minimum(i, np.maximum(kb, 54)))
    # tiny budget: the forced blocks alone set the row size
    p2 = so.StemParams(block=128, stem_blocks=4, local_blocks=2, min_blocks=0)
    _, ke2 = so.schedule(64, 1, p2)
    assert np.all(ke2 == np.minimum(i[:64], 6))


def test_config_schedule_values():
    """Per-config initial budgets and last-row budgets (floor(permille N_blk / 1000), floor(0.7 k_s))."""
    expect = {"cfg1": (64, 16, 11), "cfg2": (256, 25, 17), "cfg3": (1024, 51, 35)}
    for name, (n_blk, k_s, last) in expect.items():
        w = wl.CONFIGS[name]
        p = so.StemParams(block=w.block, budget_permille=w.budget_permille, stem_blocks=w.stem_blocks,
                          local_blocks=w.local_blocks, min_blocks=w.min_blocks)
        nb = int(so.n_blocks(w.seqlens, w.block)[0])
        assert nb == n_blk and so.k_start(nb, p) == k_s
        kb, ke = so.schedule(nb, k_s, p)
        assert kb[-1] == last
    # retained / admissible ratio of cfg 1 and cfg 3 (block counts derived by hand from the schedule)
    w = wl.CONFIGS["cfg1"]
    p = so.StemParams(block=64, budget_permille=250)
    _, ke = so.schedule(64, 16, p)
    assert int(ke.sum()) == 732 and 64 * 65 // 2 == 2080


# ------------------------------------------------------------------------------------------------
# pooling and magnitude
# ------------------------------------------------------------------------------------------------

def test_pooled_dot_is_mean_of_token_dots():
    rng = np.random.default_rng(1)
    B, T, d = 8, 44, 16  # last block partial (4 tokens)
    q = _rand_bits(rng, (T, 2, d))
    k = _rand_bits(rng, (T, 1, d))
    cu = np.array([0, T], np.int32)
    qbar = so.pool_mean(q, cu, B).astype(np.float64)
    kbar = so.pool_mean(k, cu, B).astype(np.float64)
    qf = wl.bf16_bits_to_f32(q).astype(np.float64)
    kf = wl.bf16_bits_to_f32(k).astype(np.float64)
    tok = np.einsum("thc,sc->hts", qf, kf[:, 0])  # all token dot products
    n_blk = (T + B - 1) // B
    for h in range(2):
        for r in range(n_blk):
            for j in range(n_blk):
                blk = tok[h, r * B:(r + 1) * B, j * B:(j + 1) * B]
                assert abs(qbar[h, r] @ kbar[0, j] - blk.mean()) < 1e-5
    # invariance to a permutation of the tokens inside a key block
    perm = np.arange(T)
    perm[8:16] = perm[8:16][::-1]
    kbar_p = so.pool_mean(np.ascontiguousarray(k[perm]), cu, B)
    np.testing.assert_allclose(kbar_p, kbar, atol=1e-6)


def test_pool_varlen_sequences_do_not_mix():
    rng = np.random.default_rng(2)
    B, d = 8, 16
    a = _rand_bits(rng, (20, 1, d))
    b = _rand_bits(rng, (13, 1, d))
    both = np.concatenate([a, b])
    cu = np.array([0, 20, 33], np.int32)
    pooled = so.pool_mean(both, cu, B)
    pa = so.pool_mean(a, np.array([0, 20], np.int32), B)
    pb = so.pool_mean(b, np.array([0, 13], np.int32), B)
    np.testing.assert_array_equal(pooled, np.concatenate([pa, pb], axis=1))


def test_value_magnitude_closed_form():
    rng = np.random.default_rng(3)
    B, T, d = 8, 30, 16
    v = _rand_bits(rng, (T, 2, d), scale=0.5)
    v[8:16] = 0  # a block of zero vectors: ln 0 -> clamp to 0
    cu = np.array([0, T], np.int32)
    mv = so.value_magnitude(v, cu, B)
    vf = wl.bf16_bits_to_f32(v).astype(np.float64)
    ss = (vf ** 2).sum(-1)  # [T, H]
    for h in range(2):
        for j in range(4):
            m2 = ss[j * B:(j + 1) * B, h].max()
            closed = 0.5 * math.log(max(1.0, m2))
            assert abs(mv[h, j] - closed) < 1e-6
    assert mv[0, 1] == 0.0 and mv[1, 1] == 0.0
    # small-norm vectors exercise the clamp
    tiny = _rand_bits(rng, (16, 1, d), scale=0.01)
    assert np.all(so.value_magnitude(tiny, np.array([0, 16], np.int32), B) == 0.0)


# ------------------------------------------------------------------------------------------------
# metric (Eq. 7)
# ------------------------------------------------------------------------------------------------

def _np_metric(qbar, kbar, mv, beta, scale=1.0):
    hq, hkv = qbar.shape[0], kbar.shape[0]
    g = hq // hkv
    out = np.empty((hq, qbar.shape[1], kbar.shape[1]))
    for h in range(hq):
        out[h] = scale * (qbar[h].astype(np.float64) @ kbar[h // g].astype(np.float64).T) + beta * mv[h // g][None, :]
    return out


def test_metric_matches_matmul_and_gqa_mapping():
    rng = np.random.default_rng(4)
    hq, hkv, nb, d = 4, 2, 9, 16
    qbar = rng.standard_normal((hq, nb, d)).astype(np.float32)
    kbar = rng.standard_normal((hkv, nb, d)).astype(np.float32)
    mv = np.abs(rng.standard_normal((hkv, nb))).astype(np.float32)
    for beta, scale in [(0.2, 1.0), (0.0, 1.0), (0.5, 1 / math.sqrt(d))]:
        M = so.metric(qbar, kbar, mv, np.array([nb]), beta, scale).reshape(hq, nb, nb)
        ref = _np_metric(qbar, kbar, mv, beta, scale)
        tri = np.tril(np.ones((nb, nb), bool))
        np.testing.assert_allclose(M[:, tri], ref[:, tri], rtol=0, atol=2e-6)
        assert np.all(np.isnan(M[:, ~tri])), "blocks above the diagonal are not candidates"
    # beta = 0 is the pure routing score
    M0 = so.metric(qbar, kbar, mv, np.array([nb]), 0.0).reshape(hq, nb, nb)
    np.testing.assert_allclose(M0[0, 5, :6], qbar[0, 5].astype(np.float64) @ kbar[0, :6].astype(np.float64).T, atol=2e-6)


def test_metric_rotation_invariance():
    rng = np.random.default_rng(5)
    hq, nb, d = 2, 12, 32
    qbar = rng.standard_normal((hq, nb, d)).astype(np.float32)
    kbar = rng.standard_normal((hq, nb, d)).astype(np.float32)
    mv = np.abs(rng.standard_normal((hq, nb))).astype(np.float32)
    rot, _ = np.linalg.qr(rng.standard_normal((d, d)))
    M1 = so.metric(qbar, kbar, mv, np.array([nb]), 0.2)
    M2 = so.metric((qbar @ rot).astype(np.float32), (kbar @ rot).astype(np.float32), mv, np.array([nb]), 0.2)
    ok = ~np.isnan(M1)
    np.testing.assert_allclose(M1[ok], M2[ok], atol=2e-5)


def test_metric_varlen_layout():
    rng = np.random.default_rng(6)
    d = 8
    nblk = np.array([3, 5], np.int32)
    qbar = rng.standard_normal((2, 8, d)).astype(np.float32)
    kbar = rng.standard_normal((1, 8, d)).astype(np.float32)
    mv = np.zeros((1, 8), np.float32)
    M = so.metric(qbar, kbar, mv, nblk, 0.0)
    assert M.shape == (2, 9 + 25)
    second = M[:, 9:].reshape(2, 5, 5)
    # row 2 of the second sequence against its own block 1 (global row 3+2, global block 3+1)
    assert abs(second[1, 2, 1] - float(qbar[1, 5].astype(np.float64) @ kbar[0, 4].astype(np.float64))) < 2e-6


# ------------------------------------------------------------------------------------------------
# selection
# ------------------------------------------------------------------------------------------------

def _brute_select(Mrow, r, k_eff, stem, local):
    i = r + 1
    forced = set(range(min(stem, i))) | set(range(max(0, i - local), i))
    cand = [j for j in range(i) if j not in forced]
    vals = []
    for j in cand:
        m = float(Mrow[j])
        if math.isnan(m):
            m = -math.inf
        if m == 0.0:
            m = 0.0
        vals.append(m)
    order = sorted(range(len(cand)), key=lambda q: (-vals[q], cand[q]))
    need = max(0, min(k_eff - len(forced), len(cand)))
    return sorted(forced | {cand[q] for q in order[:need]})


@pytest.mark.parametrize("ties", [False, True])
def test_select_matches_brute_force_sort(ties):
    nb, heads = 40, 3
    M = wl.make_scores(77, heads, nb, ties=ties)
    if ties:
        M[0, 30, 7] = np.nan
    p = so.StemParams(block=128, budget_permille=250, stem_blocks=2, local_blocks=3)
    _, ke = so.schedule(nb, so.k_start(nb, p), p)
    idx, cnt = so.select(M.reshape(heads, -1), np.array([nb]), ke, 2, 3)
    for h in range(heads):
        for r in range(nb):
            want = _brute_select(M[h, r], r, int(ke[r]), 2, 3)
            got = idx[h, r, :cnt[h, r]].tolist()
            assert got == want, (h, r)
            assert np.all(idx[h, r, cnt[h, r]:] == -1)


def test_select_full_budget_and_forced_blocks():
    nb, heads = 33, 2
    M = wl.make_scores(5, heads, nb)
    full = so.StemParams(block=128, budget_permille=1000, mu_num=1, mu_den=1)  # k(i) = N_blk for every row
    _, ke = so.schedule(nb, so.k_start(nb, full), full)
    idx, cnt = so.select(M.reshape(heads, -1), np.array([nb]), ke, 4, 4)
    for r in range(nb):
        assert cnt[0, r] == r + 1 and idx[0, r, :r + 1].tolist() == list(range(r + 1))
    p = so.StemParams(block=128, budget_permille=300, stem_blocks=4, local_blocks=2)
    _, ke = so.schedule(nb, so.k_start(nb, p), p)
    idx, cnt = so.select(M.reshape(heads, -1), np.array([nb]), ke, 4, 2)
    assert np.array_equal(cnt[0], ke) and np.array_equal(cnt[1], ke)
    for r in range(nb):
        row = set(idx[1, r, :cnt[1, r]].tolist())
        assert r in row and max(0, r - 1) in row
        assert set(range(min(4, r + 1))) <= row
        assert all(0 <= j <= r for j in row)
    retained = cnt[0].sum() / sum(r + 1 for r in range(nb))
    assert 0 < retained < 1


def test_metric_rank_equivalence_with_output_contribution():
    """Appendix A.1: ranking by exp(s) * ||v|| equals ranking by s + ln ||v|| (beta = 1, clamp inactive)."""
    rng = np.random.default_rng(8)
    nb, d = 24, 8
    qbar = (rng.standard_normal((1, nb, d)) * 0.5).astype(np.float32)
    kbar = (rng.standard_normal((1, nb, d)) * 0.5).astype(np.float32)
    norms = np.exp(rng.uniform(0.1, 2.0, size=(1, nb)))  # all > 1
    mv = np.log(norms).astype(np.float32)
    M = so.metric(qbar, kbar, mv, np.array([nb]), 1.0).reshape(1, nb, nb)
    ke = np.minimum(np.arange(1, nb + 1), 6).astype(np.int32)
    idx, cnt = so.select(M.reshape(1, -1), np.array([nb]), ke, 0, 1)
    contrib = np.exp(qbar[0].astype(np.float64) @ kbar[0].astype(np.float64).T) * norms[0][None, :]
    for r in range(nb):
        cand = np.arange(r)  # diagonal is forced
        need = int(ke[r]) - 1
        top = set(cand[np.argsort(-contrib[r, :r], kind="stable")[:need]].tolist()) | {r}
        assert set(idx[0, r, :cnt[0, r]].tolist()) == top


def test_value_scaling_leaves_selection_unchanged():
    rng = np.random.default_rng(9)
    T, B, d = 256, 16, 16
    q = _rand_bits(rng, (T, 2, d))
    k = _rand_bits(rng, (T, 1, d))
    v1 = rng.standard_normal((T, 1, d)).astype(np.float32) * 2.0  # norms well above 1
    cu = np.array([0, T], np.int32)
    p = so.StemParams(block=B, budget_permille=400, stem_blocks=1, local_blocks=1)
    r1 = so.prefill(q, k, _bits(v1), cu, p, rows=np.zeros((0, 2), np.int32))
    r2 = so.prefill(q, k, _bits(v1 * 4.0), cu, p, rows=np.zeros((0, 2), np.int32))  # exact power of two
    assert np.array_equal(r1["sel_idx"], r2["sel_idx"])
    np.testing.assert_allclose(r2["mv"] - r1["mv"], math.log(4.0), atol=1e-6)


# ------------------------------------------------------------------------------------------------
# attention
# ------------------------------------------------------------------------------------------------

def _torch_masked_attention(q, k, v, allowed, scale):
    """fp64 softmax attention with an explicit boolean mask [H, T, T] (library routine)."""
    qf = torch.from_numpy(wl.bf16_bits_to_f32(q).astype(np.float64)).permute(1, 0, 2)
    g = q.shape[1] // k.shape[1]
    kf = torch.from_numpy(wl.bf16_bits_to_f32(k).astype(np.float64)).permute(1, 0, 2).repeat_interleave(g, 0)
    vf = torch.from_numpy(wl.bf16_bits_to_f32(v).astype(np.float64)).permute(1, 0, 2).repeat_interleave(g, 0)
    s = torch.einsum("htd,hsd->hts", qf, kf) * scale
    s = s.masked_fill(~torch.from_numpy(allowed), -math.inf)
    p = torch.softmax(s, dim=-1)
    o = torch.einsum("hts,hsd->htd", p, vf).permute(1, 0, 2)
    lse = torch.logsumexp(s, dim=-1)
    return o.numpy(), lse.numpy()


def test_full_lists_reproduce_dense_causal_attention():
    rng = np.random.default_rng(10)
    T, B, d, hq, hkv = 150, 16, 32, 4, 2  # partial last block
    q, k, v = _rand_bits(rng, (T, hq, d)), _rand_bits(rng, (T, hkv, d)), _rand_bits(rng, (T, hkv, d))
    cu = np.array([0, T], np.int32)
    idx, cnt = so.dense_lists([T], B, hq)
    O, lse = so.attention(q, k, v, cu, B, idx, cnt)
    qf = torch.from_numpy(wl.bf16_bits_to_f32(q).astype(np.float64)).permute(1, 0, 2)[None]
    kf = torch.from_numpy(wl.bf16_bits_to_f32(k).astype(np.float64)).permute(1, 0, 2)[None].repeat_interleave(2, 1)
    vf = torch.from_numpy(wl.bf16_bits_to_f32(v).astype(np.float64)).permute(1, 0, 2)[None].repeat_interleave(2, 1)
    ref = torch.nn.functional.scaled_dot_product_attention(qf, kf, vf, is_causal=True)[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(O, ref, atol=2e-6)
    allowed = np.tril(np.ones((T, T), bool))[None].repeat(hq, 0)
    _, lse_ref = _torch_masked_attention(q, k, v, allowed, 1 / math.sqrt(d))
    np.testing.assert_allclose(lse, lse_ref, atol=2e-5)


def test_sparse_lists_match_explicit_mask_and_varlen():
    rng = np.random.default_rng(11)
    B, d, hq, hkv = 8, 16, 2, 1
    seqlens = [37, 22]
    T = sum(seqlens)
    q, k, v = _rand_bits(rng, (T, hq, d)), _rand_bits(rng, (T, hkv, d)), _rand_bits(rng, (T, hkv, d))
    cu = np.array([0, 37, 59], np.int32)
    p = so.StemParams(block=B, budget_permille=500, stem_blocks=1, local_blocks=1)
    res = so.prefill(q, k, v, cu, p)
    idx, cnt = res["sel_idx"], res["sel_cnt"]
    allowed = np.zeros((hq, T, T), bool)
    row = 0
    for b, n in enumerate(seqlens):
        t0 = cu[b]
        for r in range((n + B - 1) // B):
            for h in range(hq):
                for j in idx[h, row, :cnt[h, row]]:
                    for tq in range(r * B, min(n, (r + 1) * B)):
                        for tk in range(j * B, min(n, (j + 1) * B)):
                            if tk <= tq:
                                allowed[h, t0 + tq, t0 + tk] = True
            row += 1
    ref, lse_ref = _torch_masked_attention(q, k, v, allowed, 1 / math.sqrt(d))
    np.testing.assert_allclose(res["O"], ref, atol=2e-6)
    np.testing.assert_allclose(res["lse"], lse_ref, atol=2e-5)
    # rows inside the causal triangle are dense rows
    assert cnt[0, 0] == 1 and cnt[0, 1] == 2


def test_single_diagonal_block_is_local_causal_attention():
    rng = np.random.default_rng(12)
    T, B, d = 32, 8, 16
    q, k, v = _rand_bits(rng, (T, 1, d)), _rand_bits(rng, (T, 1, d)), _rand_bits(rng, (T, 1, d))
    cu = np.array([0, T], np.int32)
    idx = np.arange(4, dtype=np.int32).reshape(1, 4, 1)
    cnt = np.ones((1, 4), np.int32)
    O, _ = so.attention(q, k, v, cu, B, idx, cnt)
    for r in range(4):
        sl = slice(r * B, (r + 1) * B)
        allowed = np.tril(np.ones((B, B), bool))[None]
        ref, _ = _torch_masked_attention(q[sl], k[sl], v[sl], allowed, 1 / math.sqrt(d))
        np.testing.assert_allclose(O[sl], ref, atol=2e-6)


def test_row_subset_only_touches_requested_rows():
    rng = np.random.default_rng(13)
    T, B, d = 64, 16, 16
    q, k, v = _rand_bits(rng, (T, 2, d)), _rand_bits(rng, (T, 2, d)), _rand_bits(rng, (T, 2, d))
    cu = np.array([0, T], np.int32)
    idx, cnt = so.dense_lists([T], B, 2)
    full, _ = so.attention(q, k, v, cu, B, idx, cnt)
    part, _ = so.attention(q, k, v, cu, B, idx, cnt, rows=np.array([[1, 2]], np.int32))
    np.testing.assert_array_equal(part[32:48, 1], full[32:48, 1])
    assert np.all(np.isnan(part[:32])) and np.all(np.isnan(part[32:48, 0]))
