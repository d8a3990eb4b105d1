"""Pins of the CPU checker's chunked-prefill and group-shared-selection functions (no GPU).

Chunked prefill (the paper's Conclusion: the position-decay schedule carries over to chunked prefill when
global token offsets are kept): a row of a chunk depends only on its own queries and on the K / V blocks
before it, so any split of the sequences into block-aligned chunks must reproduce the one-shot result row
by row - lists bit for bit, outputs to rounding - provided the budget is evaluated at the GLOBAL row of the
full sequence.  The chunk functions are separate code from the one-shot functions (which are pinned to the
paper in test_oracle_pins.py), so this comparison pins them.  The log-sum-exp output is pinned by the
exactness of merging attention over disjoint key partitions."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import stem_oracle as so
from paper_2603_06274_b200 import workloads as wl
from tests._util import oracle_params


def _one_shot(w):
    data = wl.make_qkv(w)
    p = oracle_params(w)
    return data, p, so.prefill(data["q"], data["k"], data["v"], data["cu_seqlens"], p)


@pytest.mark.parametrize("w,splits", [
    (wl.small("chunks_b128", seqlens=(1500, 900), hq=4, hkv=2, block=128, permille=400, sink=True),
     [(0, 512, 1024, 1500), (0, 256, 640, 900)]),
    (wl.small("chunks_b64", seqlens=(1000,), hq=2, hkv=1, block=64, permille=250, stem_blocks=2, local_blocks=3,
              mu_num=1, mu_den=2),
     [(0, 64, 704, 1000)]),
])
def test_chunks_reproduce_the_one_shot_result(w, splits):
    data, p, ref = _one_shot(w)
    cu = data["cu_seqlens"]
    B = w.block
    nblk = so.n_blocks(w.seqlens, B)
    row_off = np.concatenate([[0], np.cumsum(nblk)])
    n_chunks = len(splits[0]) - 1
    for c in range(n_chunks):
        q_starts = [s[c] for s in splits]
        kv_lens = [s[c + 1] for s in splits]
        q = np.concatenate([data["q"][cu[b] + q_starts[b]:cu[b] + kv_lens[b]] for b in range(len(splits))])
        k = np.concatenate([data["k"][cu[b]:cu[b] + kv_lens[b]] for b in range(len(splits))])
        v = np.concatenate([data["v"][cu[b]:cu[b] + kv_lens[b]] for b in range(len(splits))])
        cu_q = np.concatenate([[0], np.cumsum([kv_lens[b] - q_starts[b] for b in range(len(splits))])]).astype(np.int32)
        cu_kv = np.concatenate([[0], np.cumsum(kv_lens)]).astype(np.int32)
        got = so.prefill_chunk(q, k, v, cu_q, cu_kv, q_starts, w.seqlens, p)
        rq = 0
        for b in range(len(splits)):
            r_lo, r_hi = q_starts[b] // B, -(-kv_lens[b] // B)
            # a chunk that ends inside a block sees a partial last block: only its full rows are comparable,
            # unless the chunk ends where the sequence ends
            full_hi = r_hi if kv_lens[b] == w.seqlens[b] or kv_lens[b] % B == 0 else r_hi - 1
            for r in range(r_lo, full_hi):
                R, RQ = row_off[b] + r, rq + (r - r_lo)
                assert np.array_equal(got["sel_cnt"][:, RQ], ref["sel_cnt"][:, R])
                n = ref["sel_cnt"][:, R].max()
                assert np.array_equal(got["sel_idx"][:, RQ, :n], ref["sel_idx"][:, R, :n])
                t_ref = slice(cu[b] + r * B, cu[b] + min((r + 1) * B, w.seqlens[b]))
                t_got = slice(cu_q[b] + (r - r_lo) * B, cu_q[b] + min((r - r_lo + 1) * B, kv_lens[b] - q_starts[b]))
                assert np.abs(got["O"][t_got] - ref["O"][t_ref]).max() <= 1e-6
                assert np.abs(got["lse"][:, t_got] - ref["lse"][:, t_ref]).max() <= 1e-6
            rq += r_hi - r_lo


def test_chunk_budget_is_eq3_at_the_global_row_of_the_full_sequence():
    p = so.StemParams(block=128, budget_permille=100, mu_num=7, mu_den=10, stem_blocks=0, local_blocks=1, min_blocks=0)
    total, q_start, kv_len = 128 * 300, 128 * 100, 128 * 180
    ke = so.schedule_chunk([kv_len], [q_start], [total], p)
    assert len(ke) == 80
    n_tot, k_s = 300, 30
    for local_row, got in enumerate(ke):
        i = 100 + local_row + 1                                           # 1-indexed global block row
        want = int(Fraction(k_s) - Fraction(k_s) * Fraction(3, 10) * Fraction(i, n_tot))  # floor of Eq. 3
        assert got == max(1, min(i, want))
    # evaluating the schedule on the prefix length instead would give another k_start and another slope
    wrong = so.schedule(180, so.k_start(180, p), p)[1][100:180]
    assert not np.array_equal(ke, wrong)


def test_merging_key_partitions_by_log_sum_exp_is_exact():
    w = wl.small("lse_merge", seqlens=(900, 300), hq=4, hkv=2, block=128, permille=500, v_recipe="gain_lognormal")
    data, p, ref = _one_shot(w)
    idx, cnt = ref["sel_idx"], ref["sel_cnt"]
    k_max = idx.shape[2]
    parts = []
    for part in range(2):
        # the entries of every list in even / odd positions; some rows get an empty list in one partition
        pi = np.full_like(idx, -1)
        pc = np.zeros_like(cnt)
        for h in range(idx.shape[0]):
            for R in range(idx.shape[1]):
                ent = idx[h, R, :cnt[h, R]][part::2]
                pi[h, R, :len(ent)] = ent
                pc[h, R] = len(ent)
        O, lse = so.attention(data["q"], data["k"], data["v"], data["cu_seqlens"], w.block, pi, pc)
        parts.append((O, lse))
    assert np.isneginf(parts[1][1]).any(), "rows with a single block leave the second partition empty"
    O, lse = so.merge_partitions([x[0] for x in parts], [x[1] for x in parts])
    assert np.abs(O - ref["O"]).max() <= 1e-5 * max(1.0, np.abs(ref["O"]).max())
    assert np.abs(lse - ref["lse"]).max() <= 1e-5


def test_group_metric_is_the_mean_of_the_heads_metrics():
    w = wl.small("shared", seqlens=(1300, 260), hq=6, hkv=2, block=128, permille=300, sink=True)
    data = wl.make_qkv(w)
    p = oracle_params(w)
    M, qbar, kbar, mv = so.score(data["q"], data["k"], data["v"], data["cu_seqlens"], p)
    nblk = so.n_blocks(w.seqlens, w.block)
    Mg = so.metric_shared(qbar, kbar, mv, nblk, p.beta, p.score_scale)
    g = w.num_q_heads // w.num_kv_heads
    # (a) numpy fp64: per-head Eq. 7, then the mean over the group's heads
    row_off = np.concatenate([[0], np.cumsum(nblk)])
    off = 0
    for b, nb in enumerate(nblk):
        nb = int(nb)
        for kvh in range(w.num_kv_heads):
            heads = []
            for q in range(g):
                qb = qbar[kvh * g + q, row_off[b]:row_off[b] + nb].astype(np.float64)
                kb = kbar[kvh, row_off[b]:row_off[b] + nb].astype(np.float64)
                heads.append(p.score_scale * qb @ kb.T + p.beta * mv[kvh, row_off[b]:row_off[b] + nb].astype(np.float64)[None, :])
            want = np.mean(heads, axis=0)
            got = Mg[kvh, off:off + nb * nb].reshape(nb, nb)
            tri = np.tril(np.ones((nb, nb), dtype=bool))
            assert np.isnan(got[~tri]).all()
            assert np.abs(got[tri] - want[tri]).max() <= 1e-6 * max(1.0, np.abs(want[tri]).max())
            # (b) the same as Eq. 7 on the group-mean pooled query
            qmean = np.mean([qbar[kvh * g + q, row_off[b]:row_off[b] + nb].astype(np.float64) for q in range(g)], axis=0)
            alt = p.score_scale * qmean @ kbar[kvh, row_off[b]:row_off[b] + nb].astype(np.float64).T \
                + p.beta * mv[kvh, row_off[b]:row_off[b] + nb].astype(np.float64)[None, :]
            assert np.abs(alt[tri] - want[tri]).max() <= 1e-9 * max(1.0, np.abs(want[tri]).max())
        off += nb * nb
    # with one head per group the shared metric is the per-head metric
    w1 = wl.small("shared_mha", seqlens=(700,), hq=2, hkv=2, block=64, permille=300)
    d1 = wl.make_qkv(w1)
    p1 = oracle_params(w1)
    M1, qb1, kb1, mv1 = so.score(d1["q"], d1["k"], d1["v"], d1["cu_seqlens"], p1)
    Mg1 = so.metric_shared(qb1, kb1, mv1, so.n_blocks(w1.seqlens, 64), p1.beta, p1.score_scale)
    assert np.array_equal(np.nan_to_num(M1, nan=-7.0), np.nan_to_num(Mg1, nan=-7.0))


def test_antidiagonal_metric_is_the_mean_of_the_blocks_main_antidiagonal():
    """Anti-diagonal scoring mode (Overall Algorithm; Alg. 1 step 1 comment, stride = B): pinned against the
    anti-diagonal of a numpy fp64 score matrix, and on inputs whose anti-diagonal sums have a closed form."""
    w = wl.small("antidiag", seqlens=(700, 200), hq=4, hkv=2, block=64, permille=300)
    data = wl.make_qkv(w)
    p = oracle_params(w)
    M, mv = so.score_antidiag(data["q"], data["k"], data["v"], data["cu_seqlens"], p)
    B, cu, g = w.block, data["cu_seqlens"], 2
    q = wl.bf16_bits_to_f32(data["q"]).astype(np.float64)
    k = wl.bf16_bits_to_f32(data["k"]).astype(np.float64)
    nblk = so.n_blocks(w.seqlens, B)
    row_off = np.concatenate([[0], np.cumsum(nblk)])
    off = 0
    for b, nb in enumerate(nblk):
        nb, n = int(nb), w.seqlens[b]
        for h in range(w.num_q_heads):
            S = q[cu[b]:cu[b + 1], h] @ k[cu[b]:cu[b + 1], h // g].T          # every token score of the sequence
            Sp = np.full((nb * B, nb * B), np.nan)
            Sp[:n, :n] = S
            got = M[h, off:off + nb * nb].reshape(nb, nb)
            for r in range(nb):
                for j in range(r + 1):
                    blk = Sp[r * B:(r + 1) * B, j * B:(j + 1) * B]
                    anti = np.array([blk[B - 1 - s, s] for s in range(B)])     # main anti-diagonal
                    a = np.nanmean(anti) if np.isfinite(anti).any() else 0.0  # no existing pair: the term is 0
                    want = p.score_scale * a + p.beta * mv[h // g, row_off[b] + j]
                    assert abs(got[r, j] - want) <= 1e-6 * max(1.0, abs(want))
                assert np.isnan(got[r, r + 1:]).all()
        off += nb * nb
    # closed form: q_t = a_t * u, k_t = c_t * u with |u| = 1  =>  the anti-diagonal mean of block (r, j) is
    # mean_s a[rB + B-1-s] * c[jB + s]; with a_t = t + 1 and c_t = 1 that is the mean position of the query block
    n, B, d = 256, 64, 128
    u = np.zeros(d, np.float32); u[3] = 1.0
    qf = (np.arange(1, n + 1, dtype=np.float32)[:, None] * u[None, :])[:, None, :]
    kf = np.broadcast_to(u, (n, 1, d)).astype(np.float32)
    vf = np.zeros((n, 1, d), np.float32)
    cu1 = np.array([0, n], np.int32)
    mv0 = so.value_magnitude(wl.f32_to_bf16_bits(vf), cu1, B)
    M2 = so.metric_antidiag(wl.f32_to_bf16_bits(qf), wl.f32_to_bf16_bits(kf), mv0, cu1, B, beta=0.2).reshape(4, 4)
    for r in range(4):
        assert np.allclose(M2[r, :r + 1], r * B + (B + 1) / 2.0)
