"""GPU parity on the options and edge cases of the path: full budget (dense equivalence), an
explicit k_start, the paper's 4 + 4 forced blocks with the minimum budget of 54, the 1/sqrt(d)
metric scale with beta = 0, sequences shorter than a block, the largest supported block count per
sequence, and budgets whose candidate lists take the long-list code path."""
import numpy as np
import pytest
import torch

from oracle import stem_oracle as so
from paper_2603_06274_b200 import binding, workloads as wl
from paper_2603_06274_b200.binding import StemPlan
from tests._util import check_attention, check_full_path, from_dev_bf16, to_dev

pytestmark = pytest.mark.gpu


def _dev(w):
    data = wl.make_qkv(w)
    return data, to_dev(data["q"]), to_dev(data["k"]), to_dev(data["v"])


def test_full_budget_selects_every_causal_block_and_equals_dense_mode():
    w = wl.small("full_budget", seqlens=(1100, 300), hq=4, hkv=2, block=128, permille=1000, mu_num=1, mu_den=1)
    data, q, k, v = _dev(w)
    idx_g, cnt_g, out = check_full_path(w, data, q, k, v)
    nblk = so.n_blocks(w.seqlens, w.block)
    want = np.concatenate([np.arange(1, nb + 1) for nb in nblk])
    assert np.array_equal(cnt_g, np.broadcast_to(want, cnt_g.shape))      # sel_cnt(r) = r + 1
    plan = StemPlan.from_workload(w)
    dense = torch.empty_like(out)
    binding.stem_sparse_prefill(plan, q, k, v, None, None, dense)
    assert binding.stem_check_status(plan)[0] == 0
    assert torch.equal(out.view(torch.int16), dense.view(torch.int16))     # same blocks, same order, same kernel


def test_explicit_k_start_with_linear_decay():
    w = wl.small("k_start6", seqlens=(4096,), hq=4, hkv=1, block=128, permille=0, k_start_blocks=12, mu_num=1,
                 mu_den=2, stem_blocks=2, local_blocks=1)
    data, q, k, v = _dev(w)
    _, cnt_g, _ = check_full_path(w, data, q, k, v)
    # Eq. 3 with i = r + 1: floor(12 - 6 i / 32) is 6 at i = 32 and 10 at i = 10, the last row the causal cap binds
    assert cnt_g[0, -1] == 6 and cnt_g.max() == 10 and cnt_g[0, 9] == 10 and cnt_g[0, 10] == 9


def test_paper_settings_as_printed_minimum_54_blocks():
    # 4 initial + 4 local blocks, minimum total budget 54: at 80 blocks the minimum dominates the 10 % schedule
    w = wl.small("as_printed", seqlens=(10240,), hq=2, hkv=2, block=128, permille=100, stem_blocks=4, local_blocks=4,
                 min_blocks=54)
    data, q, k, v = _dev(w)
    _, cnt_g, _ = check_full_path(w, data, q, k, v)
    assert cnt_g[0, 53] == 54 and cnt_g[0, 79] == 54 and cnt_g[0, 10] == 11


def test_routing_only_metric_with_softmax_style_scale():
    w = wl.small("sam_scaled", seqlens=(3000,), hq=4, hkv=2, block=64, permille=200, beta=0.0,
                 score_scale=float(1.0 / np.sqrt(128.0)))
    data, q, k, v = _dev(w)
    check_full_path(w, data, q, k, v)


def test_sequences_shorter_than_a_block():
    w = wl.small("tiny_seqs", seqlens=(1, 130, 64, 5), hq=2, hkv=1, block=64, permille=500, heavy_mode="window")
    data, q, k, v = _dev(w)
    check_full_path(w, data, q, k, v)


def test_largest_supported_block_count():
    # 2048 blocks in one sequence (the bitmap width of the selection kernel)
    w = wl.small("max_blocks", seqlens=(2048 * 64,), hq=1, hkv=1, block=64, permille=20, sink=True)
    data, q, k, v = _dev(w)
    check_full_path(w, data, q, k, v, n_random=8)


def test_long_candidate_lists():
    # k_start = 200 blocks: lists of up to 264 entries take the code path that keeps them in shared memory
    w = wl.small("long_lists", seqlens=(400 * 128,), hq=2, hkv=1, block=128, permille=500)
    data, q, k, v = _dev(w)
    check_full_path(w, data, q, k, v, n_random=6)


def test_equal_metrics_are_broken_by_block_id_in_the_fused_path():
    # every K token and every V token of a kv head is the same vector: a row's candidates all have the same
    # metric (also on the GPU: each column of the contraction sees the same operands), so the budget must go to the
    # candidates with the smallest block ids, in the fused path's bit-plane selection kernel too
    w = wl.small("all_ties", seqlens=(6000,), hq=4, hkv=2, block=64, permille=300)
    data = wl.make_qkv(w)
    data["k"][:] = data["k"][0:1]
    data["v"][:] = data["v"][0:1]
    q, k, v = to_dev(data["q"]), to_dev(data["k"]), to_dev(data["v"])
    idx_g, cnt_g, _ = check_full_path(w, data, q, k, v, tie_budget=0)
    r = 80                                                     # 81 causal blocks, 4 + 4 forced
    n = int(cnt_g[1, r])
    want = np.concatenate([np.arange(0, n - w.local_blocks), np.arange(r + 1 - w.local_blocks, r + 1)])
    assert np.array_equal(idx_g[1, r, :n], want)


def test_32k_layer_with_value_elements_of_order_one():
    # the 32K configuration on the value recipe V_t = g_t z_t (elements O(1), outputs ~ sqrt(d) times larger)
    w = wl.CONFIGS["cfg2"].with_(v_recipe="gain_lognormal", name="cfg2_gain_v")
    data, q, k, v = _dev(w)
    check_full_path(w, data, q, k, v, n_random=200)
