"""The failure-reporting path of the library, exercised without making any production kernel fail.

A bounded device-side wait that gives up records a code in the status words at the start of the
workspace; stem_check_status turns it into STEM_ERR_DEVICE_TIMEOUT, hands out the detail words and
clears them.  Two forms: (i) the words are written from the host, as the attention kernel and the
metric kernel would write them; (ii) the library's self-test kernel really waits (1 ms limit) on a
barrier nothing arrives at, with the routine the production kernels wait with, and records the
time-out itself.  Neither hangs, traps or faults; the context stays usable, which the tests check
by running the real path afterwards and comparing bit for bit."""
import pytest
import torch

from paper_2603_06274_b200 import binding, workloads as wl
from paper_2603_06274_b200.binding import StemPlan
from tests._util import to_dev

pytestmark = pytest.mark.gpu


def _setup():
    w = wl.small("status", seqlens=(1500, 300), hq=4, hkv=2, block=128, permille=300)
    data = wl.make_qkv(w)
    plan = StemPlan.from_workload(w)
    q, k, v = to_dev(data["q"]), to_dev(data["k"]), to_dev(data["v"])
    out = torch.empty((w.total_tokens, w.num_q_heads, 128), dtype=torch.bfloat16, device="cuda")
    return w, plan, q, k, v, out


def _run(plan, q, k, v, out):
    info = plan.info
    idx = torch.empty((plan.num_q_heads, info.total_q_blocks, info.k_max), dtype=torch.int32, device="cuda")
    cnt = torch.empty((plan.num_q_heads, info.total_q_blocks), dtype=torch.int32, device="cuda")
    binding.stem_prefill(plan, q, k, v, out, idx, cnt)
    return idx, cnt


def test_status_words_written_by_the_host_are_reported_and_cleared():
    w, plan, q, k, v, out = _setup()
    words = binding.status_words(plan)
    assert binding.stem_check_status(plan) == (binding.STEM_OK, [0, 0, 0, 0])
    # as the attention kernel records a wait that gave up: {1, CTA, role, barrier}
    words.copy_(torch.tensor([1, 37, 3, 6, 0, 0, 0, 0], dtype=torch.int32))
    st, detail = binding.stem_check_status(plan)
    assert st == binding.STEM_ERR_DEVICE_TIMEOUT and detail == [1, 37, 3, 6]
    assert int(words.abs().sum()) == 0
    assert binding.stem_check_status(plan) == (binding.STEM_OK, [0, 0, 0, 0])
    # as the metric kernel records one: words 4..6 = {2, tile, kv head}
    words.copy_(torch.tensor([0, 0, 0, 0, 2, 11, 1, 0], dtype=torch.int32))
    st, detail = binding.stem_check_status(plan)
    assert st == binding.STEM_ERR_DEVICE_TIMEOUT and detail == [2, 11, 1, 0]
    assert int(words.abs().sum()) == 0


def test_a_metric_kernel_record_survives_the_attention_launch():
    # stem_prefill enqueues scoring, then attention: the attention launch must not wipe words 4..6
    w, plan, q, k, v, out = _setup()
    _run(plan, q, k, v, out)
    assert binding.stem_check_status(plan)[0] == binding.STEM_OK
    words = binding.status_words(plan)
    words[4:7] = torch.tensor([2, 5, 0], dtype=torch.int32, device="cuda")
    binding.stem_sparse_prefill(plan, q, k, v, None, None, out)     # clears only the attention kernel's words
    st, detail = binding.stem_check_status(plan)
    assert st == binding.STEM_ERR_DEVICE_TIMEOUT and detail == [2, 5, 0, 0]


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    w, plan, q, k, v, out = _setup()
    _run(plan, q, k, v, out)
    assert binding.stem_check_status(plan)[0] == binding.STEM_OK
    before = out.clone()
    binding.stem_selftest_wait_timeout(plan)
    st, detail = binding.stem_check_status(plan)
    assert st == binding.STEM_ERR_DEVICE_TIMEOUT and detail == [1, 0, 99, 0]
    assert binding.stem_check_status(plan)[0] == binding.STEM_OK       # cleared
    out.fill_(float("nan"))
    _run(plan, q, k, v, out)
    assert binding.stem_check_status(plan)[0] == binding.STEM_OK
    assert torch.equal(out.view(torch.int16), before.view(torch.int16))
