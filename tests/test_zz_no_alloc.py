"""The allocation-free scoring entry point (stem_score_static), checked against stem_score and the
CPU checker.

Some users of the library run where device memory cannot be requested: inside a serving engine
whose pool already owns the GPU, or in callbacks where the host framework forbids allocator
calls.  For them the library keeps the pooled tensors of the scoring stage in a fixed array of
its own.  This file is collected last on purpose, so that a failure here cannot hide the result
of any other test in a run that stops at the first failure."""
import gc

import numpy as np
import pytest
import torch

from oracle import stem_oracle as so
from paper_2603_06274_b200 import binding, workloads as wl
from paper_2603_06274_b200.binding import StemPlan
from tests._util import oracle_params, to_dev

pytestmark = pytest.mark.gpu


def _allocation_requests() -> int:
    """How many blocks torch's CUDA allocator has handed out since the process started."""
    return int(torch.cuda.memory_stats().get("allocation.all.allocated", 0))


def _metric_triple(w):
    """M of the workload from stem_score (caller workspace), stem_score_static and the checker."""
    _first_call_set_up()
    data = wl.make_qkv(w)
    plan = StemPlan.from_workload(w)
    q, k, v = to_dev(data["q"]), to_dev(data["k"]), to_dev(data["v"])
    n = plan.info.metric_elems
    want = torch.full((w.num_q_heads, n), float("nan"), dtype=torch.float32, device="cuda")
    got = torch.full((w.num_q_heads, n), float("nan"), dtype=torch.float32, device="cuda")
    binding.stem_score(plan, q, k, v, want)          # existing entry point, caller workspace
    torch.cuda.synchronize()
    # the call under test must not request device memory: neither through torch's allocator nor from the driver.
    # (Counted as allocation requests, not as bytes in use: tensors left behind by earlier tests may be released by
    # Python's collector at any moment, which lowers the bytes in use without anybody having asked for memory.)
    gc.collect()
    torch.cuda.synchronize()
    torch_before = (_allocation_requests(), torch.cuda.memory_reserved())
    free_before, _ = torch.cuda.mem_get_info()
    binding.stem_score_static(plan, q, k, v, got)    # same stage, library-owned scratch
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert (_allocation_requests(), torch.cuda.memory_reserved()) == torch_before
    assert free_after == free_before, "the driver's free-memory count changed across the call"
    assert binding.stem_check_status(plan, static_scratch=True)[0] == binding.STEM_OK
    ref, *_ = so.score(data["q"], data["k"], data["v"], data["cu_seqlens"], oracle_params(w))
    return want.cpu().numpy(), got.cpu().numpy(), ref


_set_up_done = False


def _first_call_set_up():
    """The documented one-time set-up: the first call on a device resolves the address of the built-in array
    (with CUDA's lazy module loading that is also the moment the array itself becomes resident).  It is made
    here on a tiny problem so that the calls under test are ordinary, later calls."""
    global _set_up_done
    if _set_up_done:
        return
    w = wl.small("noalloc_setup", seqlens=(300,), hq=2, hkv=1, block=64, permille=500)
    data = wl.make_qkv(w)
    plan = StemPlan.from_workload(w)
    m = torch.empty((w.num_q_heads, plan.info.metric_elems), dtype=torch.float32, device="cuda")
    binding.stem_score_static(plan, to_dev(data["q"]), to_dev(data["k"]), to_dev(data["v"]), m)
    torch.cuda.synchronize()
    _set_up_done = True


def _assert_close(want, got):
    defined = ~np.isnan(want)
    assert defined.any()
    assert np.array_equal(np.isnan(got), ~defined)
    # tolerance of the metric parity test
    tol = 2e-6 * np.maximum(1.0, np.abs(want[defined])) + 1e-6
    assert np.all(np.abs(got[defined] - want[defined]) <= tol)


def test_static_scratch_matches_workspace_path_and_checker_on_two_calls_in_a_row():
    # first call: a layer that nearly fills the array (669 block rows x 12 heads x 768 bytes = 6.2 MB);
    # second call: a smaller, differently shaped one, so stale contents of the shared array would show
    # up if the result ever depended on them
    first = wl.small("noalloc_a", seqlens=(65536, 20000), hq=8, hkv=4, block=128, permille=200, sink=True)
    second = wl.small("noalloc_b", seqlens=(3000,), hq=4, hkv=2, block=64, permille=300)
    for w in (first, second):
        want, got, ref = _metric_triple(w)
        # both entry points run the same pooling and metric kernels on the same inputs: identical bits
        assert np.array_equal(np.nan_to_num(want, nan=-1.0), np.nan_to_num(got, nan=-1.0))
        _assert_close(ref, got)     # and both agree with the checker written from the paper


def test_static_scratch_rejects_problems_beyond_its_size():
    w = wl.CONFIGS["cfg3"]  # 40 heads x 1024 rows of pooled vectors in three bf16 parts: 31 MB > 8 MB
    plan = StemPlan.from_workload(w)
    dummy = torch.zeros(1024, dtype=torch.bfloat16, device="cuda")
    m = torch.zeros(1024, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.StemError) as e:
        binding.stem_score_static(plan, dummy, dummy, dummy, m)
    assert e.value.status == binding.STEM_ERR_STATIC_SCRATCH
    with pytest.raises(binding.StemError) as e:
        binding.stem_score_static(plan, dummy, dummy, dummy, None)
    assert e.value.status == binding.STEM_ERR_INVALID_ARG
