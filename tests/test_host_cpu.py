"""Host-side checks that need no GPU: the library loads, exports what the header declares,
validates configurations, and its budget table equals the checker's schedule."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import stem_oracle as so
from paper_2603_06274_b200 import binding, workloads as wl
from tests._util import oracle_params

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "stem.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(stem_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.load()
    names = _declared_functions()
    assert "stem_prefill" in names and "stem_score" in names and "stem_select" in names
    assert "stem_sparse_prefill" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in stem.h but not exported"
    assert set(names) == set(binding.EXPORTS)
    assert lib.stem_version() >= 100
    assert binding.status_string(0) == "ok"
    assert "workspace" in binding.status_string(binding.STEM_ERR_WORKSPACE)


def _config(seqlens, hq, hkv, block=128, **kw):
    cu = np.concatenate([[0], np.cumsum(seqlens)]).astype(np.int32)
    cfg = binding.StemConfig()
    cfg.batch = len(seqlens)
    cfg.cu_seqlens_host = cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
    cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.block = hq, hkv, kw.get("head_dim", 128), block
    cfg.budget_permille = kw.get("budget_permille", 100)
    cfg.k_start_blocks = kw.get("k_start_blocks", 0)
    cfg.mu_num, cfg.mu_den = kw.get("mu", (7, 10))
    cfg.stem_blocks, cfg.local_blocks, cfg.min_blocks = kw.get("stem", 4), kw.get("local", 4), kw.get("min_blocks", 0)
    cfg.beta = 0.2
    cfg.q_stride_tok, cfg.q_stride_head = kw.get("q_strides", (hq * 128, 128))
    cfg.kv_stride_tok, cfg.kv_stride_head = hkv * 128, 128
    return cfg, cu


def _budget(cfg):
    lib = binding.load()
    n = ctypes.c_int32()
    rc = lib.stem_budget_table(ctypes.byref(cfg), None, 0, ctypes.byref(n))
    if rc != 0:
        return rc, None
    out = np.empty(n.value, np.int32)
    rc = lib.stem_budget_table(ctypes.byref(cfg), out.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), n.value, None)
    return rc, out


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
def test_budget_table_equals_checker_schedule(name):
    w = wl.CONFIGS[name]
    cfg, cu = _config(w.seqlens, w.num_q_heads, w.num_kv_heads, w.block, budget_permille=w.budget_permille,
                      mu=(w.mu_num, w.mu_den), stem=w.stem_blocks, local=w.local_blocks, min_blocks=w.min_blocks)
    rc, got = _budget(cfg)
    assert rc == 0
    want = so.schedule_batch(w.seqlens, oracle_params(w))
    assert np.array_equal(got, want)


def test_budget_table_sweeps():
    rng = np.random.default_rng(0)
    for _ in range(40):
        seqlens = [int(x) for x in rng.integers(1, 9000, size=int(rng.integers(1, 4)))]
        block = int(rng.choice([64, 128]))
        kw = dict(budget_permille=int(rng.integers(0, 1001)), mu=(int(rng.integers(1, 11)), 10),
                  stem=int(rng.integers(0, 6)), local=int(rng.integers(1, 6)), min_blocks=int(rng.integers(0, 60)))
        cfg, cu = _config(seqlens, 4, 2, block, **kw)
        rc, got = _budget(cfg)
        assert rc == 0
        p = so.StemParams(block=block, budget_permille=kw["budget_permille"], mu_num=kw["mu"][0], mu_den=10,
                          stem_blocks=kw["stem"], local_blocks=kw["local"], min_blocks=kw["min_blocks"])
        assert np.array_equal(got, so.schedule_batch(seqlens, p))
    # explicit k_start in blocks (the paper's plug-in settings use fixed counts)
    cfg, cu = _config([8192], 2, 2, 128, k_start_blocks=64, mu=(7, 10), stem=0, local=1)
    rc, got = _budget(cfg)
    p = so.StemParams(block=128, k_start_blocks=64, stem_blocks=0, local_blocks=1)
    assert rc == 0 and np.array_equal(got, so.schedule_batch([8192], p))


def test_invalid_configurations_are_rejected():
    ok, _ = _config([1024], 4, 2)
    assert _budget(ok)[0] == 0
    bad = [
        (_config([1024], 4, 2, head_dim=64)[0], binding.STEM_ERR_UNSUPPORTED),
        (_config([1024], 4, 2, block=32)[0], binding.STEM_ERR_UNSUPPORTED),
        (_config([1024], 5, 2)[0], binding.STEM_ERR_UNSUPPORTED),
        (_config([1024], 4, 2, mu=(11, 10))[0], binding.STEM_ERR_INVALID_ARG),
        (_config([1024], 4, 2, mu=(0, 10))[0], binding.STEM_ERR_INVALID_ARG),
        (_config([1024], 4, 2, local=0)[0], binding.STEM_ERR_INVALID_ARG),
        (_config([1024], 4, 2, budget_permille=1001)[0], binding.STEM_ERR_INVALID_ARG),
        (_config([1024], 4, 2, q_strides=(4 * 128 + 4, 128))[0], binding.STEM_ERR_INVALID_ARG),
    ]
    for cfg, want in bad:
        assert _budget(cfg)[0] == want
    cfg, cu = _config([1024, 0 + 1], 4, 2)
    cu[2] = cu[1]  # empty sequence
    assert _budget(cfg)[0] == binding.STEM_ERR_INVALID_ARG
    lib = binding.load()
    assert lib.stem_budget_table(None, None, 0, None) == binding.STEM_ERR_INVALID_ARG
    assert lib.stem_plan_query(None, None) == binding.STEM_ERR_INVALID_ARG
    assert lib.stem_plan_destroy(None) == binding.STEM_ERR_INVALID_ARG


def test_workload_generators_are_deterministic_and_shaped():
    w = wl.small(seqlens=(300, 200), hq=4, hkv=2, block=64, sink=True)
    a, b = wl.make_qkv(w), wl.make_qkv(w)
    for k in ("q", "k", "v"):
        assert np.array_equal(a[k], b[k]) and a[k].dtype == np.uint16
    assert a["q"].shape == (500, 4, 128) and a["k"].shape == (500, 2, 128)
    assert not np.array_equal(wl.make_qkv(w, layer=1)["q"], a["q"])
    x = np.array([1.0, -2.5, 3.1415927, 1e-20, 65504.0], np.float32)
    back = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(x))
    assert np.all(np.abs(back - x) <= np.abs(x) * 2.0 ** -8)


def test_token_level_budget_is_the_schedule_with_one_token_per_block():
    # Eq. 3 at token positions (the top-2048 selector setting: k_start = 2048, mu = 0.7): the library's host table
    # against the checker's schedule with block size 1, and against the printed k_uni = 0.85 k_start
    n, k_s = 16384, 2048
    p = so.StemParams(block=1, k_start_blocks=k_s, mu_num=7, mu_den=10, stem_blocks=0, local_blocks=1)
    got = binding.stem_token_budget(n, k_s, (7, 10), 0, 1).numpy()
    assert np.array_equal(got, so.schedule(n, k_s, p)[1])
    uncapped = np.floor(k_s - k_s * 0.3 * np.arange(1, n + 1) / n)
    assert abs(uncapped.mean() / k_s - 0.85) < 1e-3
    assert got[-1] == int(0.7 * k_s) and got[0] == 1 and got[k_s + 500] == uncapped[k_s + 500]
