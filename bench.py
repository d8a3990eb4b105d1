#!/usr/bin/env python
"""Benchmark of the Stem sparse causal prefill path on B200.

One step = one fused pass of Algorithm 1 (pool -> metric + select -> sparse attention) over one
synthetic attention layer, through the C ABI (``stem_prefill``).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3] [--impl stem|reference]

The headline value is ms per layer on the 128K-token Llama-3-8B-shaped layer (cfg3); the same
line also carries the 32K layer (cfg2), per-stage times, effective TFLOP/s on the selected
blocks, achieved HBM GB/s of scoring + selection, the dense causal comparator on the same GPU,
the end-to-end time with host buffers, and the CPU checker timed on a bounded sample.
With N > 1 (torchrun) every rank runs an independent replica of the layer (the path has no
exchange step); time is the max over ranks and value is ms per layer job-wide.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}
# DRAM traffic of one sparse-attention launch (ncu: dram__bytes_read.sum + dram__bytes_write.sum),
# captured on the workload itself; a workload without a capture reports null.
NCU_ATTN_DRAM_BYTES_PER_LAUNCH = {"cfg3_llama3_8b_128k": 1706697216 + 1047956480}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons, power = [], [], set(), []
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        # the busiest half of the samples is "under load"
        sm_sorted = sorted(sm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_mhz_min": sm_sorted[0] if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "power_w_max": max(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def dist_setup(n_gpus: int):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def max_over_ranks(x: float, world: int, device: str = "cuda") -> float:
    """Largest value of x over the ranks of the default process group (x itself when there is one rank)."""
    if world == 1:
        return x
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_layer(rank: int) -> int:
    """The path has no exchange step: rank r works on its own layer (seed offset r) of the workload."""
    return rank


def run_reference(args):
    """The CPU checker, as it stands, timed on this machine's host cores on a bounded sample."""
    rank, world, _ = dist_setup(args.gpus)
    if rank != 0:
        return
    from oracle import stem_oracle as so
    from paper_2603_06274_b200 import workloads as wl
    w = wl.CONFIGS[args.workload]
    res = cpu_sample(w, so, wl, n_rows=16, steps=args.steps, warmup=args.warmup)
    line = {"impl": "reference", "metric": "stem_prefill_ms_per_layer", "value": res["value"], "unit": "ms/layer",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": res["step_ms"],
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "tokens": w.total_tokens, "q_heads": w.num_q_heads,
                       "kv_heads": w.num_kv_heads, "block": w.block, "budget_permille": w.budget_permille},
            "cpu_baseline": {"value": res["value"], "unit": "ms/layer", "cores": res["cores"], "kind": "oracle",
                             "sample": res["sample"]},
            "e2e": {"value": res["value"], "unit": "ms/layer", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def cpu_sample(w, so, wl, n_rows: int, steps: int, warmup: int):
    """Times the checker on one kv-head group of the workload (all scoring / selection stages) plus
    the attention of `n_rows` sampled rows, and scales to a whole layer by work counts."""
    g = w.num_q_heads // w.num_kv_heads
    sub = w.with_(num_q_heads=g, num_kv_heads=1, name=w.name + "_kvgroup0")
    data = wl.make_qkv(sub)
    p = so.StemParams(block=w.block, budget_permille=w.budget_permille, k_start_blocks=w.k_start_blocks,
                      mu_num=w.mu_num, mu_den=w.mu_den, stem_blocks=w.stem_blocks, local_blocks=w.local_blocks,
                      min_blocks=w.min_blocks, beta=w.beta, score_scale=w.score_scale)
    seqlens = np.diff(data["cu_seqlens"])
    nblk = so.n_blocks(seqlens, w.block)
    k_eff = so.schedule_batch(seqlens, p)
    r_tot = int(nblk.sum())
    rng = np.random.default_rng(7)
    rows = np.stack([rng.integers(0, g, n_rows), rng.integers(r_tot // 2, r_tot, n_rows)], axis=1).astype(np.int32)
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        M, *_ = so.score(data["q"], data["k"], data["v"], data["cu_seqlens"], p)
        idx, cnt = so.select(M, nblk, k_eff, w.stem_blocks, w.local_blocks)
        t1 = time.perf_counter()
        so.attention(data["q"], data["k"], data["v"], data["cu_seqlens"], w.block, idx, cnt, rows=rows, want_lse=False)
        t2 = time.perf_counter()
        if it >= warmup:
            times.append((t1 - t0, t2 - t1, t2 - t0))
    sel_t = statistics.median(t[0] for t in times)
    att_t = statistics.median(t[1] for t in times)
    step_ms = statistics.median(t[2] for t in times) * 1e3
    sample_blocks = int(cnt[rows[:, 0], rows[:, 1]].sum())
    total_blocks = int(k_eff.sum()) * w.num_q_heads
    layer_ms = (sel_t * w.num_kv_heads + att_t * total_blocks / max(sample_blocks, 1)) * 1e3
    return {"value": layer_ms, "step_ms": step_ms, "cores": so.num_threads(),
            "sample": f"scoring+selection of 1 of {w.num_kv_heads} kv-head groups in full, attention of {n_rows} "
                      f"sampled (head,row) lists ({sample_blocks} of {total_blocks} selected blocks); "
                      f"scaled to the layer by group and block counts"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--impl", default="stem", choices=["stem", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the 32K layer, the dense comparator and e2e")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "stem" else args.warmup
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import paper_2603_06274_b200 as pkg
    from paper_2603_06274_b200 import workloads as wl

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the Stem path has no CPU fallback")
    rank, world, local = dist_setup(args.gpus)
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    pkg.load()
    peaks, peak_src = load_peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def dev(bits):
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    def time_loop(fn, steps, warmup):
        """CUDA-event time of `steps` calls on the current stream after `warmup` calls; ms per call."""
        for _ in range(warmup):
            fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1) / steps, world)

    def bench_workload(w, steps, warmup, extras: bool):
        data = wl.make_qkv(w, layer=replica_layer(rank))  # every rank draws its own layer
        plan = pkg.StemPlan.from_workload(w)
        info = plan.info
        q, k, v = dev(data["q"]), dev(data["k"]), dev(data["v"])
        out = torch.empty((w.total_tokens, w.num_q_heads, 128), dtype=torch.bfloat16, device="cuda")
        idx = torch.empty((w.num_q_heads, info.total_q_blocks, info.k_max), dtype=torch.int32, device="cuda")
        cnt = torch.empty((w.num_q_heads, info.total_q_blocks), dtype=torch.int32, device="cuda")
        plan.workspace()
        res = {}
        res["fused_ms"] = time_loop(lambda: pkg.stem_prefill(plan, q, k, v, out, idx, cnt), steps, warmup)
        st, detail = pkg.stem_check_status(plan)
        if st != 0:
            raise SystemExit(f"device status {st} {detail}")
        res["launches_per_step"] = plan.last_launch_count()
        # per stage, same buffers (lists from the fused run stay valid)
        res["pool_ms"] = time_loop(lambda: pkg.stem_score(plan, q, k, v, None), steps, warmup)
        res["score_select_ms"] = time_loop(lambda: pkg.stem_select(plan, None, idx, cnt), steps, warmup)
        res["scoring_stage_ms"] = time_loop(lambda: pkg.stem_score_select(plan, q, k, v, idx, cnt), steps, warmup)
        res["attn_ms"] = time_loop(lambda: pkg.stem_sparse_prefill(plan, q, k, v, idx, cnt, out), steps, warmup)
        qkv_bytes = (w.num_q_heads + 2 * w.num_kv_heads) * w.total_tokens * 128 * 2
        pooled_bytes = (w.num_q_heads + w.num_kv_heads) * info.total_q_blocks * 128 * 4 + w.num_kv_heads * info.total_q_blocks * 4
        list_bytes = w.num_q_heads * info.total_q_blocks * (info.k_max + 1) * 4
        res["score_bytes"] = qkv_bytes + 2 * pooled_bytes + list_bytes
        res["attn_flops"] = 4.0 * 128 * info.selected_pairs
        res["dense_flops"] = 4.0 * 128 * info.causal_pairs
        res["selected_blocks"] = int(info.selected_blocks)
        res["causal_blocks"] = int(info.causal_blocks)
        if extras:
            dsteps = max(2, min(steps, 3))
            res["dense_ms"] = time_loop(lambda: pkg.stem_sparse_prefill(plan, q, k, v, None, None, out), dsteps, 1)
            # end to end through the public call with HOST buffers: H2D of Q, K, V and D2H of O every step
            hq_, hk_, hv_ = (torch.from_numpy(data[n].view(np.int16)).pin_memory() for n in ("q", "k", "v"))
            ho = torch.empty(out.shape, dtype=torch.int16).pin_memory()

            def e2e_step():
                q.view(torch.int16).copy_(hq_, non_blocking=True)
                k.view(torch.int16).copy_(hk_, non_blocking=True)
                v.view(torch.int16).copy_(hv_, non_blocking=True)
                pkg.stem_prefill(plan, q, k, v, out, idx, cnt)
                ho.copy_(out.view(torch.int16), non_blocking=True)

            res["e2e_ms"] = time_loop(e2e_step, max(2, min(steps, 5)), 1)
            res["h2d"] = int(qkv_bytes)
            res["d2h"] = int(out.numel() * 2)
        plan.close()
        return res

    w = wl.CONFIGS[args.workload]
    sampler = ClockSampler(local)
    sampler.start()
    main_res = bench_workload(w, args.steps, args.warmup, extras=not args.no_extras)
    clocks = sampler.stop()
    also = {}
    if not args.no_extras and args.workload == "cfg3":
        w2 = wl.CONFIGS["cfg2"]
        r2 = bench_workload(w2, args.steps, args.warmup, extras=True)
        also[w2.name] = {"ms_per_layer": r2["fused_ms"], "attn_ms": r2["attn_ms"], "pool_ms": r2["pool_ms"],
                         "score_select_ms": r2["score_select_ms"], "dense_ms": r2.get("dense_ms"),
                         "attn_tflops": r2["attn_flops"] / (r2["attn_ms"] * 1e-3) / 1e12,
                         "e2e_ms": r2.get("e2e_ms")}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import stem_oracle as so  # the CPU baseline leg is the one place the bench runs the checker
        c = cpu_sample(w, so, wl, n_rows=48, steps=1, warmup=0)
        cpu = {"value": c["value"], "unit": "ms/layer", "cores": c["cores"], "kind": "oracle", "sample": c["sample"]}

    if world > 1:
        dist.destroy_process_group()
    if rank != 0:
        return
    attn_tflops = main_res["attn_flops"] / (main_res["attn_ms"] * 1e-3) / 1e12
    peak_tf = peaks["bf16_tflops"]
    score_ms = main_res["scoring_stage_ms"]
    score_gbs = main_res["score_bytes"] / (score_ms * 1e-3) / 1e9
    traffic = NCU_ATTN_DRAM_BYTES_PER_LAUNCH.get(w.name)
    ms_layer = main_res["fused_ms"] / world
    line = {
        "metric": "stem_prefill_ms_per_layer", "value": ms_layer, "unit": "ms/layer", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": main_res["fused_ms"], "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "tokens": w.total_tokens, "q_heads": w.num_q_heads, "kv_heads": w.num_kv_heads,
                   "block": w.block, "budget_permille": w.budget_permille, "mu": f"{w.mu_num}/{w.mu_den}",
                   "stem_local_min": [w.stem_blocks, w.local_blocks, w.min_blocks],
                   "l2": "inputs (Q,K,V,O > 2.6 GB) exceed the 126 MB L2; no explicit flush",
                   "parallelism": "replicas" if world > 1 else "single"},
        "clocks": clocks,
        "gpu_launches": main_res["launches_per_step"] * args.steps,
        "stages_ms": {"pool": main_res["pool_ms"], "metric_plus_select": main_res["score_select_ms"],
                      "scoring_stage_one_call": main_res["scoring_stage_ms"],
                      "sparse_attention": main_res["attn_ms"], "dense_causal_same_kernel": main_res.get("dense_ms")},
        "effective_tflops": attn_tflops,
        "selected_over_causal_blocks": main_res["selected_blocks"] / main_res["causal_blocks"],
        "roofline": {"kernel": "sparse_attn_kernel", "bound": "tensor", "achieved": attn_tflops, "peak": peak_tf,
                     "unit": "TFLOP/s", "frac": attn_tflops / peak_tf, "traffic": traffic,
                     "peak_source": f"{peak_src} burst bf16 ({peak_tf}); sustained {peaks['bf16_tflops_sustained']}, "
                                    f"nominal {NOMINAL['bf16_tflops']}",
                     "frac_of_sustained": attn_tflops / peaks["bf16_tflops_sustained"],
                     "frac_of_nominal": attn_tflops / NOMINAL["bf16_tflops"]},
        "roofline_scoring": {"kernels": "pool_kernel + metric_gemm_kernel + select_planes_kernel", "bound": "hbm", "achieved": score_gbs,
                             "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": score_gbs / peaks["hbm_gbs"],
                             "frac_of_nominal": score_gbs / NOMINAL["hbm_gbs"], "bytes": main_res["score_bytes"],
                             "ms": score_ms},
        "dense_comparator": None if "dense_ms" not in main_res else {
            "ms": main_res["dense_ms"], "tflops": main_res["dense_flops"] / (main_res["dense_ms"] * 1e-3) / 1e12,
            "speedup_of_stem": main_res["dense_ms"] / main_res["fused_ms"]},
        "e2e": None if "e2e_ms" not in main_res else {
            "value": main_res["e2e_ms"] / world, "unit": "ms/layer", "h2d_bytes_per_step": main_res["h2d"],
            "d2h_bytes_per_step": main_res["d2h"]},
        "cpu_baseline": cpu,
        "also": also,
    }
    print(json.dumps(line))


if __name__ == "__main__":
    main()
