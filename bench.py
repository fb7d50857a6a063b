#!/usr/bin/env python
"""Throughput of the multi-adapter LoRA forward (tokens/s per layer step) on B200.

A step is one pass of the hot path over one decode batch: segment metadata build, shrink and
expand (lora_build_segments + lora_bgmv_apply through the C ABI).  The default workload is the
q_proj-like decode batch: 256 tokens, 4096 -> 4096, 128 resident rank-16 adapters, Zipf(1.1).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica on its
own GPU; there is no exchange step in this path.  Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "multi-LoRA tokens/s per layer step"
UNIT = "tokens/s"
ROTATION = 16          # independent input / weight sets cycled through so every step is cold
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

PAPER_CONTEXT = {
    "note": "system-level results of the paper, other hardware, context only",
    "dt_throughput_smape": "2.25-5.08 % (Digital Twin on 1 CPU core vs vLLM v0.8.5 on 1x H100 64 GB)",
    "dt_speedup": "up to 90x faster than benchmarking (~39 s vs 1 h runs, 1 CPU core, no GPU)",
    "gpu_reduction": "-2.4 of 4 H100 GPUs on average (60 % fewer) vs dLoRAProactive / LoRAServe",
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=48000)
    ap.add_argument("--warmup", type=int, default=160)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=200)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--algo", type=int, default=None,
                    help="apply path: 0 fused cluster kernel (default), 1 two-phase kernels")
    ap.add_argument("--cluster", type=int, default=None, help="fused path: cluster size 1/2/4/8")
    ap.add_argument("--tile-m", type=int, default=None, help="rows per tile of the segment metadata")
    ap.add_argument("--tune", nargs="*", default=[], metavar="KEY=VALUE",
                    help="lora_pool_set_tuning pairs, e.g. 2=1 (no programmatic dependent launch)")
    return ap.parse_args()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def bench_workload():
    """Config 1 with ROTATION independent copies of the projection (weights and activations)."""
    from paper_2602_24044_b200 import workloads as W
    wl = W.make_config(1)
    wl.targets = wl.targets * ROTATION
    wl.calls = list(range(ROTATION))
    return wl


def algorithmic_bytes(wl, target=0):
    """Bytes one apply must move: x, y_base (active rows), y, and each distinct adapter's A and B
    at true rank, once."""
    d_in, d_out = wl.targets[target]
    act = wl.active_mask()
    T, Ta = wl.T, int(act.sum())
    b = 2 * T * d_in + 2 * Ta * d_out + 2 * T * d_out
    for s in wl.distinct_slots():
        b += 2 * int(wl.ranks[s]) * (d_in + d_out)
    return b


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.path = os.path.join("/tmp", "lora_bench_clocks_%d.csv" % os.getpid())

    def start(self):
        try:
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.out,
                stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [v.strip() for v in line.split(",")]
                if len(f) < 7:
                    continue
                try:
                    sm.append(float(f[0]))
                    mx.append(float(f[1]))
                except ValueError:
                    continue
                for n, v in zip(names, f[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            os.unlink(self.path)
        except Exception:
            pass
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(mx)) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def time_oracle(wl, budget_s=12.0, max_reps=2000, warm=1):
    """The CPU oracle as it stands on all host cores, on whole batches of the workload."""
    from oracle import lora_oracle as orc
    cores = orc.host_cores()
    x_h, yb_h = wl.activations(0)
    acts = (x_h, yb_h)
    orc.apply_workload(wl, 0, threads=cores, acts=acts)        # builds, warms
    # time only the oracle's loops: widen inputs once outside
    from paper_2602_24044_b200 import workloads as W
    x, yb = W.bf16_to_f64(x_h), W.bf16_to_f64(yb_h)
    N = wl.num_slots
    A, B = [None] * N, [None] * N
    for s in wl.distinct_slots():
        a, b = wl.adapter_weights(int(s), 0)
        A[s], B[s] = W.bf16_to_f64(a), W.bf16_to_f64(b)
    loaded = np.array([1 if A[i] is not None else 0 for i in range(N)], np.int32)
    def one():
        orc.apply(x, yb, wl.slot_idx, A, B, wl.ranks, wl.scales.astype(np.float64), loaded, cores)
        orc.build_segments(wl.slot_idx, wl.loaded, wl.ranks, wl.tile_m, wl.long_min)

    for _ in range(warm):
        one()
    reps, t_total = 0, 0.0
    while t_total < budget_s and reps < max_reps:
        t0 = time.perf_counter()
        one()
        t_total += time.perf_counter() - t0
        reps += 1
    return {"value": wl.T * reps / t_total, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d whole batches of the bench workload (%d tokens each), %.1f s of "
                      "fp64 loops on %d threads" % (reps, wl.T, t_total, cores),
            "ms_per_step": 1e3 * t_total / reps, "reps": reps}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = bench_workload()
    from oracle import lora_oracle as orc
    orc.build()
    # each step = one whole batch of the workload through the oracle; at most ~2 minutes in all
    t = time_oracle(wl, budget_s=120.0, max_reps=max(1, args.steps), warm=max(1, min(args.warmup, 20)))
    line = {"impl": "reference", "metric": METRIC, "value": t["value"], "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "steps_timed": t["reps"], "ms_per_step": t["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "config1 decode BGMV: 256 tokens, 4096->4096, 128 adapters "
                                   "rank 16, Zipf(1.1)"},
            "cpu_baseline": {k: t[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": t["value"], "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    args = parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist

    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200 import build as lbuild
    from paper_2602_24044_b200.harness import Session, bf16_tensor

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        lbuild.build()
    if world > 1:
        dist.barrier()

    wl = bench_workload()
    if args.tile_m is not None:
        wl.tile_m = args.tile_m
    d_in, d_out = wl.targets[0]
    T = wl.T
    tuning = {}
    if args.algo is not None:
        tuning[0] = args.algo
    if args.cluster is not None:
        tuning[1] = args.cluster
    for kv in args.tune:
        k, v = kv.split("=")
        tuning[int(k)] = int(v)
    s = Session(wl, device="cuda:%d" % local, a_layout=lb.A_RANK_MAJOR, tuning=tuning)
    dev = s.device
    xs, ybs, ys, metas = [], [], [], []
    meta_words = lb.segments_bytes(T, wl.num_slots, wl.tile_m) // 4
    for c in range(ROTATION):
        x_h, yb_h = wl.activations(c)
        xs.append(bf16_tensor(x_h, dev))
        ybs.append(bf16_tensor(yb_h, dev))
        ys.append(torch.empty((T, d_out), dtype=torch.bfloat16, device=dev))
        metas.append(torch.empty(meta_words, dtype=torch.int32, device=dev))
    torch.cuda.synchronize()

    def step(i):
        c = i % ROTATION
        lb.build_segments(s.pool, s.slot_idx_dev, T, wl.tile_m, wl.long_min, metas[c],
                          stream=s.compute)
        lb.bgmv_apply(s.pool, c, xs[c], d_in, ybs[c], d_out, ys[c], d_out, s.slot_idx_dev, T,
                      metas[c], s.ws, stream=s.compute)

    def apply_only(i):
        c = i % ROTATION
        lb.bgmv_apply(s.pool, c, xs[c], d_in, ybs[c], d_out, ys[c], d_out, s.slot_idx_dev, T,
                      metas[c], s.ws, stream=s.compute)

    def capture(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s.compute):
            for i in range(ROTATION):
                fn(i)
        return g

    # warm-up (also sets kernel attributes before capture)
    with torch.cuda.stream(s.compute):
        for i in range(max(args.warmup, 3)):
            step(i)
    torch.cuda.synchronize()
    l0 = lb.launch_count()
    g_step = capture(step)
    launches_per_rotation = lb.launch_count() - l0
    g_apply = capture(apply_only)
    torch.cuda.synchronize()

    def run_steps(K, graph, fn):
        with torch.cuda.stream(s.compute):
            for _ in range(K // ROTATION):
                graph.replay()
            for i in range(K % ROTATION):
                fn(i)

    run_steps(ROTATION * 4, g_step, step)
    torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    K = args.steps
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    l0 = lb.launch_count()
    e0.record(s.compute)
    run_steps(K, g_step, step)
    e1.record(s.compute)
    torch.cuda.synchronize()
    launches = (K // ROTATION) * launches_per_rotation + (lb.launch_count() - l0)
    if world > 1:
        dist.barrier()
    ms = e0.elapsed_time(e1)
    if world > 1:
        t = torch.tensor([ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())

    # the apply alone (dominant kernels), same rotation, for the roofline figure
    Kr = max(ROTATION, min(K, 16000) // ROTATION * ROTATION)
    r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    r0.record(s.compute)
    run_steps(Kr, g_apply, apply_only)
    r1.record(s.compute)
    torch.cuda.synchronize()
    apply_ms = r0.elapsed_time(r1) / Kr
    clocks = sampler.stop() if rank == 0 else None

    # end to end: host buffers in, host result out, every step (C entry point lora_apply_host)
    xh = [bf16_tensor(wl.activations(c)[0], pin=True) for c in range(2)]
    ybh = [bf16_tensor(wl.activations(c)[1], pin=True) for c in range(2)]
    yh = [torch.empty((T, d_out), dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    sh = torch.from_numpy(wl.slot_idx.copy()).pin_memory()
    sd = torch.empty(T, dtype=torch.int32, device=dev)

    def e2e_step(i):
        c = i % 2
        lb.apply_host(s.pool, i % ROTATION, 0, xh[c], ybh[c], yh[c], sh, T, wl.tile_m, wl.long_min,
                      xs[c], ybs[c], ys[c], sd, metas[c], s.ws, s.compute)

    for i in range(5):
        e2e_step(i)
    torch.cuda.synchronize()
    Ke = args.e2e_steps
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for i in range(Ke):
        e2e_step(i)
    s.compute.synchronize()
    e2e_s = time.perf_counter() - t0
    if world > 1:
        t = torch.tensor([e2e_s], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    h2d = 2 * T * (d_in + d_out) + 4 * T
    d2h = 2 * T * d_out

    if rank != 0:
        s.close()
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    alg = algorithmic_bytes(wl)
    achieved = alg / (apply_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": world * T * K / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": K, "warmup": args.warmup, "ms_per_step": ms / K, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16 in/out, fp32 accumulate",
        "data": "synthetic",
        "config": {
            "workload": "config1 decode BGMV: 256 tokens, 4096->4096, 128 resident adapters rank 16, "
                        "Zipf(1.1) over slots (%d distinct)" % len(wl.distinct_slots()),
            "step": "lora_build_segments + lora_bgmv_apply (grouped), one layer step",
            "cache": "cold: %d rotating input/weight sets (%.0f MB touched per rotation, L2 is 126 MB)"
                     % (ROTATION, ROTATION * alg / 1e6),
            "launch": "CUDA graph of %d consecutive steps replayed" % ROTATION,
            "multi_gpu": "independent replicas, no collective",
        },
        "roofline": {
            "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "peak_source": "%s copy bandwidth" % peak_kind,
            "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
            "kernel": ("lora_bgmv_apply: shrink_kernel + expand_kernel (two launches)"
                       if tuning.get(0) == 1 else "lora_bgmv_apply: fused_kernel (one launch)"),
            "algorithmic_bytes_per_launch": alg,
            "us_per_launch": apply_ms * 1e3, "traffic": None,
        },
        "step_GBps": alg / (ms / K * 1e-3) / 1e9,
        "e2e": {"value": world * T * Ke / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "api": "lora_apply_host", "steps": Ke},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "paper_context": PAPER_CONTEXT,
    }
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = {k: v for k, v in time_oracle(wl).items()
                                if k not in ("ms_per_step", "reps")}
    print(json.dumps(line))
    s.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
