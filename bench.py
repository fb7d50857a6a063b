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

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# captures summarised under profiles/ (None: no capture of the current kernel on that workload)
NCU_TRAFFIC = {1: 22.9e6, (4, "layer"): 269.7e6, 3: 171.1e6}

PAPER_CONTEXT = {
    "note": "system-level results of the paper, other hardware, context only",
    "dt_throughput_smape": "2.25-5.08 % (Digital Twin on 1 CPU core vs vLLM v0.8.5 on 1x H100 64 GB)",
    "dt_speedup": "up to 90x faster than benchmarking (~39 s vs 1 h runs, 1 CPU core, no GPU)",
    "gpu_reduction": "-2.4 of 4 H100 GPUs on average (60 % fewer) vs dLoRAProactive / LoRAServe",
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--config", type=int, default=1, choices=[0, 1, 2, 3, 4],
                    help="workload: 1 (default) is the headline decode batch; the others are the parity configurations")
    ap.add_argument("--warmup", type=int, default=160)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=200)
    ap.add_argument("--e2e-lanes", type=int, default=3, help="streams (with their staging buffers) the end-to-end steps rotate over")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--algo", type=int, default=None,
                    help="apply path: 0 fused cluster kernel (default), 1 two-phase kernels")
    ap.add_argument("--cluster", type=int, default=None, help="fused path: cluster size 1/2/4/8")
    ap.add_argument("--tile-m", type=int, default=None, help="rows per tile of the segment metadata")
    ap.add_argument("--multi", default="layer", choices=["off", "groups", "layer"],
                    help="config 4: projections per launch: off = one lora_bgmv_apply each; groups = "
                         "{q,k,v} {o} {gate,up} {down} (the projections whose inputs exist together in a "
                         "transformer layer); layer = all seven of a layer in one lora_bgmv_apply_multi")
    ap.add_argument("--sweep", action="store_true",
                    help="instead of the benchmark line: apply latency against the number of distinct adapters, "
                         "the rank and the batch size, and swap-in latency against the adapter size, with the "
                         "linear fits the paper's performance model uses (Section 5.2, Eq. 1)")
    ap.add_argument("--layers", type=int, default=32,
                    help="config 4: transformer layers in the step (fewer only for profiling captures)")
    ap.add_argument("--tune", nargs="*", default=[], metavar="KEY=VALUE",
                    help="lora_pool_set_tuning pairs, e.g. 2=1 (no programmatic dependent launch)")
    return ap.parse_args()


def max_over_ranks(value, device=None):
    """The largest `value` of all ranks (every rank gets it); the identity without a process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world, tokens_per_step, steps, ms):
    """Tokens per second of all replicas together: every rank ran `steps` steps of its own batch in
    `ms` milliseconds (the slowest rank's time)."""
    return world * tokens_per_step * steps / (ms * 1e-3)


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


def time_oracle(wl, budget_s=12.0, max_reps=20000, warm=1):
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
    t = time_oracle(wl, budget_s=120.0, max_reps=max(1, args.steps or 48000), warm=max(1, min(args.warmup, 20)))
    line = {"impl": "reference", "metric": METRIC, "value": t["value"], "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "steps_timed": t["reps"], "ms_per_step": t["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_text(1, wl)},
            "cpu_baseline": {k: t[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": t["value"], "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


WORKLOAD_TEXT = {
    0: "config0 decode BGMV tiny: 16 tokens, 1024->1024, 8 adapters rank 8, uniform slots",
    1: "config1 decode BGMV: 256 tokens, 4096->4096, 128 resident adapters rank 16, Zipf(1.1) over slots",
    2: "config2 prefill SGMV: 32 requests, lognormal prompt lengths (median 512, clip 32..2048), "
       "4096->14336 and 14336->4096, 64 adapters ranks {8,16,32}",
    3: "config3 mixed chunked prefill SGMV: 512 decode tokens + 4 chunks of 512, fused QKV 4096->6144, "
       "384 adapters ranks {8,16,32,64}, Zipf(0.9)",
    4: "config4 full 32-layer decode step, Llama-3-8B shapes, LoRA on all 7 projections, 256 tokens, "
       "256 adapters rank 16, Zipf(1.1)",
}


def workload_text(cfg, wl):
    """The `config.workload` string of a configuration: the same for both arms of the benchmark."""
    return WORKLOAD_TEXT[cfg] + " (%d tokens, %d distinct adapters)" % (wl.T, len(wl.distinct_slots()))


def case_workload(cfg, layers=32):
    """The workload object of a configuration, with the rotation of independent copies that keeps
    every step cold in L2 for the small ones."""
    from paper_2602_24044_b200 import workloads as W
    wl = W.make_config(cfg, layers=layers) if cfg == 4 else W.make_config(cfg)
    rotation = 1
    if cfg in (0, 1):
        rotation = ROTATION
    elif cfg == 3:
        rotation = 2
    n_proj = len(wl.targets)
    if rotation > 1:
        wl.targets = wl.targets * rotation
        wl.calls = list(range(len(wl.targets)))
    return wl, rotation, n_proj


# ---------------------------------------------------------------------------------------------
# Sweep: the two estimators of the paper's performance model that this library's kernels
# determine (Section 5.2, Eq. 1): the adapter overhead of the forward pass, modelled as linear in
# the number of adapters in the batch (Overhead_A = K6 * A + K7, Section 5.1: linear growth, a jump
# from no adapter to one, little influence of the rank), and Lat_load(S_A), the time to bring an
# adapter of a given size from CPU memory.
# ---------------------------------------------------------------------------------------------
def run_sweep(args):
    import torch
    from paper_2602_24044_b200 import binding as lb
    from paper_2602_24044_b200 import build as lbuild
    from paper_2602_24044_b200 import workloads as W
    from paper_2602_24044_b200.harness import Session, bf16_tensor

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(0)
    lbuild.build()
    dev = torch.device("cuda", 0)
    sampler = ClockSampler(0)
    sampler.start()
    N, ROT, ACTS, D_IN, D_OUT, T_MAX = 128, 8, 32, 4096, 4096, 1024
    out = {"sweep": "apply latency (one projection 4096->4096, cold: %d rotating weight copies, %d rotating "
                    "activation sets) and swap-in latency" % (ROT, ACTS), "apply": [], "fits": [], "load": []}
    rng = np.random.default_rng(26022404)
    acts = [(torch.randn((T_MAX, D_IN), device=dev).to(torch.bfloat16),
             torch.randn((T_MAX, D_OUT), device=dev).to(torch.bfloat16),
             torch.empty((T_MAX, D_OUT), dtype=torch.bfloat16, device=dev)) for _ in range(ACTS)]

    def time_graph(s, fn, n_calls):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s.compute):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(s.compute):
            for _ in range(3):
                g.replay()
            a.record(s.compute)
            g.replay()
            b.record(s.compute)
        torch.cuda.synchronize()
        n = max(3, int(np.ceil(60.0 / max(a.elapsed_time(b), 1e-3))))
        with torch.cuda.stream(s.compute):
            a.record(s.compute)
            for _ in range(n):
                g.replay()
            b.record(s.compute)
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e3 / (n * n_calls)

    for rank in (8, 16, 32, 64):
        wl = W.make_custom(T_MAX, D_IN, D_OUT, N, rank, r_max=64, scale=2.0, tile_m=8, seed=100 + rank)
        wl.targets = wl.targets * ROT
        wl.calls = list(range(ROT))
        s = Session(wl, a_layout=lb.A_RANK_MAJOR, T_cap=T_MAX)
        points = [(256, D) for D in (0, 1, 2, 4, 8, 16, 32, 64, 128)] + \
                 [(T, min(T, 64)) for T in (64, 128, 512, 1024)]
        for T, D in points:
            # one table per slot group, so that consecutive applies use different adapters
            groups = max(1, N // max(D, 1))
            metas, sidx = [], []
            for gidx in range(min(groups, 8)):
                if D == 0:
                    idx = np.full(T, -1, np.int32)
                else:
                    idx = (gidx * D + (np.arange(T) % D)).astype(np.int32)
                    rng.shuffle(idx)
                d = torch.from_numpy(idx).to(dev)
                m = torch.empty(lb.segments_bytes(T, N, 8) // 4, dtype=torch.int32, device=dev)
                lb.build_segments(s.pool, d, T, 8, 128, m, stream=s.compute)
                metas.append(m)
                sidx.append(d)
            n_calls = ACTS

            def calls():
                for k in range(n_calls):
                    x, yb, y = acts[k % ACTS]
                    j = k % len(metas)
                    lb.bgmv_apply(s.pool, k % ROT, x[:T], D_IN, yb[:T], D_OUT, y[:T], D_OUT, sidx[j], T,
                                  metas[j], s.ws, stream=s.compute)
            with torch.cuda.stream(s.compute):
                calls()
            torch.cuda.synchronize()
            us = time_graph(s, calls, n_calls)
            bytes_ = 2 * T * D_IN + (4 if D else 0) * T * D_OUT + 2 * D * rank * (D_IN + D_OUT)
            out["apply"].append({"rank": rank, "T": T, "distinct_adapters": D, "us_per_apply": round(us, 3),
                                 "algorithmic_MB": round(bytes_ / 1e6, 3),
                                 "us_at_measured_peak": round(bytes_ / measured_peak()[0] * 1e-3, 3)})
        st = lb.pool_check_status(s.pool, s.compute)
        assert st[1] == 0, "a bounded device-side wait expired"
        s.close()
        pts = [(p["distinct_adapters"], p["us_per_apply"]) for p in out["apply"]
               if p["rank"] == rank and p["T"] == 256 and p["distinct_adapters"] >= 1]
        A = np.array([[d, 1.0] for d, _ in pts])
        yv = np.array([u for _, u in pts])
        (k6, k7), res, _, _ = np.linalg.lstsq(A, yv, rcond=None)
        zero = [p["us_per_apply"] for p in out["apply"] if p["rank"] == rank and p["T"] == 256
                and p["distinct_adapters"] == 0][0]
        pred = A @ np.array([k6, k7])
        out["fits"].append({"rank": rank, "T": 256, "model": "us = K6 * A + K7 over A = 1 .. 128 adapters in the batch",
                            "K6_us_per_adapter": round(float(k6), 4), "K7_us": round(float(k7), 3),
                            "max_abs_residual_us": round(float(np.abs(pred - yv).max()), 3),
                            "us_without_adapter": round(zero, 3),
                            "jump_0_to_1_us": round(pts[0][1] - zero, 3),
                            "bytes_model_slope_us_per_adapter": round(2 * rank * (D_IN + D_OUT) / measured_peak()[0] * 1e-3, 4)})

    # Lat_load: one adapter of Llama-3-8B shape (7 projections x 32 layers) from pinned host memory
    targets = W.LLAMA3_8B_TARGETS * 32
    for rank in (8, 16, 32, 64):
        wl = W.make_custom(8, 64, 64, 2, rank, r_max=rank, seed=200 + rank)
        wl.targets = targets
        wl.calls = [0]
        wl.weight_mode = "lora"
        s = Session(wl, slots=[])
        per = sum(a + b for a, b in targets) * rank * 2
        packed = torch.empty(per // 2, dtype=torch.bfloat16).pin_memory()
        mats_a = [torch.empty((rank, a), dtype=torch.bfloat16).pin_memory() for a, _ in targets]
        mats_b = [torch.empty((rank, b), dtype=torch.bfloat16).pin_memory() for _, b in targets]
        res = {}
        for name, A_, B_, layout in (("one_buffer", [packed] * len(targets), [packed] * len(targets), lb.PACKED),
                                     ("per_matrix", mats_a, mats_b, lb.A_RANK_MAJOR)):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            lb.pool_load_slot(s.pool, 0, rank, 2.0, A_, B_, layout, s.load, None, True)
            torch.cuda.synchronize()
            reps = 3
            a.record(s.load)
            for k in range(reps):
                lb.pool_load_slot(s.pool, k % 2, rank, 2.0, A_, B_, layout, s.load, None, True)
            b.record(s.load)
            torch.cuda.synchronize()
            res[name] = a.elapsed_time(b) / reps
        out["load"].append({"rank": rank, "adapter_MB": round(per / 1e6, 1),
                            "ms_one_buffer": round(res["one_buffer"], 3), "ms_per_matrix": round(res["per_matrix"], 3),
                            "GBps_one_buffer": round(per / res["one_buffer"] / 1e6, 1),
                            "GBps_per_matrix": round(per / res["per_matrix"] / 1e6, 1)})
        s.close()
    ld = out["load"]
    A = np.array([[p["adapter_MB"], 1.0] for p in ld])
    (m, c), _, _, _ = np.linalg.lstsq(A, np.array([p["ms_one_buffer"] for p in ld]), rcond=None)
    out["fits"].append({"model": "Lat_load ms = a * S_A[MB] + b (one pinned buffer per adapter)",
                        "a_ms_per_MB": round(float(m), 5), "b_ms": round(float(c), 3)})
    out["clocks"] = sampler.stop()
    out["peak_GBps"] = measured_peak()[0]
    print(json.dumps(out))


def main():
    args = parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.sweep:
        return run_sweep(args)

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

    cfg = args.config
    wl, rotation, n_proj = case_workload(cfg, args.layers)
    if args.tile_m is not None:
        wl.tile_m = args.tile_m
    T = wl.T
    tuning = {}
    if args.algo is not None:
        tuning[0] = args.algo
    if args.cluster is not None:
        tuning[1] = args.cluster
    for kv in args.tune:
        k, v = kv.split("=")
        tuning[int(k)] = int(v)
    dev = torch.device("cuda", local)
    if cfg == 4:
        # 256 slots x 83.9 MB: every slot is filled by a swap-in from ONE pinned host adapter (the
        # values do not influence the timing; addresses and sizes are those of 256 distinct adapters)
        s = Session(wl, device="cuda:%d" % local, slots=[], tuning=tuning)
        blobs = s.host_adapter(0, lb.A_RANK_MAJOR)
        for slot in range(wl.num_slots):
            s.load_slot(slot, a_layout=lb.A_RANK_MAJOR, src_slot=0, blobs=blobs)
        torch.cuda.synchronize()
    else:
        s = Session(wl, device="cuda:%d" % local, a_layout=lb.A_RANK_MAJOR, tuning=tuning)

    # device buffers: one set per rotation index; a set holds the step's applies in order
    act_sets = min(rotation, ROTATION) if cfg != 4 else 4     # config 4: activations of 4 layers cycle
    sets, metas = [], []
    meta_words = lb.segments_bytes(T, wl.num_slots, wl.tile_m) // 4
    n_sets = rotation if cfg != 4 else 1
    acts = {}
    multi = args.multi if (cfg == 4 and tuning.get(0) != 1) else "off"
    share = {1: 0, 2: 0, 5: 4} if multi != "off" else {}     # k, v read q's input; up reads gate's
    for r in range(n_sets):
        calls = []
        for j in range(len(wl.calls) // n_sets):
            call = r * (len(wl.calls) // n_sets) + j
            key = call if cfg != 4 else call % (7 * act_sets)
            if cfg == 4 and (call % 7) in share and key not in acts:
                # same device tensor for the shared input, own y_base and y
                kx = key - (call % 7) + share[call % 7]
                _, yb_h = wl.activations(key)
                acts[key] = (acts[kx][0], bf16_tensor(yb_h, dev),
                             torch.empty(yb_h.shape, dtype=torch.bfloat16, device=dev))
            if key not in acts:
                x_h, yb_h = wl.activations(key)
                acts[key] = (bf16_tensor(x_h, dev), bf16_tensor(yb_h, dev),
                             torch.empty(yb_h.shape, dtype=torch.bfloat16, device=dev))
            x, yb, y = acts[key]
            calls.append((s.target_pos[wl.calls[call]], x, yb, y))
        sets.append(calls)
        metas.append(torch.empty(meta_words, dtype=torch.int32, device=dev))
    torch.cuda.synchronize()
    sgmv = wl.kind == "sgmv"

    # config 4 with several projections per launch: item lists built once
    launches_multi = None
    if multi != "off":
        shapes = {"layer": [[4, 5, 6, 0, 3, 1, 2]], "groups": [[0, 1, 2], [3], [4, 5], [6]]}[multi]
        launches_multi = []
        for layer in range(len(sets[0]) // 7):
            for grp in shapes:
                items = []
                for p in grp:
                    tp, x, yb, y = sets[0][7 * layer + p]
                    items.append((tp, x, x.shape[1], yb, yb.shape[1], y, y.shape[1]))
                launches_multi.append(lb.make_apply_items(items))

    def apply_calls(r):
        if launches_multi is not None:
            for items in launches_multi:
                lb.bgmv_apply_multi(s.pool, items, s.slot_idx_dev, T, metas[r], s.ws, stream=s.compute)
            return
        for tp, x, yb, y in sets[r]:
            if sgmv:
                lb.sgmv_apply(s.pool, tp, x, x.shape[1], yb, yb.shape[1], y, y.shape[1], metas[r], T, s.ws,
                              stream=s.compute)
            else:
                lb.bgmv_apply(s.pool, tp, x, x.shape[1], yb, yb.shape[1], y, y.shape[1], s.slot_idx_dev,
                              T, metas[r], s.ws, stream=s.compute)

    def step(i):
        r = i % n_sets
        lb.build_segments(s.pool, s.slot_idx_dev, T, wl.tile_m, wl.long_min, metas[r], stream=s.compute)
        apply_calls(r)

    def apply_only(i):
        apply_calls(i % n_sets)

    def capture(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s.compute):
            for i in range(n_sets):
                fn(i)
        return g

    # warm-up (also sets kernel attributes before capture)
    with torch.cuda.stream(s.compute):
        for i in range(max(min(args.warmup, 8 * n_sets), 3)):
            step(i)
    torch.cuda.synchronize()
    l0 = lb.launch_count()
    g_step = capture(step)
    launches_per_rotation = lb.launch_count() - l0
    g_apply = capture(apply_only)
    torch.cuda.synchronize()

    MIN_REGION_MS = 200.0      # every timed region lasts at least this long

    def all_ranks_max_int(v):
        return int(round(max_over_ranks(v, dev)))

    def time_graph(graph, min_replays):
        """Milliseconds for `n` back-to-back replays of a captured graph on the compute stream, with
        n >= min_replays chosen so that the region lasts at least MIN_REGION_MS.  The graph is
        replayed three times untimed first; nothing but whole replays runs inside the region."""
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(s.compute):
            for _ in range(3):
                graph.replay()
            a.record(s.compute)
            graph.replay()
            b.record(s.compute)
        torch.cuda.synchronize()
        one = max(a.elapsed_time(b), 1e-4)
        n = all_ranks_max_int(max(min_replays, int(np.ceil(MIN_REGION_MS / one))))
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        with torch.cuda.stream(s.compute):
            a.record(s.compute)
            for _ in range(n):
                graph.replay()
            b.record(s.compute)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        return max_over_ranks(a.elapsed_time(b), dev), n

    def run_steps(K, graph, fn):
        """K steps as whole replays (K rounded up to a multiple of the graph's step count)."""
        with torch.cuda.stream(s.compute):
            for _ in range((K + n_sets - 1) // n_sets):
                graph.replay()

    K_req = args.steps if args.steps is not None else {0: 48000, 1: 48000, 2: 300, 3: 3000, 4: 100}[cfg]
    W_ = max(args.warmup, 3)
    run_steps(W_, g_step, step)
    torch.cuda.synchronize()
    lb.pool_reset_status(s.pool, s.compute)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ms, n_rep = time_graph(g_step, (K_req + n_sets - 1) // n_sets)
    K = n_rep * n_sets
    launches = n_rep * launches_per_rotation

    # the applies alone (dominant kernel), same rotation, for the roofline figure
    calls_per_step = len(sets[0])
    launches_per_step = len(launches_multi) if launches_multi is not None else calls_per_step
    apply_total_ms, n_apply_rep = time_graph(g_apply, 1)
    apply_ms = apply_total_ms / (n_apply_rep * n_sets) / launches_per_step
    # the same applies with ONE input / weight set replayed (small configurations: everything stays
    # in L2), reported beside the cold figure and labelled as warm
    warm_us = None
    if n_sets > 1:
        gw = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gw, stream=s.compute):
            for _ in range(n_sets):
                apply_calls(0)
        warm_ms, n_warm = time_graph(gw, 1)
        warm_us = warm_ms * 1e3 / (n_warm * n_sets * launches_per_step)
    # a bounded device-side wait that expired anywhere above invalidates the numbers
    try:
        status_words = lb.pool_check_status(s.pool, s.compute)
    except lb.LoraError:
        status_words = [int(v) for v in s.status()]
    clocks = sampler.stop() if rank == 0 else None

    # swap-in on the side stream while steps run (config 4: 16 misses per step)
    swap = None
    if cfg == 4 and rank == 0:
        blobs = s.host_adapter_packed(0)      # one pinned buffer per adapter: a single DMA per miss
        adapter_bytes = int(blobs[0][0].numel()) * 2
        steps_sw = 5
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0e, l1e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        ev0.record(s.compute)
        l0e.record(s.load)
        for i in range(steps_sw):
            for v in wl.swap_victims:
                lb.pool_load_slot(s.pool, v, int(wl.ranks[v]), float(wl.scales[v]), blobs[0], blobs[1],
                                  lb.PACKED, s.load, None, True)
            run_steps(1, g_step, step)
        ev1.record(s.compute)
        l1e.record(s.load)
        torch.cuda.synchronize()
        swap = {"misses_per_step": len(wl.swap_victims), "adapter_bytes": adapter_bytes,
                "h2d_GBps": steps_sw * len(wl.swap_victims) * adapter_bytes / (l0e.elapsed_time(l1e) * 1e6),
                "ms_per_step_compute_while_loading": ev0.elapsed_time(ev1) / steps_sw,
                "ms_per_step_of_loads": l0e.elapsed_time(l1e) / steps_sw,
                "note": "victim slots are not referenced by the step's tokens; loads run on the side "
                        "stream concurrently with the compute stream"}

    # end to end: host buffers in, host result out, every step (C entry point lora_apply_host)
    d_in0, d_out0 = wl.targets[wl.calls[0]]
    Ke = args.e2e_steps if cfg in (0, 1) else max(3, min(args.e2e_steps, 10))
    x_h, yb_h = wl.activations(0)
    NL = args.e2e_lanes
    xh = [bf16_tensor(x_h, pin=True) for _ in range(NL)]
    ybh = [bf16_tensor(yb_h, pin=True) for _ in range(NL)]
    yh = [torch.empty((T, d_out0), dtype=torch.bfloat16).pin_memory() for _ in range(NL)]
    sh = torch.from_numpy(wl.slot_idx.copy()).pin_memory()
    tp0, xd0, ybd0, yd0 = sets[0][0]
    # lanes (stream + device staging buffers each), used in turn: the host-to-device copy of one
    # step overlaps the compute and the device-to-host copy of the steps before it
    lanes = []
    for lane in range(NL):
        lanes.append({
            "stream": s.compute if lane == 0 else torch.cuda.Stream(dev),
            "x": xd0 if lane == 0 else torch.empty_like(xd0),
            "yb": ybd0 if lane == 0 else torch.empty_like(ybd0),
            "y": yd0 if lane == 0 else torch.empty_like(yd0),
            "sidx": torch.empty(T, dtype=torch.int32, device=dev),
            "meta": metas[0] if lane == 0 else torch.empty_like(metas[0]),
            "ws": s.ws if lane == 0 else torch.empty_like(s.ws),
        })

    def e2e_step(i):
        c = i % NL
        L = lanes[c]
        lb.apply_host(s.pool, tp0, 1 if sgmv else 0, xh[c], ybh[c], yh[c], sh, T, wl.tile_m, wl.long_min,
                      L["x"], L["yb"], L["y"], L["sidx"], L["meta"], L["ws"], L["stream"])

    def e2e_run(n):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for i in range(n):
            e2e_step(i)
        for L in lanes:
            L["stream"].synchronize()
        return time.perf_counter() - t0

    e2e_run(8)
    # as many steps as make the region last 0.2 s, at least the number asked for
    Ke = all_ranks_max_int(max(Ke, int(np.ceil(0.2 / max(e2e_run(8) / 8, 1e-6)))))
    if world > 1:
        dist.barrier()
    e2e_s = max_over_ranks(e2e_run(Ke), dev)
    h2d = 2 * T * (d_in0 + d_out0) + 4 * T
    d2h = 2 * T * d_out0

    if rank != 0:
        s.close()
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    alg_calls = [algorithmic_bytes(wl, wl.calls[j]) for j in range(calls_per_step)]
    # an input shared by several projections of a launch is counted once
    alg = sum(alg_calls) - sum(2 * T * wl.targets[wl.calls[j]][0]
                               for j in range(calls_per_step) if (j % 7) in share)
    achieved = alg / launches_per_step / (apply_ms * 1e-3) / 1e9
    fused = tuning.get(0) != 1
    line = {
        "metric": METRIC, "value": whole_job_value(world, T, K, ms), "unit": UNIT, "n_gpus": world,
        "steps": K_req, "steps_timed": K, "warmup": args.warmup, "ms_per_step": ms / K,
        "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "accumulate": "fp32",
        "data": "synthetic",
        "config": {
            "workload": workload_text(cfg, wl),
            "step": "lora_build_segments + %s, one %s" % (
                "%d x lora_sgmv_apply" % calls_per_step if sgmv else
                "%d x lora_bgmv_apply (grouped)" % calls_per_step if launches_multi is None else
                "%d x lora_bgmv_apply_multi (%d projections; %s; q/k/v and gate/up share their input)" % (
                    launches_per_step, calls_per_step,
                    "one launch per layer" if multi == "layer" else "{q,k,v} {o} {gate,up} {down} per launch"),
                "layer step" if cfg != 4 else "32-layer step (tokens/s per layer step = value x 32)"),
            "cache": ("cold: %d rotating input/weight sets (%.0f MB touched per rotation, L2 is 126 MB)"
                      % (n_sets, n_sets * alg / 1e6)) if n_sets > 1 else
                     "cold: one step touches %.0f MB, more than the 126 MB L2" % (alg / 1e6),
            "launch": "CUDA graph of %d consecutive step(s); every timed region is whole replays of a "
                      "graph already replayed three times, repeated for at least %.0f ms" % (n_sets, MIN_REGION_MS),
            "multi_gpu": "independent replicas, no collective",
        },
        "roofline": {
            "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "peak_source": "%s copy bandwidth" % peak_kind,
            "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
            "kernel": ("shrink_kernel + expand_kernel (two launches per apply)" if not fused
                       else "tc_shrink_kernel + tc_expand_kernel + stream_kernel (one apply; tc_expand dominates)"
                       if cfg == 2 else "stream_kernel (one launch per apply, every rank)" if cfg == 3
                       else "decode_kernel (one launch per %s)" % ("apply" if launches_multi is None else
                                                                    "layer" if multi == "layer" else "group of projections")),
            "algorithmic_bytes_per_launch": alg / launches_per_step,
            "us_per_launch": apply_ms * 1e3, "traffic": NCU_TRAFFIC.get((4, multi) if cfg == 4 else cfg) if fused else None,
            "averaged_over": "%d launches per step" % launches_per_step,
            "warm_l2_us_per_launch": warm_us,
        },
        "step_GBps": alg / (ms / K * 1e-3) / 1e9,
        "e2e": {"value": whole_job_value(world, T, Ke, e2e_s * 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "api": "lora_apply_host (first projection of the step), %d streams used in turn" % NL,
                "steps": Ke},
        "gpu_launches": int(launches),
        "device_status_words": status_words,
        "clocks": clocks,
        "paper_context": PAPER_CONTEXT,
    }
    if status_words[1] != 0:
        line["invalid"] = "a bounded device-side wait expired during the run (status word 1 = %d)" % status_words[1]
    if swap is not None:
        line["swap_in"] = swap
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = {k: v for k, v in time_oracle(wl).items()
                                if k not in ("ms_per_step", "reps")}
    print(json.dumps(line))
    s.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
