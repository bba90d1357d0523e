#!/usr/bin/env python
"""Benchmark of the Flora hot path on B200: gradient GB/s per Flora step.

A step is one accumulation cycle of Algorithm 1 over the GPT-2-small-shaped weight set
(12 x {768x2304, 768x768, 768x3072, 3072x768}, bf16, r = 32): tau = 8 compressions
(C += G A^T, one fresh gradient set each), one decompress-apply (W -= lr/tau * C A) and the
reset of C.  `value` = gradient bytes consumed per step / device time of the step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl flora|reference]

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica of the
same work on its own GPU (the path has no exchange step); times are the max over ranks.
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

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2402_03293_b200 import replicas  # noqa: E402
from paper_2402_03293_b200 import workloads as wl  # noqa: E402

WORKLOAD = "gpt2_small_set"
METRIC = "gradient GB/s per Flora step (compress+decompress-apply)"
LR = 1e-3
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under profiles/
# (None once a kernel has changed since its counters were taken)
NCU_TRAFFIC_COMPRESS = 182438144
NCU_TRAFFIC_DECOMPRESS = 291994368


# ------------------------------------------------------------------------------------------ helpers
def algorithmic_bytes(w: wl.Workload):
    """Bytes each operation must move (A costs none: it is regenerated)."""
    eb = w.elem_bytes
    state = sum(n * w.r * 4 for n, _ in w.shapes)
    compress = w.elements * eb + 2 * state            # read G once, read + write C
    decompress = 2 * w.elements * eb + state          # read + write W, read C
    return compress, decompress


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s)"


class ClockSampler:
    """nvidia-smi clock / throttle samples while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                for name, flag in zip(names, r[3:7]):
                    if flag.lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------ reference arm
def oracle_sample_step(w: wl.Workload, layers: int, state):
    """One Flora step of the CPU oracle over the first `layers` transformer blocks (4 matrices each)."""
    from oracle import flora_oracle as orc
    import numpy as np
    count = 4 * layers
    if not state:
        state["G"] = [[wl.as_numpy(wl.gradient(w, i, k)) for i in range(count)] for k in range(w.tau)]
        state["W"] = [wl.as_numpy(wl.weight(w, i, std=0.02)) for i in range(count)]
        state["C"] = [np.zeros((w.shapes[i][0], w.r), dtype=np.float32) for i in range(count)]
        state["epoch"] = 0
    t0 = time.perf_counter()
    for i in range(count):
        n, m = w.shapes[i]
        A = orc.projection(1000 * state["epoch"] + i, w.r, m, w.dtype)
        state["C"][i][:] = 0
        for k in range(w.tau):
            orc.compress_accumulate(state["G"][k][i], A, state["C"][i])
        orc.decompress_apply(state["W"][i], state["C"][i], A, LR, 1.0 / w.tau)
    state["epoch"] += 1
    dt = time.perf_counter() - t0
    grad_bytes = w.tau * sum(n * m for n, m in w.shapes[:count]) * w.elem_bytes
    return dt, grad_bytes


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import flora_oracle as orc
    w = wl.WORKLOADS[WORKLOAD]
    layers = 4
    state = {}
    for _ in range(args.warmup):
        oracle_sample_step(w, layers, state)
    total_t, total_b = 0.0, 0
    for _ in range(args.steps):
        dt, b = oracle_sample_step(w, layers, state)
        total_t += dt
        total_b += b
    value = total_b / total_t / 1e9
    sample = f"each step: one full cycle (tau={w.tau} compress + 1 decompress-apply) over {layers} of 12 transformer blocks (4 matrices)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "r": w.r, "tau": w.tau, "matrices": 4 * layers, "note": "CPU oracle on host cores, bounded sample"},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": orc.max_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------ our arm
def run_flora(args):
    from paper_2402_03293_b200 import binding as fb

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the Flora path has no CPU implementation")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device(dev))

    def barrier():
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    fb.load()
    w = wl.WORKLOADS[WORKLOAD]
    count = len(w.shapes)
    # tau gradient sets (1.36 GB in total, far larger than the 126 MB L2), weights, sketches
    G = [[wl.gradient(w, i, k, device=dev, base_seed=rank) for i in range(count)] for k in range(w.tau)]
    W = [wl.weight(w, i, device=dev, std=0.02) for i in range(count)]
    C = [torch.zeros(n, w.r, device=dev) for n, _ in w.shapes]
    sets = [fb.FloraSet(G[k], W, C) for k in range(w.tau)]
    epoch = [0]

    def seeds():
        return fb.seed_array([fb.flora_derive_seed(17, i, epoch[0]) for i in range(count)])

    def step(marks=None):
        s = seeds()
        if marks is not None:
            marks[0].record()
        for k in range(w.tau):
            sets[k].compress_accumulate(s)
        if marks is not None:
            marks[1].record()
        sets[0].decompress_apply(s, LR, 1.0 / w.tau)
        if marks is not None:
            marks[2].record()
        sets[0].zero_state()
        epoch[0] += 1

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = fb.flora_launch_count()
    # three event marks per step inside the timed region: before the compressions, between them and the
    # decompression, after it (per-kernel durations for the roofline block come from these)
    marks = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        step(marks[i])
    e1.record()
    barrier()
    launches = fb.flora_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    if fb.flora_device_status() != 0:
        raise RuntimeError("a device-side wait timed out during the timed region")
    grad_bytes_step = w.tau * w.elements * w.elem_bytes
    agg = replicas.aggregate_throughput(grad_bytes_step, args.steps, e0.elapsed_time(e1), dist, dev)
    ms, value = agg["ms"], agg["gbs"]

    comp_bytes, dec_bytes = algorithmic_bytes(w)
    c_avg = sum(m[0].elapsed_time(m[1]) for m in marks) / (args.steps * w.tau)     # ms per compress launch
    d_avg = sum(m[1].elapsed_time(m[2]) for m in marks) / args.steps              # ms per decompress launch
    peak, peak_src = measured_peak()
    comp_gbs, dec_gbs = comp_bytes / (c_avg * 1e-3) / 1e9, dec_bytes / (d_avg * 1e-3) / 1e9
    step_roof_ms = (w.tau * comp_bytes + dec_bytes) / (peak * 1e9) * 1e3
    roofline = {"bound": "hbm", "kernel": "compress_tc_kernel (C += G A^T), one launch over the weight set, 8 launches per step",
                "achieved": comp_gbs, "peak": peak, "unit": "GB/s", "frac": comp_gbs / peak, "traffic": NCU_TRAFFIC_COMPRESS,
                "peak_source": peak_src, "bytes_per_launch": comp_bytes, "us_per_launch": 1e3 * c_avg,
                "decompress_apply": {"kernel": "decompress_tc_kernel", "achieved": dec_gbs, "frac": dec_gbs / peak,
                                     "bytes_per_launch": dec_bytes, "us_per_launch": 1e3 * d_avg, "traffic": NCU_TRAFFIC_DECOMPRESS},
                "step_frac_of_roofline": step_roof_ms / (ms / args.steps)}

    # end to end: gradients start in pinned host memory, the updated weights are read back
    e2e = None
    e2e_steps = max(1, min(args.steps, 3))
    hostG = [[g.cpu().pin_memory() for g in G[k]] for k in range(w.tau)]
    hostW = [torch.empty(n, m, dtype=wl.torch_dtype(w.dtype)).pin_memory() for n, m in w.shapes]

    # the read-back of a step's weights runs on a second stream, so it shares the (full-duplex) link with the next
    # step's uploads; it must have finished before the next decompression overwrites the weights
    main, side = torch.cuda.current_stream(), torch.cuda.Stream()
    updated, read_back = torch.cuda.Event(), torch.cuda.Event()
    read_back.record(side)

    def e2e_step():
        s = seeds()
        for k in range(w.tau):
            sets[k].compress_accumulate_from_host(hostG[k], s)
        main.wait_event(read_back)
        sets[0].decompress_apply(s, LR, 1.0 / w.tau)
        updated.record(main)
        side.wait_event(updated)
        sets[0].read_weights_to_host(hostW, stream=side)
        read_back.record(side)
        sets[0].zero_state()
        epoch[0] += 1

    e2e_step()
    barrier()
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    main.wait_event(read_back)              # the last step's weights have arrived in host memory
    e1.record()
    barrier()
    e2e_agg = replicas.aggregate_throughput(grad_bytes_step, e2e_steps, e0.elapsed_time(e1), dist, dev)
    e2e = {"value": e2e_agg["gbs"], "unit": "GB/s",
           "h2d_bytes_per_step": grad_bytes_step, "d2h_bytes_per_step": w.elements * w.elem_bytes, "steps": e2e_steps}

    cpu_baseline = None
    if rank == 0 and world == 1:
        from oracle import flora_oracle as orc
        state = {}
        dt, b = oracle_sample_step(w, 12, state)
        cycles = 1
        while dt < 10.0 and cycles < 12:                       # about 10 s of oracle work, whole cycles only
            dt2, b2 = oracle_sample_step(w, 12, state)
            dt, b, cycles = dt + dt2, b + b2, cycles + 1
        cpu_baseline = {"value": b / dt / 1e9, "unit": "GB/s", "cores": orc.max_threads(), "kind": "oracle",
                        "sample": f"{cycles} full cycle(s) (tau={w.tau} compress + decompress-apply) over all 48 matrices, {dt:.1f} s wall"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "matrices": count, "r": w.r, "tau": w.tau, "elements": w.elements,
                       "step": "8 x compress_accumulate + decompress_apply + zero C",
                       "l2": "inputs larger than L2: 8 rotating gradient sets, 1.36 GB per step",
                       "multi_gpu": "independent replicas, no collective"},
            "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
        }
        print(json.dumps(line), flush=True)
    for s in sets:
        s.close()
    if dist:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="flora", choices=["flora", "reference"])
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "flora" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_flora(args)


if __name__ == "__main__":
    main()
