#!/usr/bin/env python
"""Benchmark of the Flora hot path on B200: gradient GB/s per Flora step.

The default workload is the GPT-2-XL-shaped weight set (48 x {1600x4800, 1600x1600, 1600x6400, 6400x1600}, bf16
gradients with 1 % outliers, r = 256, tau = 16, beta = 0.9): a step is one accumulation cycle of Algorithm 1 feeding
Algorithm 2 -- tau compressions C += G A_acc^T (a fresh gradient set each), M <- beta M + (1-beta)/tau C A_acc A_mom^T,
the update W -= lr M A_mom, and the reset of C.  `value` = gradient bytes consumed per step / device time of the step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl flora|reference] [--workload NAME] [--rank R]

Other workloads: an accumulation workload runs tau compressions + one decompress-apply per step; a momentum
workload runs one momentum step + one decompress-apply per step, with the momentum transfer at the steps
Algorithm 2 resamples at.  With N > 1 (launched by torch.distributed.run) every rank runs an independent replica of
the same work on its own GPU (the path has no exchange step); times are the max over ranks.
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

from paper_2402_03293_b200 import hostlogic  # noqa: E402
from paper_2402_03293_b200 import replicas  # noqa: E402
from paper_2402_03293_b200 import workloads as wl  # noqa: E402

DEFAULT_WORKLOAD = "gpt2_xl_set"
METRIC = "gradient GB/s per Flora step (compress+decompress-apply)"
LR = 1e-3
FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS = 6650.0, 1400.0
NOMINAL_HBM_GBS, NOMINAL_BF16_TFLOPS = 8000.0, 2250.0
MIN_TIMED_SECONDS = 1.5        # the K-step block is repeated until this much device time has been measured
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu captures summarised
# under profiles/ (absent = not captured since the kernel last changed).  The benchmark's weight set is too large for a
# multi-pass capture: the compression figure is the capture of the same kernel on one 4096 x 11008 matrix at r = 256
# (99.5 MB for 98.6 MB algorithmic, profiles/compress_pair_kernel_single_bf16_4096x11008_r256.md), scaled by the
# algorithmic bytes of this workload (traffic grows with the elements streamed: G is read once, C read and written once).
NCU_TRAFFIC = {("gpt2_xl_set", 256, "compress"): int(4050124800 * 99.52 / 98.57)}


# ------------------------------------------------------------------------------------------ helpers
def op_costs(w: wl.Workload, r: int):
    """Algorithmic bytes and flops of each operation over the weight set (A costs no bytes: it is regenerated)."""
    eb = w.elem_bytes
    state = sum(n * r * 4 for n, _ in w.shapes)
    flops = 2 * w.elements * r
    transfer_flops = sum(2 * r * r * m + 2 * n * r * r for n, m in w.shapes)
    return {
        "compress": (w.elements * eb + 2 * state, flops),                 # read G once, read + write the sketch
        "compress_first": (w.elements * eb + state, flops),               # the cycle's first: the sketch is only written
        "momentum": (w.elements * eb + 2 * state, flops),
        "decompress": (2 * w.elements * eb + state, flops),               # read + write W, read the sketch
        "transfer": (2 * state, transfer_flops),                          # read + write M
        "transfer_axpby": (3 * state, transfer_flops),                    # read C, read + write M
        "momentum_resampled": (w.elements * eb + 4 * state, flops + transfer_flops),
        "zero": (state, 0),
    }


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d["bf16_tflops_sustained"]), "measured (MEASURED_PEAKS.json: hbm_gbs, bf16_tflops_sustained)"
    except Exception:
        return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, "fallback (6.65 TB/s, 1.4 PFLOP/s sustained)"


def roofline_block(kernel: str, nbytes: int, flops: int, us: float, hbm: float, tf: float, source: str):
    """Roofline of one launch: the slower of its bytes at the HBM peak and its flops at the tensor peak."""
    t_hbm, t_tensor = nbytes / (hbm * 1e9) * 1e6, flops / (tf * 1e12) * 1e6
    nominal_us = max(nbytes / (NOMINAL_HBM_GBS * 1e9), flops / (NOMINAL_BF16_TFLOPS * 1e12)) * 1e6
    if t_hbm >= t_tensor:
        bound, achieved, peak, unit = "hbm", nbytes / us / 1e3, hbm, "GB/s"
    else:
        bound, achieved, peak, unit = "tensor", flops / us / 1e6, tf, "TFLOP/s"
    return {"bound": bound, "kernel": kernel, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
            "frac_of_nominal": nominal_us / us, "nominal": "8 TB/s HBM, 2.25 PFLOP/s dense bf16",
            "bytes_per_launch": nbytes, "flops_per_launch": flops, "us_per_launch": us, "hbm_side_us": t_hbm, "tensor_side_us": t_tensor,
            "peak_source": source}


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
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                power.append(float(r[2]))
                for name, flag in zip(names, r[3:7]):
                    if flag.lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "sm_mhz_min": min(sm) if sm else None, "power_w_max": max(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------ the step
class Rotating:
    """The set operations over a ring of gradient sets that share weights and sketches: every compression takes
    the next gradient set, so no launch finds its input in L2.  Marks the stream with an event whenever the kind
    of operation changes (the per-kernel durations of the roofline block come from these marks)."""

    def __init__(self, sets, host_sets=None):
        self.sets, self.host_sets, self.k = sets, host_sets, 0
        self._h = sets[0]._h
        self.marks = None           # list of (kind, event) while a timed block records
        self.counts = {}
        self.last = None

    def mark(self, kind):
        if self.marks is not None:
            self.counts[kind] = self.counts.get(kind, 0) + 1
            if kind != self.last:
                ev = torch.cuda.Event(enable_timing=True)
                ev.record()
                self.marks.append((kind, ev))
                self.last = kind

    def _next(self):
        s = self.sets[self.k % len(self.sets)]
        if self.host_sets is not None:          # end-to-end leg: this micro-step's gradients come from pinned host memory
            s.upload_gradients(self.host_sets[self.k % len(self.host_sets)])
        self.k += 1
        return s

    def compress_accumulate(self, seeds, stream=None):
        self.mark("compress")
        self._next().compress_accumulate(seeds, stream)

    def compress_overwrite(self, seeds, stream=None):
        self.mark("compress_first")
        self._next().compress_overwrite(seeds, stream)

    def momentum_step(self, beta, seeds, stream=None):
        self.mark("momentum")
        self._next().momentum_step(beta, seeds, stream)

    def momentum_step_resampled(self, beta, old, new, stream=None):
        self.mark("momentum_resampled")
        self._next().momentum_step_resampled(beta, old, new, stream)

    def resample_transfer(self, old, new, stream=None):
        self.mark("transfer")
        self.sets[0].resample_transfer(old, new, stream)

    def transfer_axpby_from(self, src, old, new, a, b, stream=None):
        self.mark("transfer_axpby")
        self.sets[0].transfer_axpby_from(src, old, new, a, b, stream)

    def decompress_apply(self, seeds, lr, scale, stream=None):
        self.mark("decompress")
        self.sets[0].decompress_apply(seeds, lr, scale, stream)

    def zero_state(self, stream=None):
        self.mark("zero")
        self.sets[0].zero_state(stream)


def make_stepper(w: wl.Workload, acc: Rotating, mom, count: int, base_seed: int, exchange=None):
    """One Flora step of the workload's mode as a closure, sequenced by the host classes of Algorithms 1 and 2."""
    if w.mode == "accumulate":
        cyc = hostlogic.AccumulationCycle(acc, count, w.tau, base_seed)

        def step():
            for _ in range(w.tau):
                cyc.accumulate()
            if exchange:
                exchange()
            cyc.apply(LR)
        return step, f"{w.tau} x compress (the first overwrites C, the others accumulate) + decompress_apply"
    if w.mode == "momentum":
        st = hostlogic.MomentumState(acc, count, w.beta, w.kappa, base_seed)
        n = [0]

        def step():
            # resampling at every step multiplies the state by about sqrt(m/r) each time: restart it every fourth step
            if w.kappa == 1 and n[0] % 4 == 0:
                acc.zero_state()
            st.step(LR)
            n[0] += 1
        what = "momentum_step + decompress_apply"
        what += (", with the transfer fused into every step (kappa = 1; M restarts from zero every 4th step)" if w.kappa == 1
                 else f"; resampling + transfer every {w.kappa} steps")
        return step, what
    both = hostlogic.AccumulatedMomentum(acc, mom, count, w.tau, w.beta, w.kappa, base_seed)

    def step():
        for _ in range(w.tau):
            both.accumulate()
        if exchange:
            exchange()
        both.apply(LR)
    return step, (f"{w.tau} x compress into C (the first overwrites, the others accumulate) + transfer_axpby "
                  f"(M <- beta M + (1-beta)/tau C A_acc A_mom^T) + decompress_apply of M; M resampled every {w.kappa} steps")


# ------------------------------------------------------------------------------------------ reference arm (CPU oracle)
class OracleSample:
    """The workload's step on a sample of rows of the first transformer block's matrices, on the CPU oracle."""

    def __init__(self, w: wl.Workload, r: int, rows: int, lr: float = LR):
        import numpy as np
        self.np, self.w, self.r, self.lr = np, w, r, lr
        block = 4 if "gpt2" in w.name else (7 if "t5" in w.name else 1)
        self.ids = list(range(min(block, len(w.shapes))))
        self.rows = [min(rows, w.shapes[i][0]) for i in self.ids]
        self.micro = max(1, w.tau)
        self.G = [[wl.as_numpy(wl.gradient(w, i, k))[:n].copy() for i, n in zip(self.ids, self.rows)] for k in range(min(self.micro, 2))]
        self.W = [wl.as_numpy(wl.weight(w, i, std=0.02))[:n].copy() for i, n in zip(self.ids, self.rows)]
        self.C = [np.zeros((n, r), dtype=np.float32) for n in self.rows]
        self.M = [np.zeros((n, r), dtype=np.float32) for n in self.rows]
        self.t = 0

    def grad_bytes(self):
        return self.micro * sum(n * self.w.shapes[i][1] for i, n in zip(self.ids, self.rows)) * self.w.elem_bytes

    def step(self):
        from oracle import flora_oracle as orc
        w, r, t = self.w, self.r, self.t
        t0 = time.perf_counter()
        for j, i in enumerate(self.ids):
            m = w.shapes[i][1]
            if w.mode == "accumulate":
                A = orc.projection(1000 * t + i, r, m, w.dtype)
                self.C[j][:] = 0
                for k in range(w.tau):
                    orc.compress_accumulate(self.G[k % len(self.G)][j], A, self.C[j])
                orc.decompress_apply(self.W[j], self.C[j], A, self.lr, 1.0 / w.tau)
            elif w.mode == "momentum":
                epoch = t // w.kappa if w.kappa else 0
                A = orc.projection(1000 * epoch + i, r, m, w.dtype)
                if w.kappa and t % w.kappa == 0 and t > 0:
                    if w.kappa == 1 and t % 4 == 0:
                        self.M[j][:] = 0
                    A_old = orc.projection(1000 * (epoch - 1) + i, r, m, w.dtype)
                    orc.momentum_step_resampled(self.G[0][j], A_old, A, w.beta, self.M[j])
                else:
                    orc.momentum_step(self.G[0][j], A, w.beta, self.M[j])
                orc.decompress_apply(self.W[j], self.M[j], A, self.lr, 1.0)
            else:
                A_acc = orc.projection(1000 * t + i, r, m, w.dtype)
                A_mom = orc.projection(7_000_000 + i, r, m, w.dtype)
                self.C[j][:] = 0
                for k in range(w.tau):
                    orc.compress_accumulate(self.G[k % len(self.G)][j], A_acc, self.C[j])
                orc.transfer_axpby(self.M[j], self.C[j], A_acc, A_mom, (1.0 - w.beta) / w.tau, w.beta)
                orc.decompress_apply(self.W[j], self.M[j], A_mom, self.lr, 1.0)
        self.t += 1
        return time.perf_counter() - t0

    def describe(self):
        names = ", ".join(f"{n} of {self.w.shapes[i][0]} rows of a {self.w.shapes[i][0]}x{self.w.shapes[i][1]} matrix" for i, n in zip(self.ids, self.rows))
        return f"the whole step on the first rows of one transformer block's matrices ({names}); GB/s is per row processed, so it extrapolates linearly"


def sample_parity(w: wl.Workload, r: int, fb, rows: int = 48) -> dict:
    """The first step of the workload on a few rows of one transformer block's matrices, on the GPU path and on the
    oracle (part of the cpu_baseline leg): normwise maximum error of the compressed state and of the weight update."""
    import numpy as np
    from oracle import flora_oracle as orc
    dev = "cuda"

    def to_gpu(a):                                   # stored bytes -> device tensor (bf16 travels as its bit patterns)
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16).copy()).to(dev).view(torch.bfloat16)
        return torch.from_numpy(a.copy()).to(dev)

    def vals(a):
        return (orc.bf16_bits_to_f32(a) if a.dtype == np.uint16 else a).astype(np.float64)

    def err(x, y):
        return float(np.max(np.abs(x - y)) / max(float(np.max(np.abs(y))), 1e-300))

    # a step size that makes the update about half as large as the weights, so that its error is not hidden below the
    # bf16 spacing of W (the benchmark's own step is far smaller): found from one oracle step with step size 1
    probe = OracleSample(w, r, rows, 1.0)
    before = [vals(x) for x in probe.W]
    probe.step()
    moved = max(float(np.max(np.abs(vals(x) - b))) for x, b in zip(probe.W, before))
    lr = 0.5 * max(float(np.max(np.abs(b))) for b in before) / max(moved, 1e-30)
    ref = OracleSample(w, r, rows, lr)
    G = [[to_gpu(g) for g in gs] for gs in ref.G]
    W0 = [vals(x) for x in ref.W]
    W = [to_gpu(x) for x in ref.W]
    C = [torch.full((n, r), float("nan"), device=dev) for n in ref.rows]      # a cycle's first compression overwrites
    M = [torch.zeros(n, r, device=dev) for n in ref.rows]
    ref.step()
    ids = ref.ids                                    # the oracle sample's seeds at t = 0 are the matrix numbers
    if w.mode == "accumulate":
        sets = [fb.FloraSet(G[0], W, C)]
        for k in range(w.tau):
            sets[0].rebind_gradients(G[k % len(G)])
            (sets[0].compress_overwrite if k == 0 else sets[0].compress_accumulate)(ids)
        sets[0].decompress_apply(ids, lr, 1.0 / w.tau)
        state, state_ref = C, ref.C
    elif w.mode == "momentum":
        sets = [fb.FloraSet(G[0], W, M)]
        sets[0].momentum_step(w.beta, ids)
        sets[0].decompress_apply(ids, lr, 1.0)
        state, state_ref = M, ref.M
    else:
        acc, mom = fb.FloraSet(G[0], None, C), fb.FloraSet(None, W, M)
        sets = [acc, mom]
        s_mom = [7_000_000 + i for i in ids]
        for k in range(w.tau):
            acc.rebind_gradients(G[k % len(G)])
            (acc.compress_overwrite if k == 0 else acc.compress_accumulate)(ids)
        mom.transfer_axpby_from(acc, ids, s_mom, (1.0 - w.beta) / w.tau, w.beta)
        mom.decompress_apply(s_mom, lr, 1.0)
        state, state_ref = M, ref.M
    torch.cuda.synchronize()
    e_state = max(err(s_.cpu().numpy().astype(np.float64), sr.astype(np.float64)) for s_, sr in zip(state, state_ref))
    e_upd = max(err(W[j].float().cpu().numpy().astype(np.float64) - W0[j], vals(ref.W[j]) - W0[j]) for j in range(len(ids)))
    for s_ in sets:
        s_.close()
    return {"state_max_rel_err": e_state, "weight_update_max_rel_err": e_upd, "tolerance": 2e-2, "step_size": lr,
            "what": f"first step on {rows} rows of each matrix of one transformer block: GPU path against the CPU oracle, "
                    "max |x - ref| / max |ref| of the compressed state and of W - W0, at a step size that moves the weights by half their size"}


def sized_oracle_sample(w: wl.Workload, r: int, seconds_per_step: float) -> OracleSample:
    """A sample whose step takes about `seconds_per_step` on this host (sized from a small probe)."""
    probe = OracleSample(w, r, 16)
    dt = probe.step()
    rows = int(max(8, min(max(n for n, _ in w.shapes), 16 * seconds_per_step / max(dt, 1e-4))))
    return OracleSample(w, r, rows)


def select_workload(args):
    w = wl.WORKLOADS[args.workload]
    r = args.rank or w.r
    return w, r


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import flora_oracle as orc
    w, r = select_workload(args)
    # the whole run (warm-up + steps) should end within about two minutes
    per_step = max(0.05, min(3.0, 120.0 / max(1, args.steps + args.warmup)))
    sample = sized_oracle_sample(w, r, per_step)
    for _ in range(args.warmup):
        sample.step()
    total_t = sum(sample.step() for _ in range(args.steps))
    value = sample.grad_bytes() * args.steps / total_t / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "r": r, "tau": w.tau, "mode": w.mode, "note": "CPU oracle on host cores, bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": orc.max_threads(), "kind": "oracle", "sample": sample.describe()},
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
    w, r = select_workload(args)
    if w.dtype != "bf16":
        raise RuntimeError("the benchmark runs the bf16 workloads; the fp32 single matrix is a parity case")
    count = len(w.shapes)
    grad_set_bytes = w.elements * w.elem_bytes
    # gradient sets that rotate: together far larger than the 126 MB L2 (at least 1 GB), at most tau of them
    n_sets = max(2, min(max(w.tau, 4), -(-(1 << 30) // grad_set_bytes)))
    if grad_set_bytes > (2 << 30):
        n_sets = 4
    G = [[wl.gradient(w, i, k, device=dev, base_seed=rank) for i in range(count)] for k in range(n_sets)]
    W = [wl.weight(w, i, device=dev, std=0.02) for i in range(count)]
    C = [torch.zeros(n, r, device=dev) for n, _ in w.shapes]
    both = w.mode == "accumulate+momentum"
    M = [torch.zeros(n, r, device=dev) for n, _ in w.shapes] if both else None
    sets = [fb.FloraSet(G[k], None if both else W, C) for k in range(n_sets)]
    mset = fb.FloraSet(None, W, M) if both else None
    acc = Rotating(sets)
    mom = Rotating([mset]) if both else None
    # --exchange sketches (N > 1, accumulation workloads): the ranks are data-parallel workers that hold different
    # micro-batches and the same seeds; they sum their sketches C over NCCL before the update (linearity, Section 2.2)
    exchange = None
    if args.exchange == "sketches" and dist and w.mode != "momentum":
        exchange = lambda: replicas.allreduce_sketches(C, dist)
    step, what = make_stepper(w, acc, mom, count, base_seed=17 + (0 if exchange else rank), exchange=exchange)
    if exchange:
        what += "; sketches summed over ranks (all-reduce of C) before the update"

    def begin_marks():
        for rot in (acc, mom):
            if rot is not None:
                rot.marks, rot.counts, rot.last = shared_marks, shared_counts, None

    def timed_block(k):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(k):
            step()
            end = torch.cuda.Event(enable_timing=True)
            end.record()
            shared_marks.append(("end", end))
            for rot in (acc, mom):
                if rot is not None:
                    rot.last = None
        e1.record()
        return e0, e1

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = fb.flora_launch_count()
    shared_marks, shared_counts = [], {}
    begin_marks()
    # K steps form a block; blocks repeat until enough device time has been measured; the median block is reported
    blocks, spent = [], 0.0
    while True:
        e0, e1 = timed_block(args.steps)
        barrier()
        blocks.append(e0.elapsed_time(e1))
        spent += blocks[-1] * 1e-3
        done = spent >= args.min_seconds or len(blocks) >= 200
        if dist:                        # all ranks stop together
            flag = torch.tensor([1.0 if done else 0.0], device=dev)
            dist.all_reduce(flag, op=dist.ReduceOp.MAX)
            done = bool(flag.item())
        if done:
            break
    launches_per_block = (fb.flora_launch_count() - launches0) // len(blocks)
    clocks = sampler.stop() if rank == 0 else None
    for rot in (acc, mom):
        if rot is not None:
            rot.marks = None
    if fb.flora_device_status() != 0:
        raise RuntimeError("a device-side wait timed out during the timed region")
    grad_bytes_step = (w.tau if w.mode != "momentum" else 1) * grad_set_bytes
    agg = replicas.aggregate_throughput(grad_bytes_step, args.steps, statistics.median(blocks), dist, dev)
    ms, value = agg["ms"], agg["gbs"]

    # per-operation durations from the marks recorded inside the timed blocks
    spent_ms, kinds = {}, {}
    for (k0, ev0), (_, ev1) in zip(shared_marks, shared_marks[1:]):
        if k0 != "end":
            spent_ms[k0] = spent_ms.get(k0, 0.0) + ev0.elapsed_time(ev1)
    for k, total in spent_ms.items():
        kinds[k] = 1e3 * total / shared_counts[k]                    # microseconds per launch group of that kind
    costs = op_costs(w, r)
    hbm, tf, src = measured_peaks()
    k1 = "compress_pair_kernel" if r > 64 else "compress_tc_kernel"
    k2 = "decompress_pair_kernel" if r > 128 else "decompress_tc_kernel"
    names = {"compress": k1 + " (C += G A^T), one launch over the weight set", "momentum": k1 + " as the momentum update",
             "compress_first": k1 + " (C <- G A^T, the first compression of a cycle)",
             "momentum_resampled": "gram + apply + compress kernels (Algorithm 2's resampling step)",
             "decompress": ("sketch_to_bf16_kernel + " if r > 64 else "") + k2 + " (W -= lr S A), one launch over the weight set",
             "transfer": "gram + apply kernels (M <- M A_old A_new^T)", "transfer_axpby": "gram + apply kernels (M <- beta M + a C A_acc A_mom^T)"}
    main_kind = "compress" if "compress" in kinds else ("momentum" if "momentum" in kinds else "momentum_resampled")
    roofline = roofline_block(names[main_kind], costs[main_kind][0], costs[main_kind][1], kinds[main_kind], hbm, tf, src)
    roofline["launches_per_step"] = shared_counts[main_kind] // (args.steps * len(blocks))
    roofline["traffic"] = NCU_TRAFFIC.get((w.name, r, main_kind))
    roofline["other_kernels"] = {k: roofline_block(names[k], costs[k][0], costs[k][1], us, hbm, tf, src) | {"traffic": NCU_TRAFFIC.get((w.name, r, k))}
                                 for k, us in kinds.items() if k in names and k != main_kind}
    step_bound_us = sum(max(costs[k][0] / (hbm * 1e9), costs[k][1] / (tf * 1e12)) * 1e6 * shared_counts[k] for k in kinds if k in costs) \
        / (args.steps * len(blocks))
    roofline["step_frac_of_roofline"] = step_bound_us / (1e3 * ms / args.steps)

    # end to end: every micro-step's gradients start in pinned host memory, the updated weights are read back
    e2e_steps = 2 if grad_bytes_step > (8 << 30) else max(1, min(args.steps, 3))
    n_host = min(n_sets, 2)
    hostG = [[g.cpu().pin_memory() for g in G[k]] for k in range(n_host)]
    hostW = [torch.empty(n, m, dtype=wl.torch_dtype(w.dtype)).pin_memory() for n, m in w.shapes]
    acc.host_sets = hostG
    wset = mset if both else sets[0]
    # the read-back of a step's weights runs on a second stream, so it shares the (full-duplex) link with the next
    # step's uploads; it must have finished before the next decompression overwrites the weights
    main_stream, side = torch.cuda.current_stream(), torch.cuda.Stream()
    updated, read_back = torch.cuda.Event(), torch.cuda.Event()
    read_back.record(side)

    def e2e_step():
        main_stream.wait_event(read_back)
        step()
        updated.record(main_stream)
        side.wait_event(updated)
        wset.read_weights_to_host(hostW, stream=side)
        read_back.record(side)

    e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    main_stream.wait_event(read_back)              # the last step's weights have arrived in host memory
    e1.record()
    barrier()
    acc.host_sets = None
    e2e_agg = replicas.aggregate_throughput(grad_bytes_step, e2e_steps, e0.elapsed_time(e1), dist, dev)
    e2e = {"value": e2e_agg["gbs"], "unit": "GB/s", "h2d_bytes_per_step": grad_bytes_step,
           "d2h_bytes_per_step": w.elements * w.elem_bytes, "steps": e2e_steps,
           "api": "flora_set_upload_gradients + the step's set calls + flora_set_read_weights_to_host, pinned host buffers"}

    cpu_baseline, parity = None, None
    if rank == 0 and world == 1:
        from oracle import flora_oracle as orc
        sample = sized_oracle_sample(w, r, 4.0)
        total_t, n_steps = 0.0, 0
        while total_t < 10.0 and n_steps < 6:
            total_t += sample.step()
            n_steps += 1
        cpu_baseline = {"value": sample.grad_bytes() * n_steps / total_t / 1e9, "unit": "GB/s", "cores": orc.max_threads(), "kind": "oracle",
                        "sample": f"{n_steps} step(s), {total_t:.1f} s wall: " + sample.describe()}
        parity = sample_parity(w, r, fb)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "matrices": count, "r": r, "tau": w.tau, "beta": w.beta, "kappa": w.kappa, "elements": w.elements,
                       "step": what,
                       "l2": f"inputs larger than L2: {n_sets} rotating gradient sets of {grad_set_bytes / 1e9:.2f} GB, a different one per compression",
                       "timed": f"{len(blocks)} block(s) of {args.steps} steps, {spent:.2f} s of device time; value is the median block",
                       "multi_gpu": "data-parallel ranks, all-reduce of the sketches" if exchange else "independent replicas, no collective"},
            "roofline": roofline, "cpu_baseline": cpu_baseline, "parity": parity, "e2e": e2e, "gpu_launches": int(launches_per_block), "clocks": clocks,
            "ms_x_mhz_per_step": (ms / args.steps) * clocks["sm_mhz"] if clocks and clocks.get("sm_mhz") else None,
        }
        print(json.dumps(line), flush=True)
    for s in sets:
        s.close()
    if mset:
        mset.close()
    if dist:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="flora", choices=["flora", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=[n for n in wl.CONFIG_ORDER if wl.WORKLOADS[n].dtype == "bf16"])
    ap.add_argument("--rank", type=int, default=0, help="rank r of the sketches (default: the workload's)")
    ap.add_argument("--exchange", default="none", choices=["none", "sketches"],
                    help="N > 1 only: none = independent replicas (default); sketches = data-parallel ranks that all-reduce C")
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_SECONDS,
                    help="repeat the block of --steps steps until this much device time has been measured (0: one block, e.g. under a profiler)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "flora" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_flora(args)


if __name__ == "__main__":
    main()
