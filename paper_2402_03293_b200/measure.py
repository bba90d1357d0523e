"""Per-operation timings of the library on one of the named workloads.

    python -m paper_2402_03293_b200.measure gpt2_xl_set
    python -m paper_2402_03293_b200.measure single_bf16_4096x11008 --rank 128 --ops compress decompress

Each operation (compress-accumulate, momentum step, decompress-apply, resample transfer, and the resampling
momentum step that combines the last two) runs over the whole
weight set of the workload, back to back, with the inputs resident in device memory; the time is taken with
CUDA events around `--iters` launches after three warm-up launches.  Gradient sets rotate so that a launch
never finds its input in L2.  One JSON line per run: microseconds per launch and algorithmic GB/s
(compress: G read once, sketch read and written; decompress: W read and written, sketch read).

The same script, run with few iterations, is a convenient target for `ncu -k regex:<kernel>`.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as fb
from . import workloads as wl

OPS = ("compress", "momentum", "decompress", "transfer", "momentum_resampled")


def main() -> None:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("workload", choices=[n for n in wl.CONFIG_ORDER if wl.WORKLOADS[n].dtype == "bf16"])
    ap.add_argument("--rank", type=int, default=0, help="rank r of the sketch (default: the workload's)")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--ops", nargs="+", choices=OPS, default=list(OPS))
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise RuntimeError("needs a CUDA device: the Flora path has no CPU implementation")
    fb.load()
    w = wl.WORKLOADS[args.workload]
    r = args.rank or w.r
    dev = "cuda"
    count = len(w.shapes)
    n_sets = 4 if w.elements * 2 * 4 < 20e9 else 2          # rotating gradient sets, together larger than L2
    G = [[torch.randn(n, m, device=dev).mul_(w.grad_var ** 0.5).to(torch.bfloat16) for (n, m) in w.shapes] for _ in range(n_sets)]
    W = [torch.randn(n, m, device=dev).mul_(0.02).to(torch.bfloat16) for (n, m) in w.shapes]
    # the sketches start with unit-normal values: an operation timed alone then moves the same kind of data as after the
    # others (with all-zero sketches the tensor cores draw less power and the clock, and the figure, rise)
    C = [torch.randn(n, r, device=dev) for n, _ in w.shapes]
    sets = [fb.FloraSet(G[k], W, C) for k in range(n_sets)]
    seeds = fb.seed_array(list(range(1, count + 1)))
    new_seeds = fb.seed_array(list(range(1001, count + 1001)))
    state = sum(n * r * 4 for n, _ in w.shapes)
    compress_bytes = w.elements * 2 + 2 * state
    decompress_bytes = 2 * w.elements * 2 + state

    def timed(fn, iters):
        for i in range(3):
            fn(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters * 1e3            # microseconds

    out = {"workload": args.workload, "r": r, "matrices": count, "iters": args.iters}
    if "compress" in args.ops:
        t = timed(lambda i: sets[i % n_sets].compress_accumulate(seeds), args.iters)
        out["compress_us"], out["compress_gbs"] = round(t, 1), round(compress_bytes / t / 1e3)
    if "momentum" in args.ops:
        t = timed(lambda i: sets[i % n_sets].momentum_step(0.9, seeds), args.iters)
        out["momentum_us"], out["momentum_gbs"] = round(t, 1), round(compress_bytes / t / 1e3)
    if "decompress" in args.ops:
        t = timed(lambda i: sets[0].decompress_apply(seeds, 1e-4, 1.0), args.iters)
        out["decompress_us"], out["decompress_gbs"] = round(t, 1), round(decompress_bytes / t / 1e3)
    if "transfer" in args.ops:
        t = timed(lambda i: sets[0].resample_transfer(seeds, new_seeds), max(1, args.iters // 4))
        out["transfer_us"] = round(t, 1)
    if "momentum_resampled" in args.ops:
        t = timed(lambda i: sets[i % n_sets].momentum_step_resampled(0.9, seeds, new_seeds), max(1, args.iters // 4))
        out["momentum_resampled_us"] = round(t, 1)
    for s in sets:
        s.close()
    if fb.flora_device_status() != 0:
        raise RuntimeError("a device-side wait timed out")
    print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
