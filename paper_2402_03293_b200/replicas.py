"""Multi-GPU form of the measurement: independent replicas.

The path has no exchange step (every matrix, and every row of a matrix, is an independent unit), so N GPUs run
N copies of the same step and only timing information crosses ranks: the slowest rank's device time, and the
sum of the bytes all ranks processed.  These helpers hold that bookkeeping so that it can be tested with the
`gloo` backend on CPU.
"""
from __future__ import annotations

import torch


def max_over_ranks(value: float, dist=None, device: str = "cpu") -> float:
    """The largest `value` over all ranks (every rank gets it); identity without a process group."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(bytes_per_rank: float, steps: int, ms_this_rank: float, dist=None, device: str = "cpu") -> dict:
    """Whole-job GB/s of `steps` steps: bytes of all ranks over the slowest rank's time (weak scaling)."""
    world = dist.get_world_size() if (dist is not None and dist.is_initialized()) else 1
    ms = max_over_ranks(ms_this_rank, dist, device)
    return {"world": world, "ms": ms, "ms_per_step": ms / steps,
            "gbs": world * bytes_per_rank * steps / (ms * 1e-3) / 1e9}


def allreduce_sketches(sketches, dist=None, bucket_bytes: int = 256 << 20) -> None:
    """Data-parallel exchange step: sums the n x r sketches of all ranks in place (every rank gets the sum).

    Compression is linear in the gradient (C(G1 + G2) = C(G1) + C(G2) for one projection, Section 2.2), so ranks that
    hold different micro-batches and the same seeds can exchange their sketches instead of their n x m gradients:
    m / r times fewer bytes on the wire.  The sketches travel in buckets of at most `bucket_bytes` (one collective
    each), through whatever backend the process group has (NCCL between GPUs, gloo on CPU).  Identity without a
    process group.  This is plumbing around the library's calls, not part of them: the sum over ranks is the
    collective's, every rank then runs the same decompress-apply."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return
    group, size = [], 0

    def flush():
        nonlocal group, size
        if not group:
            return
        flat = torch.cat([s.reshape(-1) for s in group])
        dist.all_reduce(flat, op=dist.ReduceOp.SUM)
        offset = 0
        for s in group:
            s.copy_(flat[offset:offset + s.numel()].view_as(s))
            offset += s.numel()
        group, size = [], 0

    for s in sketches:
        nbytes = s.numel() * s.element_size()
        if group and size + nbytes > bucket_bytes:
            flush()
        group.append(s)
        size += nbytes
    flush()
