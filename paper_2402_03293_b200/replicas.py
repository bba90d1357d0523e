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
