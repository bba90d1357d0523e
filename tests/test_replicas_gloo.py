"""The N > 1 bookkeeping of bench.py (independent replicas: max of the times, sum of the bytes) with two gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2402_03293_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
        agg = replicas.aggregate_throughput(bytes_per_rank=2e9, steps=4, ms_this_rank=ms, dist=dist)
        out.put((rank, agg, replicas.max_over_ranks(float(rank), dist)))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_sum_of_bytes_over_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, agg, mx in results:
        assert agg["world"] == 2 and agg["ms"] == 15.0 and agg["ms_per_step"] == 3.75
        assert abs(agg["gbs"] - 2 * 2e9 * 4 / 15e-3 / 1e9) < 1e-9
        assert mx == 1.0


def test_single_process_is_identity():
    agg = replicas.aggregate_throughput(1e9, 2, 4.0)
    assert agg == {"world": 1, "ms": 4.0, "ms_per_step": 2.0, "gbs": 1e9 * 2 / 4e-3 / 1e9}
