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


def _dp_worker(rank, world, port, out):
    """One data-parallel rank: compresses its own gradients with the shared seeds (CPU oracle), then exchanges sketches."""
    import numpy as np
    from oracle import flora_oracle as orc
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        shapes, r = [(24, 40), (7, 96), (33, 12)], 8
        sketches = []
        for i, (n, m) in enumerate(shapes):
            G = np.random.default_rng(100 * rank + i).standard_normal((n, m)).astype(np.float32)
            C = np.zeros((n, r), dtype=np.float32)
            orc.compress_accumulate(G, orc.projection(50 + i, r, m, "f32"), C)
            sketches.append(torch.from_numpy(C))
        replicas.allreduce_sketches(sketches, dist, bucket_bytes=1500)       # small buckets: several collectives
        out.put((rank, [s.numpy().copy() for s in sketches]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_allreduce_of_sketches_equals_the_sketch_of_the_summed_gradient():
    """Linearity of the compression (Section 2.2): what two ranks get by summing their sketches is the sketch of the
    sum of their gradients, so the exchange step may carry n x r instead of n x m values."""
    import numpy as np
    from oracle import flora_oracle as orc
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_dp_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = dict(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    shapes, r = [(24, 40), (7, 96), (33, 12)], 8
    for i, (n, m) in enumerate(shapes):
        total = sum(np.random.default_rng(100 * rank + i).standard_normal((n, m)).astype(np.float64) for rank in range(2))
        want = total @ orc.projection(50 + i, r, m, "f32").astype(np.float64).T
        for rank in range(2):
            assert np.array_equal(results[rank][i], results[0][i])          # every rank holds the same sum
            assert np.abs(results[rank][i] - want).max() <= 1e-5 * np.abs(want).max()
    sk = [torch.ones(3, 2)]
    replicas.allreduce_sketches(sk, None)                                    # no process group: nothing happens
    assert torch.equal(sk[0], torch.ones(3, 2))
