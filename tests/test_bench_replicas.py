"""The multi-GPU path of bench.py is N independent replicas: no data-path collective, only the
max-over-ranks of the timings.  Exercised here with two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = [10.0 + 5.0 * rank, 30.0 - 7.0 * rank, 1.0]
        got = bench.max_over_ranks(mine, "cpu")
        if rank == 0:
            out.put(got)
    finally:
        dist.destroy_process_group()


def test_timings_are_the_maximum_over_replicas_and_throughput_adds_up():
    sys.path.insert(0, ROOT)
    import bench
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert got == [15.0, 30.0, 1.0]
    # two replicas, 7 tokens each per step, slowest replica 20 ms per step -> 700 tokens/s for the job
    assert abs(bench.aggregate_value(2, 7, 20.0) - 700.0) < 1e-9
