"""The multi-rank bookkeeping of bench.py on CPU: two gloo ranks, no GPU.

The path shards nothing across GPUs (units are independent: N replicas), so the only
cross-rank logic is the max over ranks of the timings and the whole-job sum of units.
"""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench

    mine = [10.0 + rank, 2.0 - rank, 5.0, 7.0 * (rank + 1)]
    got = bench.aggregate_over_ranks(mine, world, torch.device("cpu"), dist)
    if rank == 0:
        out.put(got)
    dist.barrier()
    dist.destroy_process_group()


def test_timings_are_max_over_ranks_and_value_sums_replicas():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    assert out.get() == [11.0, 2.0, 5.0, 14.0]
    sys.path.insert(0, ROOT)
    import bench

    one = bench.whole_job_value(256, 8, 256, 5, 1, 100.0)
    two = bench.whole_job_value(256, 8, 256, 5, 2, 100.0)
    assert two == 2 * one == 2 * 256 * 8 * 256 * 5 / 0.1
    assert bench.decode_bytes_per_unit_step(410, 128, 2) == 2 * 410 * 256 + 20 * 410 + 6 * 256
