"""The N > 1 path of bench.py on CPU: two gloo ranks, max-over-ranks timing and the whole-job
aggregate of independent replicas (the path shards with no collective; only the timing is reduced)."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = [10.0, 25.0][rank]                       # rank 1 is the slow one
        dist.barrier()
        slow = bench.reduce_max_over_ranks(ms, dist, "cpu")
        value = bench.whole_job_value(1e9, world, slow, 1e9)
        out.put((rank, slow, value))
    finally:
        dist.destroy_process_group()


def test_two_rank_timing_and_aggregate():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slow, value in got:
        assert slow == 25.0                              # every rank sees the slowest rank's time
        assert value == pytest.approx(2 * 1e9 / 25e-3 / 1e9)   # 2 replicas of 1 GB in 25 ms = 80 GB/s


def test_single_rank_is_identity():
    assert bench.reduce_max_over_ranks(3.5, None, "cpu") == 3.5
    assert bench.whole_job_value(8e9, 1, 1000.0, 1e9) == pytest.approx(8.0)
