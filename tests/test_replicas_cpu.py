"""The only multi-rank logic of the benchmark (replicas, max time over ranks, summed bytes) on two gloo ranks."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 10.0 * (rank + 1)            # rank 1 is the slow replica
        total_ms = bench.max_over_ranks(local_ms, torch.device("cpu"))
        value = bench.aggregate_gbs(n_elements=1 << 20, steps=5, world=world, total_ms=total_ms)
        out[rank] = (total_ms, value)
    finally:
        dist.destroy_process_group()


def test_two_replicas_take_the_slowest_rank_and_sum_the_bytes():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    total_ms, value = res[0]
    assert total_ms == 20.0
    assert value == pytest.approx(world * 4.0 * (1 << 20) * 5 / 20e-3 / 1e9)


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    assert bench.aggregate_gbs(1000, 2, 1, 1.0) == pytest.approx(4.0 * 1000 * 2 / 1e-3 / 1e9)
