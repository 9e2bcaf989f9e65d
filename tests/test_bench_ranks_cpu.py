"""The N > 1 path of bench.py is 'replicas only': ranks run independently and only the timing is
aggregated (max time over ranks, units summed).  Exercised here with 2 gloo ranks on CPU."""
import os
import socket
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch
    import torch.distributed as dist
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 if rank == 0 else 25.0            # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, torch.device("cpu"))
    value = bench.whole_job_value(units_per_step=2.0, steps=100, ms=ms, world=world)
    out[rank] = (ms, value)
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_with_gloo():
    import torch.multiprocessing as mp
    mgr = mp.Manager()
    out = mgr.dict()
    port = _free_port()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert out[0] == out[1]
    ms, value = out[0]
    assert ms == 25.0                                  # slowest rank decides
    assert value == pytest.approx(2 * 2.0 * 100 / 0.025)


def test_single_rank_needs_no_process_group():
    import torch
    import bench
    assert bench.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    assert bench.whole_job_value(1.0, 10, 5.0, 1) == pytest.approx(10 / 0.005)
