"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own batch (weak scaling, no
data-path collective); the slowest rank defines the step time and the rate counts every rank's images."""
import os
import socket
import sys

import pytest
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
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 1 is the slow one
    ms_total, ms_e2e = bench.reduce_max([10.0 + 5.0 * rank, 20.0 - 3.0 * rank], dist, "cpu")
    dist.barrier()
    out[rank] = (ms_total, ms_e2e, bench.whole_job_rate(64, world, 5, ms_total))
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_count_all_images():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms_total, ms_e2e, rate = res[0]
    assert ms_total == 15.0 and ms_e2e == 20.0
    assert rate == pytest.approx(64 * 2 * 5 / 15e-3)


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max([3.0, 4.0], None, "cpu") == [3.0, 4.0]
    assert bench.whole_job_rate(64, 1, 10, 20.0) == pytest.approx(32000.0)
