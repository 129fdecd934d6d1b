"""The benchmark's N > 1 arithmetic on CPU: two gloo ranks, no exchange on the data path, the job's rate is the
sum of the ranks' work over the slowest rank's time."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    import torch.distributed as dist

    sys.path.insert(0, ROOT)
    import bench

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    # rank 1 is the slow one: 2 s for the same 10 units
    rate, elapsed = bench.whole_job_rate(10.0, 1.0 + rank, world, dist, None)
    out[rank] = (rate, elapsed)
    dist.barrier()
    dist.destroy_process_group()


def test_whole_job_rate_takes_the_slowest_rank():
    torch = pytest.importorskip("torch")
    import torch.multiprocessing as mp

    with mp.Manager() as mgr:
        out = mgr.dict()
        port = 29500 + os.getpid() % 2000
        mp.spawn(_rank, args=(2, port, out), nprocs=2, join=True)
        assert dict(out) == {0: (10.0, 2.0), 1: (10.0, 2.0)}  # 2 ranks x 10 units / 2 s


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.whole_job_rate(8.0, 2.0, 1) == (4.0, 2.0)
