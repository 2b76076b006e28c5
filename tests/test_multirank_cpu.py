"""The N > 1 path of the benchmark is "replicas only": no data-path collective, one max-reduction of
the per-rank step time.  Covered here with two gloo ranks on the CPU."""
import os
import sys

import pytest
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
    ms_local = 2.0 + 3.0 * rank            # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local)
    value = bench.whole_job_gbs(10 ** 9, ms, world)
    dist.barrier()
    out[rank] = (ms, value)
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_whole_job_rate():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        ms, value = res[rank]
        assert ms == 5.0                                   # max over ranks, on every rank
        assert value == pytest.approx(2 * 1e9 / 5e-3 / 1e9)  # both replicas' bytes over the slowest time


def test_single_process_is_its_own_maximum():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.25) == 1.25
    assert bench.whole_job_gbs(2 * 10 ** 9, 1.0, 1) == pytest.approx(2000.0)
