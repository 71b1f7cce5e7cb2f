"""The multi-GPU leg of bench.py on CPU: two gloo ranks, no data-path collective (replicas only),
the timed region's duration is the maximum over the ranks and the reported value is the whole
job's (world x one replica's work / the slowest rank's time)."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    local_ms = 10.0 + 5.0 * rank            # rank 1 is the slow one
    dist.barrier()
    total = bench.max_over_ranks_ms(local_ms)
    out[rank] = (total, bench.whole_job_tops(2.0e12, world, total / 4))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_whole_job():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in range(world):
        total, tops = res[rank]
        assert total == pytest.approx(15.0)                     # max over ranks, on every rank
        assert tops == pytest.approx(2 * 2.0e12 / (15.0 / 4 * 1e-3) / 1e12)


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks_ms(3.25) == 3.25
    assert bench.whole_job_tops(1e12, 1, 1.0) == pytest.approx(1000.0)
