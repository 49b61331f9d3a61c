"""The N > 1 bookkeeping of bench.py (replicas only) on two gloo ranks, CPU only."""

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
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    t_ms, t_e2e = bench.max_over_ranks([100.0 + 50.0 * rank, 300.0 - 100.0 * rank])
    out[rank] = (t_ms, t_e2e, bench.job_throughput(world, 131072, t_ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_rank_and_whole_job_tokens():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    t_ms, t_e2e, value = res[0]
    assert t_ms == 150.0 and t_e2e == 300.0
    assert abs(value - 2 * 131072 / 0.150) < 1e-6


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.job_throughput(1, 1000, 500.0) == 2000.0
