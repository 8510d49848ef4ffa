"""The N > 1 path of the benchmark on CPU: two gloo ranks, replicas only (max-over-ranks time, summed units)."""
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
    from paper_2203_04738_b200.replicas import job_throughput, max_over_ranks
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    dist.barrier()
    worst = max_over_ranks(ms)
    out[rank] = (worst, job_throughput(2048 * 32, worst, world))
    dist.destroy_process_group()


def test_two_replicas_report_slowest_time_and_summed_units():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0
    assert abs(res[0][1] - 2 * 2048 * 32 / 15e-3) < 1e-6


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    from paper_2203_04738_b200.replicas import job_throughput, max_over_ranks
    assert max_over_ranks(3.5) == 3.5
    assert job_throughput(100, 10.0, 1) == 100 / 10e-3
