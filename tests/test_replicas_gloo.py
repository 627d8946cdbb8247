"""The multi-GPU path is "replicas only": ranks run independent sequences and the benchmark joins
their timings with one MAX reduction.  This runs that host logic on CPU with two gloo ranks."""
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
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 4.0 + 1.5 * rank                       # rank 1 is the slow replica
    slow = bench.slowest_rank_ms(local_ms, dist, "cpu")
    dist.barrier()
    out.put((rank, slow, bench.job_us_per_timestep(slow, 512, world)))
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_replica():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slow, us in got:
        assert slow == pytest.approx(5.5)                              # max over ranks, seen by both
        assert us == pytest.approx(5.5e3 / (512 * 2))                  # two replicas' timesteps per slowest time


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.slowest_rank_ms(3.25) == 3.25
    assert bench.job_us_per_timestep(4.0, 400, 1) == pytest.approx(10.0)
