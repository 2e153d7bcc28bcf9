"""The N > 1 path of the benchmark on CPU: two gloo ranks, each a replica with its own step time;
the job's time is the maximum over ranks and the job's rate counts both ranks' work."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_2607_01844_b200 import launch


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    assert launch.env_world() == (rank, rank, world)
    assert launch.init("gloo") == world
    launch.barrier()
    ms = launch.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow one
    rate = launch.job_throughput(3.0e12, ms, world)
    launch.barrier()
    out.put((rank, ms, rate))
    torch.distributed.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_time_and_the_summed_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, rate in res:
        assert ms == 15.0
        assert abs(rate - 2 * 3.0e12 / 15e-3) < 1e-3 * rate


def test_single_process_needs_no_process_group():
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert launch.env_world() == (0, 0, 1)
    assert launch.max_over_ranks(7.5) == 7.5
    assert launch.job_throughput(2.0, 1000.0, 1) == 2.0
