"""The N > 1 path of bench.py (independent replicas, time = max over ranks) on CPU with gloo, world size 2."""
import os
import socket
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, values = bench.aggregate(dist, world, 128, 10, [50.0 + 20.0 * rank, 70.0 - 5.0 * rank])
    dist.barrier()
    if rank == 0:
        out.put((ms, values))
    dist.destroy_process_group()


def test_two_ranks_report_max_time_and_whole_job_throughput():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ms, values = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ms == [70.0, 70.0]                                     # slowest rank of each measurement
    assert abs(values[0] - 2 * 128 * 10 / 0.070) < 1e-6           # images of both replicas over that time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    ms, values = bench.aggregate(None, 1, 64, 5, [25.0])
    assert ms == [25.0] and abs(values[0] - 64 * 5 / 0.025) < 1e-9
