"""The N > 1 path of bench.py on CPU with gloo, world size 2: timing aggregation (max over ranks) and the
data-parallel gradient exchange (mean over ranks of the flat gradient buffer), the latter checked with the oracle:
the mean of the two half-batch gradients is the full-batch gradient (images are independent up to the batch mean)."""
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


def _dp_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import numpy as np
    import torch.distributed as dist
    import bench
    from oracle import bsr_oracle as O
    from paper_2405_10951_b200 import synth
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = synth.CONFIGS["tiny_fp32"].with_(trainable=(2, 3, 4, 5))
    images, labels, task_ids, params = synth.make_workload(cfg, peaked=True)        # the same on both ranks
    half = cfg.batch // world
    sl = slice(rank * half, (rank + 1) * half)
    mine = O.train_step(cfg, params, images[sl], labels[sl], task_ids[sl])           # this rank's share
    names = sorted(mine["grads"])
    flat = torch.tensor(np.concatenate([mine["grads"][n].ravel() for n in names]))
    bench.dp_average(dist, world, flat)
    if rank == 0:
        full = O.train_step(cfg, params, images, labels, task_ids)
        want = np.concatenate([full["grads"][n].ravel() for n in names])
        out.put(float(np.abs(flat.numpy() - want).max() / np.abs(want).max()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_average_their_gradients_into_the_full_batch_gradient():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_dp_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    err = out.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert err < 1e-12
