"""The multi-GPU path of the benchmark shards requests across ranks with no collective on the data
path; the only exchange is the maximum of the per-rank timings.  Checked here with two gloo ranks
on the CPU: every rank draws its own batch of the same shape, and the reduced time is the slowest
rank's."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2605_02218_b200 import workloads


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    seed = bench.rank_seed("c1", rank)
    wl = workloads.make_config("c1", seed=seed, n_vis=64, n_txt=4, d=32, keep=8)
    per_rank_ms = [1.0 + rank, 10.0 - rank]
    reduced = bench.reduce_max(per_rank_ms, dist, torch.device("cpu"))
    out.put((rank, seed, float(wl.X.float().sum()), tuple(wl.X.shape), reduced))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_by_seed_and_reduce_max():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, sum0, shape0, red0), (r1, s1, sum1, shape1, red1) = got
    assert s0 != s1 and shape0 == shape1          # same shape, different contents
    assert sum0 != sum1
    assert red0 == red1 == [2.0, 10.0]            # max over ranks of each timing


def test_single_process_reduce_is_identity():
    assert bench.reduce_max([3.0, 4.0], None, torch.device("cpu")) == [3.0, 4.0]
