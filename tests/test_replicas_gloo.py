"""The multi-GPU protocol of bench.py (replicas, max-over-ranks timing, summed tokens) on two CPU
ranks over gloo."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2604_26881_b200 import replicas
from paper_2604_26881_b200 import workloads as W


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # every rank draws its own batch
        wl = W.WORKLOADS["tiny"]
        x, tenant, _ = W.make_tokens(wl, seed=replicas.rank_seed(0, rank))
        checksum = float(x.to(torch.float64).sum())
        replicas.barrier(world)
        ms = 10.0 * (rank + 1)                  # rank 1 is the slow one
        value, ms_step = replicas.aggregate_throughput(x.shape[0], 5, ms, world)
        mx = replicas.max_over_ranks([ms, 100.0 - ms], world)
        total = replicas.sum_over_ranks(1.0 + rank, world)
        replicas.barrier(world)
        out[rank] = (checksum, value, ms_step, mx, total)
    finally:
        dist.destroy_process_group()


def test_two_ranks_aggregate_like_the_benchmark():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    assert r0[0] != r1[0]                                   # different batches per rank
    # 2 ranks x 64 tokens x 5 steps over the slowest rank's 20 ms
    assert abs(r0[1] - 2 * 64 * 5 / 20e-3) < 1e-6 and r0[1] == r1[1]
    assert r0[2] == 4.0 and r1[2] == 4.0
    assert r0[3] == [20.0, 90.0] and r1[3] == [20.0, 90.0]
    assert r0[4] == 3.0 and r1[4] == 3.0


def test_single_rank_needs_no_process_group():
    assert replicas.max_over_ranks([1.5, 2.5], 1) == [1.5, 2.5]
    v, ms = replicas.aggregate_throughput(32, 10, 2.0, 1)
    assert abs(v - 32 * 10 / 2e-3) < 1e-9 and ms == 0.2
