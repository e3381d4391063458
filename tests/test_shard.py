"""Replica sharding over ranks, exercised with two gloo processes on the CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2412_00099_b200 import shard


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cpu = torch.device("cpu")
    lo, hi = shard.stream_range(257, rank, world)
    t_max = shard.reduce_max(10.0 + rank, cpu)           # slowest rank decides the time
    n = shard.reduce_sum(hi - lo, cpu)                   # counters add up
    out[rank] = (lo, hi, t_max, n, shard.replica_seed(1, rank))
    dist.destroy_process_group()


def test_two_rank_replicas():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    assert r0[0] == 0 and r0[1] == r1[0] and r1[1] == 257          # disjoint cover
    assert r0[2] == r1[2] == 11.0 and r0[3] == r1[3] == 257.0
    assert r0[4] == 1 and r1[4] != r0[4]


def test_single_process_passthrough():
    assert shard.reduce_max(3.5, None) == 3.5 and shard.reduce_sum(7, None) == 7.0
