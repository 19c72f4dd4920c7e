"""Host logic of the multi-GPU benchmark path (independent replicas, no collective on the data
path) on two CPU ranks over gloo: the timed value is the slowest rank's, every rank agrees on
it, and the reported throughput counts every replica's tokens."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = bench.rank_max(1.5 + rank, world, torch.device("cpu"))     # rank 1 is the slower one
        dist.barrier()
        out[rank] = (ms, bench.replicas_tokens_per_s(world, 65536, ms))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_sum_of_tokens():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, value = res[0]
    assert ms == 2.5
    assert abs(value - 2 * 65536 / 2.5e-3) < 1e-6


def test_single_rank_needs_no_process_group():
    assert bench.rank_max(3.25, 1, None) == 3.25
    assert bench.replicas_tokens_per_s(1, 1000, 2.0) == 500000.0
