"""The N > 1 path of the benchmark (independent replicas, max-over-ranks timing) on two gloo ranks."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2603_06588_b200 import replicas


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dist.barrier()
        mine = [0.010 * (rank + 1), 0.5 - 0.1 * rank]          # rank 1 is slower on the first, faster on the second
        got = replicas.max_over_ranks(mine, torch.device("cpu"))
        out[rank] = (got, replicas.replica_throughput(64, got[0], world))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_take_the_slowest_ranks_time():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mgr = mp.get_context("spawn").Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    for rank in (0, 1):
        got, thr = out[rank]
        assert got == [0.020, 0.5]
        assert abs(thr - 2 * 64 / 0.020) < 1e-9


def test_single_process_is_the_identity():
    assert replicas.max_over_ranks([1.5, 2.5], torch.device("cpu")) == [1.5, 2.5]
    assert replicas.replica_throughput(10, 2.0, 1) == 5.0
