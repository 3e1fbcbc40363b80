"""The multi-GPU path is independent replicas: bytes add up, the slowest rank sets the time.
Checked with two gloo ranks on CPU."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2405_11425_b200.pipeline import aggregate_throughput


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_bytes = 1000.0 * (rank + 1)          # rank 0: 1000 B, rank 1: 2000 B
        local_seconds = 2.0 if rank == 0 else 3.0
        dist.barrier()
        q.put((rank,) + aggregate_throughput(local_bytes, local_seconds))
    finally:
        dist.destroy_process_group()


def test_two_replicas_aggregate():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 3000.0, 3.0), (1, 3000.0, 3.0)]


def test_single_process_is_identity():
    assert aggregate_throughput(5.0, 2.0) == (5.0, 2.0)
