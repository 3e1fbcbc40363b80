"""The multi-GPU path is independent replicas: bytes add up, the slowest rank sets the time.
Checked with two gloo ranks on CPU."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import numpy as np

from paper_2405_11425_b200.binding import RRError, rr_finish_spread_ppm
from paper_2405_11425_b200.binding import rr_rebalance_weights as rebalanced_weights
from paper_2405_11425_b200.pipeline import (Groups, Reach, aggregate_throughput, load_calibration,
                                             save_calibration)


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


def test_rebalancing_moves_work_towards_groups_that_finished_early():
    # three groups with true capacities 2 : 1 : 1 given equal work: the first finishes in half
    # the time; one update makes the weights proportional to the capacities
    w = rebalanced_weights([100, 100, 100], [500, 1000, 1000])
    assert w.sum() in range(999_990, 1_000_010)
    assert abs(w[0] / w[1] - 2.0) < 1e-3 and w[1] == w[2]
    # a fixed point: work already proportional to capacity -> same finish -> same weights
    w2 = rebalanced_weights(w, [7000, 7000, 7000])
    assert np.abs(w.astype(np.int64) - w2.astype(np.int64)).max() <= 1
    # a group that never ran keeps a token weight, never zero
    w3 = rebalanced_weights([100, 100], [1000, 0])
    assert w3[1] >= 1 and w3[0] > 100 * w3[1]
    assert rr_finish_spread_ppm([1000, 980, 0]) == 20_000
    with pytest.raises(RRError):
        rebalanced_weights([1, 1], [0, 0])


def test_calibration_round_trip_is_bound_to_the_card(tmp_path):
    g = Groups(np.array([0, 0, 1, 1, 2, 2], np.uint16), 3, 47.0)
    r = Reach(True, 4600.0, 70 << 30, [(1 << 30, 5400.0)])
    path = tmp_path / "card.json"
    g.probe_stats = {"overlap_min": 0.985, "pairs_below_goal": 0, "reruns": 0, "relaunched": 0}
    save_calibration(path, "abc123", g, r, weights=[5, 6, 7],
                     extra={"region_bytes": 123 << 20, "weights_per_window": [1, 2, 3, 4, 5, 6]})
    g2, r2, w2 = load_calibration(path, "abc123", 6)
    assert np.array_equal(g2.group_of_sm, g.group_of_sm) and g2.n_groups == 3 and g2.sizes == [2, 2, 2]
    assert r2.cliff and r2.reach_bytes == 70 << 30 and list(w2) == [5, 6, 7]
    assert r2.sweep == [(1 << 30, 5400.0)] and g2.overlap_min == 0.985
    g3, r3, w3, extra = load_calibration(path, "abc123", 6, with_extra=True)
    assert extra["region_bytes"] == 123 << 20 and extra["weights_per_window"] == [1, 2, 3, 4, 5, 6]
    assert g3.probe_stats["pairs_below_goal"] == 0
    with pytest.raises(ValueError):
        load_calibration(path, "another-card", 6)
    with pytest.raises(ValueError):
        load_calibration(path, "abc123", 8)
