"""The N > 1 path of bench.py is replicas only: every rank runs the same step and the job value
is the sum of the ranks' units over the slowest rank's time.  Checked here with two gloo ranks on
the CPU (no GPU, no NCCL)."""
from __future__ import annotations

import os
import socket
import sys

import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 0 takes 2 s for 10 units, rank 1 takes 4 s for 10 units
    value, slowest = bench.aggregate_over_ranks(10.0, 2.0 * (rank + 1), dist, None)
    q.put((rank, value, slowest))
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_two_gloo_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, slowest in got:
        assert slowest == 4.0 and value == 20.0 / 4.0


def test_single_rank_is_plain_ratio():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(30.0, 2.0) == (15.0, 2.0)
    assert bench.n_relax(18, 200) == 4_010_803_200 and bench.n_states(18, 200) == 471_859_200
    assert bench.n_relax(8, 24) == 86_016 and bench.n_relax(1, 5) == 0
