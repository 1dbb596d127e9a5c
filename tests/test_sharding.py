"""Multi-rank host logic on CPU: two gloo ranks run the library's sharded solve
(``sharding.solve_sharded``, with the oracle standing in for the device) and the
gathered arrays equal the full-batch solution on every rank."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_shard_range_partitions_the_batch():
    from paper_2407_14843_b200.sharding import shard_range
    for n in (0, 1, 7, 64, 86400):
        for world in (1, 2, 3, 8):
            spans = [shard_range(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard_range(4, 2, 2)


def _worker(rank, world, port, n_total, ret):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2407_14843_b200 import workloads
        from paper_2407_14843_b200.sharding import solve_sharded
        import oracle
        wl = workloads.make_workload(2, n_total)
        # the library's sharded solve with the oracle standing in for the device
        full = solve_sharded(wl, lambda block: oracle.solve_batch(block, n_threads=1))
        ret[rank] = {k: v.numpy() for k, v in full.items()}
    finally:
        dist.destroy_process_group()


def test_two_rank_gather_equals_full_batch(oracle_mod):
    from paper_2407_14843_b200 import workloads
    n_total, world = 37, 2          # odd: the shards differ in size
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    ret = ctx.Manager().dict()
    procs = [ctx.Process(target=_worker, args=(r, world, port, n_total, ret)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    ref = oracle_mod.solve_batch(workloads.make_workload(2, n_total))
    for r in range(world):
        for k in ("h", "c", "b", "total_cost", "latency_buckets", "status"):
            assert np.array_equal(ret[r][k], ref[k]), (r, k)
