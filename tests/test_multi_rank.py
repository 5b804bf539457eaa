"""Two ranks on CPU (gloo): requests are split between the ranks, each rank replays its share on its own
(host-only) pool, bit-exact against the oracle's model, and only the counters are reduced."""
import os
import socket
import sys

import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, results):
    sys.path.insert(0, ROOT); sys.path.insert(0, os.path.join(ROOT, "tests"))
    import copy
    import torch.distributed as dist
    from oracle import OracleReplay
    from paper_2502_11517_b200 import build
    from paper_2502_11517_b200.sharding import aggregate, shard_range, shard_script_ops
    from pasta_workloads import cfg3_batched
    from lib_replay import LibReplay, make_pool
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    build()
    script = cfg3_batched(9, 1, prefix_range=(40, 200))
    n_req = 9
    mine = copy.copy(script)
    mine.ops = shard_script_ops(script.ops, rank, world, n_req)
    pool = make_pool(mine, host_only=True)
    lib = LibReplay(mine, pool)
    ora = OracleReplay(mine, with_kv=False)
    for i, op in enumerate(mine.ops):
        lib.apply(i)
        if op[0] == "step":
            ora.model.reserve(op[1]); ora.next_op += 1
        else:
            ora.apply(i)
    assert pool.dump() == ora.model.dump()
    begin, end = shard_range(n_req, rank, world)
    queries = len(mine.ops[-1][1])
    total, worst = aggregate(float(queries), 1.0 + rank)
    results[rank] = (begin, end, queries, total, worst, len(script.ops[-1][1]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_split_requests_and_reduce_counters():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        results = mgr.dict()
        mp.spawn(_worker, args=(world, port, results), nprocs=world, join=True)
        r0, r1 = results[0], results[1]
    assert (r0[0], r0[1], r1[0], r1[1]) == (0, 5, 5, 9)           # contiguous, disjoint, covering
    assert r0[2] + r1[2] == r0[5] == r1[5]                         # every query belongs to exactly one rank
    assert r0[3] == r1[3] == r0[2] + r1[2] and r0[4] == r1[4] == 2.0   # sum of units, slowest rank's time


def test_shard_ranges_partition_any_count():
    sys.path.insert(0, ROOT)
    from paper_2502_11517_b200.sharding import shard_range
    for n in (0, 1, 7, 8, 64, 257):
        for world in (1, 2, 3, 8):
            cuts = [shard_range(n, r, world) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
            sizes = [e - b for b, e in cuts]
            assert max(sizes) - min(sizes) <= 1
