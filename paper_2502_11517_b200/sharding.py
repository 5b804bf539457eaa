"""Multi-GPU use of the path: requests are independent, so ranks share nothing but the final numbers.

Each rank owns a pool on its own GPU and a contiguous block of the requests; no collective touches K, V,
queries or outputs.  The only communication is the reduction of the benchmark's counters.
"""
from __future__ import annotations

from typing import List, Tuple


def shard_range(n_items: int, rank: int, world: int) -> Tuple[int, int]:
    """[begin, end) of the items owned by `rank`: contiguous blocks whose sizes differ by at most one."""
    if not (0 <= rank < world) or n_items < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_items, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def shard_script_ops(ops: List[tuple], rank: int, world: int, n_requests: int):
    """The operations of a workload script that concern this rank's requests, with request ids renumbered
    from 0 so that each rank's pool hands out the ids the script expects."""
    begin, end = shard_range(n_requests, rank, world)
    out = []
    for op in ops:
        if op[0] == "step":
            entries = tuple((r - begin, t, n) for r, t, n in op[1] if begin <= r < end)
            if entries:
                out.append(("step", entries))
        elif begin <= op[1] < end:
            out.append((op[0], op[1] - begin) + tuple(op[2:]))
    return out


def aggregate(units: float, seconds: float, group=None) -> Tuple[float, float]:
    """(units processed by all ranks, slowest rank's time) — whole-job throughput is their ratio."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return units, seconds
    dev = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    total = torch.tensor([units], dtype=torch.float64, device=dev)
    worst = torch.tensor([seconds], dtype=torch.float64, device=dev)
    dist.all_reduce(total, op=dist.ReduceOp.SUM, group=group)
    dist.all_reduce(worst, op=dist.ReduceOp.MAX, group=group)
    return float(total.item()), float(worst.item())
