"""Multi-GPU sharding of the eviction path.

Units (sequence, KV head) never exchange data (every head of every sequence evicts on its own, Section 3), so
the path shards by sequence with no data-path collective. The only communication is the reduction of timings
for the benchmark: whole-job throughput = units processed by all ranks / max over ranks of the device time.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_range(n_seq: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous, balanced split of n_seq sequences: the first n_seq % world ranks get one more."""
    if not (0 <= rank < world):
        raise ValueError(f"rank {rank} outside world of {world}")
    base, extra = divmod(n_seq, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def job_throughput(units_local: float, seconds_local: float, device="cpu", group=None) -> tuple[float, float, float]:
    """(total units over ranks, max seconds over ranks, units/s of the whole job). Works without a process group."""
    vals = torch.tensor([units_local, seconds_local], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized():
        total = vals[:1].clone()
        worst = vals[1:].clone()
        dist.all_reduce(total, op=dist.ReduceOp.SUM, group=group)
        dist.all_reduce(worst, op=dist.ReduceOp.MAX, group=group)
        units, secs = float(total.item()), float(worst.item())
    else:
        units, secs = float(units_local), float(seconds_local)
    return units, secs, units / secs
