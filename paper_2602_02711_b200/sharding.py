"""Host-side helpers for running the path on several GPUs (one process per GPU).

The path partitions by rows of X (independent agent steps / tokens): every rank holds the full
weights and its own rows, and there is no exchange step, so the only collectives are the barrier
and the max/sum reductions of the timing harness.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_range(total: int, rank: int, world: int):
    """Contiguous, near-equal split of range(total): returns (begin, end) of this rank's part."""
    if world < 1 or not 0 <= rank < world or total < 0:
        raise ValueError("bad shard arguments")
    base, extra = divmod(total, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def is_distributed() -> bool:
    return dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1


def barrier():
    if is_distributed():
        dist.barrier()


def _reduce(value: float, op, device) -> float:
    if not is_distributed():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, dist.ReduceOp.MAX, device)


def sum_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, dist.ReduceOp.SUM, device)


def job_throughput(units_this_rank: float, seconds_this_rank: float, device="cpu") -> float:
    """Whole-job throughput: units summed over ranks divided by the slowest rank's time."""
    total = sum_over_ranks(units_this_rank, device)
    t = max_over_ranks(seconds_this_rank, device)
    return total / t
