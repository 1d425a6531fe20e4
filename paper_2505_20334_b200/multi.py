"""Host-side helpers for running the eviction step on several GPUs of one node.

The (layer, batch, KV head) units are independent (Section 4.3: Eq. 4 is evaluated per head), so a
multi-GPU job needs no data-path collective: every rank evicts its own shard and only the timing
is reduced. These helpers hold that logic so that it can be tested with the ``gloo`` backend on CPU.
"""
from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist


def shard_units(n_units: int, world_size: int, rank: int) -> Tuple[int, int]:
    """Contiguous, balanced [begin, end) range of unit numbers owned by `rank` (sizes differ by at
    most one; ranks beyond the number of units get an empty range)."""
    if world_size < 1 or not 0 <= rank < world_size:
        raise ValueError("bad rank / world size")
    base, extra = divmod(n_units, world_size)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: MAX all-reduce over the default process group (a no-op without one)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(tokens_per_rank_per_step: List[int] | int, world_size: int,
                           ms_per_step_max: float) -> float:
    """Aggregate prompt tokens per second of the job: all ranks' tokens over the slowest rank's time."""
    if isinstance(tokens_per_rank_per_step, int):
        total = tokens_per_rank_per_step * world_size
    else:
        total = sum(tokens_per_rank_per_step)
    return total / (ms_per_step_max * 1e-3)
