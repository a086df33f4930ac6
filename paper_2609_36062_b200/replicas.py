"""Multi-GPU layout of the prefill: independent replicas, no collective on the data path.

(batch, head) pairs share nothing but integer geometry, so N ranks run N independent copies of the
workload (or disjoint slices of its heads).  The only communication is bookkeeping for the benchmark:
a barrier around the timed region and a MAX-reduction of the per-rank times.  These helpers hold that
bookkeeping so that it can be exercised on CPU with the gloo backend.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def head_slice(total_heads: int, rank: int, world: int) -> range:
    """Contiguous, balanced slice of batch*heads units owned by `rank` (units are independent problems)."""
    base, extra = divmod(total_heads, world)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def max_over_ranks(values, device="cpu") -> list[float]:
    """Element-wise maximum over all ranks of a short list of floats (identity without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_throughput(units_per_rank: float, seconds_this_rank: float, device="cpu") -> float:
    """Whole-job throughput: units processed by all ranks divided by the slowest rank's time."""
    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    slowest = max_over_ranks([seconds_this_rank], device)[0]
    return world * units_per_rank / slowest
