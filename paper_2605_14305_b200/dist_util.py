"""Host-side helpers for running the verification step on several GPUs of one node.

Speculative windows are independent (the only cross-row dependency, the first rejection,
lives inside one window), so the path shards by windows with no data-path collective:
every rank verifies its own windows on its own GPU ("replicas").  What the ranks share is
bookkeeping only: distinct random streams, a barrier around timed regions and the maximum
of the per-rank device times.
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist

_GOLDEN = 0x9E3779B97F4A7C15


def rank_seed(seed: int, rank: int) -> int:
    """A 64-bit seed per rank: distinct ranks get distinct Philox keys for the same base seed."""
    return (int(seed) + _GOLDEN * int(rank)) & 0xFFFFFFFFFFFFFFFF


def shard_windows(total_windows: int, rank: int, world: int) -> Tuple[int, int]:
    """(first window, number of windows) of this rank when ``total_windows`` are split as evenly
    as possible (the first ``total % world`` ranks get one more)."""
    if world < 1 or not (0 <= rank < world) or total_windows < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(total_windows, world)
    count = base + (1 if rank < extra else 0)
    first = rank * base + min(rank, extra)
    return first, count


def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    vals = [float(v) for v in values]
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return vals
    t = torch.tensor(vals, dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def aggregate_rate(units_per_rank_per_step: int, steps: int, elapsed_ms_max: float, world: int) -> float:
    """Whole-job units per second: every rank processed ``units_per_rank_per_step * steps`` units
    in at most ``elapsed_ms_max`` milliseconds."""
    return units_per_rank_per_step * world * steps / (elapsed_ms_max * 1e-3)
