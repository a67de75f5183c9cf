"""Host-side helpers for running on several GPUs of one node.

The attention path shards over (batch, head) with no exchange step: every (b,h)
is an independent problem with its own decay rate and state.  So multi-GPU means
one process per GPU working on its own slice (or its own replica of the workload)
and NO collective on the data path; torch.distributed is used only for the barrier
and for the max-over-ranks of the timings.
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def head_range(rank: int, world: int, n_bh: int) -> Tuple[int, int]:
    """Contiguous range [lo, hi) of flattened (b,h) indices owned by `rank`; sizes differ by at most one."""
    if not (0 <= rank < world) or n_bh < 0:
        raise ValueError("bad rank/world/count")
    base, extra = divmod(n_bh, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device=None) -> float:
    """MAX of a host scalar over all ranks (identity when not initialised)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier() -> None:
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
