"""How the path spreads over several GPUs: every (batch, head) unit is independent in all
stages, so ranks take disjoint sets of units and no data-path collective is needed.  The
only communication is the max-over-ranks of the measured time (and a barrier)."""
from __future__ import annotations

import os


def env_rank_world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def unit_partition(n_units: int, rank: int, world: int) -> range:
    """Contiguous, disjoint, covering split of n_units (batch, head) units over `world` ranks;
    the first n_units % world ranks take one unit more."""
    if world <= 0 or not (0 <= rank < world):
        raise ValueError("bad rank/world")
    base, extra = divmod(n_units, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def rank_seed(seed: int, rank: int) -> int:
    """Weak scaling: every rank runs the whole workload on its own seeded draw."""
    return seed + 7919 * rank


def max_over_ranks(value: float, backend_device=None) -> float:
    """Max of a scalar over all ranks (no-op without an initialised process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=backend_device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, backend_device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=backend_device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
