"""Host-side helpers for running the path on several GPUs.

Every quantity of the path is per (layer, head): contexts (layers) or heads are dealt out to the
ranks and no collective runs inside the path.  The only cross-rank traffic is bookkeeping: a
barrier around a timed region and the maximum of the per-rank times.  These helpers hold that
bookkeeping so that it can be exercised on CPU ranks (gloo) as well as on GPUs (nccl).
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def partition(n_items: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous [start, end) share of n_items for `rank`: sizes differ by at most one and the
    first n_items % world ranks hold the larger shares."""
    if world < 1 or not (0 <= rank < world) or n_items < 0:
        raise ValueError("bad partition arguments")
    base, extra = divmod(n_items, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def assign_layers(n_layers: int, world: int) -> List[List[int]]:
    """Layer ids per rank (each layer is one context; contexts never talk to each other)."""
    return [list(range(*partition(n_layers, world, r))) for r in range(world)]


def max_over_ranks(values: Sequence[float], device: torch.device | str = "cpu") -> List[float]:
    """Element-wise maximum over all ranks of a short list of floats (e.g. elapsed times)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_throughput(units_per_rank: float, seconds_per_rank: float,
                         device: torch.device | str = "cpu") -> Tuple[float, float]:
    """Whole-job throughput: the units all ranks processed divided by the slowest rank's time.
    Returns (throughput, slowest_seconds)."""
    world = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
    t = torch.tensor([units_per_rank], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    slowest = max_over_ranks([seconds_per_rank], device)[0]
    return t.item() / slowest, slowest
