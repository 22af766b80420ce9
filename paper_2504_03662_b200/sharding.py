"""Running one batch of search instances on several GPUs.

Instances are independent, so the batch is cut into contiguous slices of about
equal work (sum of layers), each rank searches its slice with the single-GPU
path, and the small results (optimal cost, plan, memory, status per instance)
are gathered on every rank.  Nothing is exchanged while the tables are built.
The gather runs over torch.distributed (NCCL on GPUs, gloo in CPU tests).
"""
from __future__ import annotations

from typing import Callable, Dict, List, Tuple

import numpy as np
import torch
import torch.distributed as dist

from .inputs import Workload


def partition(L: np.ndarray, world: int) -> List[Tuple[int, int]]:
    """Contiguous [start, end) per rank with the sum of layers as even as a prefix cut allows.

    Every instance belongs to exactly one slice; slices may be empty when world > B.
    """
    L = np.asarray(L, np.int64).clip(min=0)
    B = len(L)
    csum = np.concatenate([[0], np.cumsum(L)])
    total = int(csum[-1])
    cuts = [0]
    for r in range(1, world):
        target = total * r / world
        k = int(np.searchsorted(csum, target, side="left"))
        # the boundary nearest to the target, never before the previous cut
        if k > 0 and abs(csum[k - 1] - target) <= abs(csum[min(k, B)] - target):
            k -= 1
        cuts.append(min(max(k, cuts[-1]), B))
    cuts.append(B)
    return [(cuts[r], cuts[r + 1]) for r in range(world)]


def gather_results(local: Dict[str, np.ndarray], bounds: List[Tuple[int, int]], Lmax: int,
                   device: torch.device, group=None) -> Dict[str, np.ndarray]:
    """All-gather per-instance results so that every rank holds the whole batch, in instance order."""
    world = len(bounds)
    width = max(e - s for s, e in bounds)
    n = local["opt_cost"].shape[0]
    # one int32 row per instance: opt_cost, mem_used, status, plan[Lmax]; padded to the widest slice
    buf = torch.full((max(width, 1), 3 + Lmax), -1, dtype=torch.int32)
    if n:
        buf[:n, 0] = torch.from_numpy(np.ascontiguousarray(local["opt_cost"], np.int32))
        buf[:n, 1] = torch.from_numpy(np.ascontiguousarray(local["mem_used"], np.int32))
        buf[:n, 2] = torch.from_numpy(np.ascontiguousarray(local["status"], np.int32))
        buf[:n, 3:] = torch.from_numpy(np.ascontiguousarray(local["plan"], np.int32))
    buf = buf.to(device)
    parts = [torch.empty_like(buf) for _ in range(world)]
    dist.all_gather(parts, buf, group=group)
    rows = np.concatenate([p.cpu().numpy()[: e - s] for p, (s, e) in zip(parts, bounds)], axis=0)
    return dict(opt_cost=rows[:, 0].copy(), mem_used=rows[:, 1].copy(), status=rows[:, 2].copy(), plan=rows[:, 3:].copy())


def search_sharded(w: Workload, local_search: Callable[[Workload], Dict[str, np.ndarray]],
                   device: torch.device, group=None) -> Dict[str, np.ndarray]:
    """Search the batch across the ranks of `group`.

    local_search runs the single-GPU path on a sub-batch and returns opt_cost, plan, mem_used and
    status arrays (on a GPU rank: SearchBuffers(...).step() followed by .results()).
    """
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    bounds = partition(w.L, world)
    s, e = bounds[rank]
    if e > s:
        local = local_search(w.take(slice(s, e)))
    else:
        local = dict(opt_cost=np.zeros(0, np.int32), mem_used=np.zeros(0, np.int32), status=np.zeros(0, np.int32),
                     plan=np.zeros((0, w.Lmax), np.int32))
    return gather_results(local, bounds, w.Lmax, device, group)
