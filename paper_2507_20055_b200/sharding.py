"""Splitting a batch of input boxes over ranks (one process per GPU).

Boxes are bounded independently of one another (the analysis is tensorised
over the batch, Section 3.2), and the network's weights are small, so the
multi-GPU form of the path is: every rank holds all the weights, bounds a
contiguous slice of the boxes, and keeps (or gathers) its slice of the
output.  There is no exchange step inside the analysis itself.

Host logic only: no certifier arithmetic here.
"""
from __future__ import annotations

from typing import List, Tuple

import numpy as np


def box_shard(batch: int, rank: int, world: int) -> Tuple[int, int]:
    """[start, stop) of the boxes rank `rank` of `world` bounds: contiguous, in rank order,
    sizes differing by at most one, the first batch % world ranks taking the larger share."""
    if batch < 0 or world < 1 or not (0 <= rank < world):
        raise ValueError("box_shard: bad arguments")
    base, extra = divmod(batch, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def shard_sizes(batch: int, world: int) -> List[int]:
    return [box_shard(batch, r, world)[1] - box_shard(batch, r, world)[0] for r in range(world)]


def gather_bounds(lb_local, ub_local, batch: int, group=None):
    """All-gathers the ranks' slices of the bounds ([boxes of this rank][n_total] torch tensors on
    the process group's device) into the full [batch][n_total] pair on every rank.
    A rank whose slice is empty takes part with a zero-row tensor."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    sizes = shard_sizes(batch, world)
    n_total = lb_local.shape[1]
    widest = max(sizes) if sizes else 0
    out = []
    for local in (lb_local, ub_local):
        assert local.shape[0] == sizes[dist.get_rank(group)], "slice does not match box_shard"
        padded = torch.zeros((widest, n_total), dtype=local.dtype, device=local.device)
        padded[: local.shape[0]] = local
        parts = [torch.empty_like(padded) for _ in range(world)]
        dist.all_gather(parts, padded, group=group)
        out.append(torch.cat([p[:s] for p, s in zip(parts, sizes)], dim=0))
    return out[0], out[1]


def shard_centers(centers: np.ndarray, rank: int, world: int) -> np.ndarray:
    a, b = box_shard(centers.shape[0], rank, world)
    return np.ascontiguousarray(centers[a:b])
