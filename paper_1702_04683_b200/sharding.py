"""Host-side plan for a parameter server sharded over several GPUs (one process per GPU).

Eq. 3-5 treat every parameter on its own, so the server state (Theta, history heads, ring)
can be cut into contiguous parameter ranges, one per rank.  Every update's index list is
ascending, hence the part of an update that belongs to a rank is ONE contiguous slice of its
(index, value) arrays: routing an update is a pair of binary searches per rank, and the exchange
is a variable-size all-to-all.  Received slices land in the owner's own memory before any kernel
reads them; arrival order and pull timestamps are global metadata every rank knows.

This module only cuts and routes; the arithmetic stays in the library (``adacomp_apply`` on each
owner, with indices made local to its range).  It works with any ``torch.distributed`` backend
that has point-to-point send / recv (``nccl`` on GPUs, ``gloo`` on CPU for tests).
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np
import torch
import torch.distributed as dist

RANGE_ALIGN = 1024      # shard boundaries fall on the apply kernel's parameter ranges


def parameter_ranges(n_params: int, world: int) -> List[Tuple[int, int]]:
    """Contiguous [lo, hi) per rank, boundaries multiples of RANGE_ALIGN (the last one ends at n_params)."""
    blocks = (n_params + RANGE_ALIGN - 1) // RANGE_ALIGN
    cuts = [min(n_params, (blocks * r // world) * RANGE_ALIGN) for r in range(world)] + [n_params]
    return [(cuts[r], cuts[r + 1]) for r in range(world)]


def slice_points(idx_sorted: torch.Tensor, ranges: Sequence[Tuple[int, int]]) -> List[int]:
    """Positions that cut one update's ascending index list into the ranks' slices (len = world + 1).
    ``idx_sorted`` holds non-negative int64 indices."""
    bounds = torch.tensor([r[0] for r in ranges] + [ranges[-1][1]], dtype=idx_sorted.dtype, device=idx_sorted.device)
    return torch.searchsorted(idx_sorted, bounds).tolist()


def exchange_updates(idx: torch.Tensor, val: torch.Tensor, ranges: Sequence[Tuple[int, int]], group=None):
    """Every rank calls this with its local workers' updates, ``idx`` [W_local, K] (int64, ascending
    rows) and ``val`` [W_local, K].  Returns, for this rank's parameter range, the slices of ALL
    ranks' updates: a list over source ranks of (idx_local [n], val [n], counts [W_src]) where
    idx_local is relative to this rank's ``lo`` and counts[w] is the slice length of source worker w.
    """
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    lo_me = ranges[rank][0]
    W = idx.shape[0]
    cuts = [slice_points(idx[w], ranges) for w in range(W)]
    # what I send to each destination: per-worker counts, then the concatenated slices
    send_counts = [torch.tensor([cuts[w][d + 1] - cuts[w][d] for w in range(W)], dtype=torch.int64) for d in range(world)]
    recv_counts = [torch.empty(W, dtype=torch.int64) for _ in range(world)]       # same worker count on every rank
    reqs = []
    for d in range(world):
        if d == rank:
            recv_counts[d].copy_(send_counts[d])
        else:
            reqs.append(dist.isend(send_counts[d], d, group=group))
            reqs.append(dist.irecv(recv_counts[d], d, group=group))
    for r in reqs:
        r.wait()
    send_idx = [torch.cat([idx[w, cuts[w][d]:cuts[w][d + 1]] for w in range(W)]).contiguous() for d in range(world)]
    send_val = [torch.cat([val[w, cuts[w][d]:cuts[w][d + 1]] for w in range(W)]).contiguous() for d in range(world)]
    out = []
    reqs = []
    for s in range(world):
        n = int(recv_counts[s].sum())
        out.append((torch.empty(n, dtype=idx.dtype, device=idx.device), torch.empty(n, dtype=val.dtype, device=val.device),
                    recv_counts[s]))
    for peer in range(world):
        if peer == rank:
            out[peer][0].copy_(send_idx[peer])
            out[peer][1].copy_(send_val[peer])
            continue
        reqs.append(dist.isend(send_idx[peer], peer, group=group))
        reqs.append(dist.irecv(out[peer][0], peer, group=group))
    for r in reqs:
        r.wait()
    reqs = []
    for peer in range(world):
        if peer == rank:
            continue
        reqs.append(dist.isend(send_val[peer], peer, group=group))
        reqs.append(dist.irecv(out[peer][1], peer, group=group))
    for r in reqs:
        r.wait()
    return [(i - lo_me, v, c) for i, v, c in out]
