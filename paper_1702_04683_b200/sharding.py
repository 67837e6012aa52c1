"""Host-side plan for a parameter server sharded over several GPUs (one process per GPU).

Eq. 3-5 treat every parameter on its own, so the server state (Theta, history heads, ring)
can be cut into contiguous parameter ranges, one per rank.  Every update's index list is
ascending, hence the part of an update that belongs to a rank is ONE contiguous slice of its
(index, value) arrays: routing an update is a pair of binary searches per rank, and the exchange
is a variable-size all-to-all.  Received slices land in the owner's own memory before any kernel
reads them; arrival order and pull timestamps are global metadata every rank knows.

This module only cuts and routes; the arithmetic stays in the library (``adacomp_apply`` on each
owner, with indices made local to its range: ``ShardedServer``).  It works with any
``torch.distributed`` backend that has point-to-point send / recv (``nccl`` on GPUs, ``gloo`` on CPU
for tests).  No kernel is ever handed another GPU's memory.
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


def as_index64(idx: torch.Tensor) -> torch.Tensor:
    """Indices as non-negative int64: int32 tensors hold uint32 bit patterns (what adacomp_select emits)."""
    if idx.dtype == torch.int32:
        return idx.to(torch.int64) & 0xFFFFFFFF
    return idx.to(torch.int64)


def slice_points(idx_sorted: torch.Tensor, ranges: Sequence[Tuple[int, int]]) -> List[int]:
    """Positions that cut one update's ascending index list into the ranks' slices (len = world + 1).
    ``idx_sorted``: int64, or int32 holding uint32 bit patterns."""
    wide = as_index64(idx_sorted)
    bounds = torch.tensor([r[0] for r in ranges] + [ranges[-1][1]], dtype=torch.int64, device=wide.device)
    return torch.searchsorted(wide, bounds).tolist()


def exchange_updates(idx: torch.Tensor, val: torch.Tensor, ranges: Sequence[Tuple[int, int]], group=None):
    """Every rank calls this with its local workers' updates, ``idx`` [W_local, K] (ascending rows;
    int64, or int32 holding uint32 bit patterns: the type travels as it is) and ``val`` [W_local, K].
    Returns, for this rank's parameter range, the slices of ALL ranks' updates: a list over source
    ranks of (idx_local [n], val [n], counts [W_src]) where idx_local is relative to this rank's
    ``lo`` and counts[w] is the slice length of source worker w.
    """
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    lo_me = ranges[rank][0]
    W = idx.shape[0]
    cuts = [slice_points(idx[w], ranges) for w in range(W)]
    # what I send to each destination: per-worker counts, then the concatenated slices
    # (the counts travel from the tensors' device: NCCL moves device memory only)
    send_counts = [torch.tensor([cuts[w][d + 1] - cuts[w][d] for w in range(W)], dtype=torch.int64, device=idx.device)
                   for d in range(world)]
    recv_counts = [torch.empty(W, dtype=torch.int64, device=idx.device) for _ in range(world)]   # same worker count on every rank
    reqs = []
    for d in range(world):
        if d == rank:
            recv_counts[d].copy_(send_counts[d])
        else:
            reqs.append(dist.isend(send_counts[d], d, group=group))
            reqs.append(dist.irecv(recv_counts[d], d, group=group))
    for r in reqs:
        r.wait()
    recv_counts = [c.cpu() for c in recv_counts]
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
    return [((as_index64(i) - lo_me).to(idx.dtype), v, c) for i, v, c in out]


class ShardedServer:
    """One rank's share of Algorithm 2's server when the parameters are cut over several GPUs.

    Rank r owns parameters [lo_r, hi_r) (``parameter_ranges``) with everything Eq. 3-5 need for them:
    its slice of Theta, their history, a timestamp that ticks once per update like everybody else's.
    ``step`` takes the updates of the workers THIS rank hosts, routes every update's slices to their
    owners (``exchange_updates``: point-to-point over the process group, received into the owner's own
    memory), and applies what arrived for this rank's range in the global arrival order with
    ``adacomp_apply`` (indices relative to ``lo``).  Since Eq. 3-5 treat every parameter on its own,
    the shards together hold exactly what one server over all parameters would hold.

    ``applier`` is the local server: by default a ``binding.Server`` over ``theta_shard`` (CUDA); any
    object with the same ``apply`` / ``timestamp`` serves (the CPU test passes the oracle).
    """

    def __init__(self, theta_shard: torch.Tensor, n_params_total: int, workers_per_rank: int, history_pairs: int,
                 max_window_updates: int, group=None, applier=None):
        self.group = group
        self.world, self.rank = dist.get_world_size(group), dist.get_rank(group)
        self.ranges = parameter_ranges(n_params_total, self.world)
        self.lo, self.hi = self.ranges[self.rank]
        if theta_shard.numel() != self.hi - self.lo:
            raise ValueError("theta_shard must hold this rank's parameter range")
        self.workers_per_rank = int(workers_per_rank)
        if applier is None:
            from . import binding                     # the CUDA library; fails loudly if it is not built
            applier = binding.Server(theta_shard, history_pairs, max_window_updates)
        self.applier = applier

    @property
    def timestamp(self) -> int:
        return self.applier.timestamp

    def step(self, idx: torch.Tensor, val: torch.Tensor, order, pull_ts, lr: float, want_sigma: bool = False):
        """``idx`` / ``val`` [workers_per_rank, K]: the updates of this rank's workers (global worker id =
        rank * workers_per_rank + row).  ``order[b]`` = global id of the worker whose update arrives b-th,
        ``pull_ts[b]`` its pull timestamp: the same arrays on every rank.  Returns None, or with
        ``want_sigma`` (sigma, begin, count): the staleness counts of this rank's slices, slice of global
        worker w at sigma[begin[w] : begin[w] + count[w]]."""
        if idx.shape[0] != self.workers_per_rank:
            raise ValueError("one row per hosted worker")
        got = exchange_updates(idx, val, self.ranges, self.group)
        flat_idx = torch.cat([g[0] for g in got]) if got else idx.new_empty(0)
        flat_val = torch.cat([g[1] for g in got]) if got else val.new_empty(0)
        counts = torch.cat([g[2] for g in got]).to(torch.int64)            # by global worker id: source rank, then row
        begin = torch.cumsum(counts, 0) - counts
        order = np.asarray(order, dtype=np.int64)
        b_np, c_np = begin.numpy().astype(np.uint64), counts.numpy().astype(np.uint32)
        sigma = torch.empty_like(flat_idx, dtype=torch.int32) if want_sigma else None
        if flat_idx.dtype != torch.int32:
            flat_idx = flat_idx.to(torch.int32)       # local indices fit: a shard holds fewer than 2^31 parameters
        self.applier.apply(flat_idx, flat_val, b_np[order], c_np[order], np.asarray(pull_ts, dtype=np.uint64), lr,
                           sigma_out=sigma)
        return (sigma, b_np, c_np) if want_sigma else None
