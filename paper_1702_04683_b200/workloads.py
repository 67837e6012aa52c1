"""Seeded synthetic inputs: gradient vectors, initial parameters, arrival schedules.

This module only *generates inputs*.  It holds none of the method's arithmetic
(no selection, no keep-count rule, no staleness, no update) so that the CUDA
library and the CPU oracle can both be fed from it without sharing any logic.

The five workloads stand in for the paper's MNIST-CNN gradients (section
"Experimental setup and competitors"), which need a dataset and a trained model:
same kind of object (one dense fp32 gradient vector per worker, cut into
per-tensor ranges), sizes from a few hundred to 10^8 entries, and value
distributions chosen to exercise selection (Gaussian, heavy-tailed with exact
ties, Laplace with per-tensor scales).  Arrival order inside a round is a seeded
random permutation, mirroring the random wait the paper's platform inserts
between computation and push ("Experimental platform").
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

Fraction = Tuple[int, int]


def resnet50_tensor_sizes() -> List[int]:
    """Parameter-tensor sizes of a ResNet-50: stem conv 7x7x3x64 + bn; stages of
    [3,4,6,3] bottleneck blocks (1x1, 3x3, 1x1 convs, each followed by bn weight and
    bias; a 1x1 downsample conv + bn in the first block of each stage), expansion 4;
    fc 2048x1000 + bias.  161 tensors, 25,557,032 entries."""
    sizes = [7 * 7 * 3 * 64, 64, 64]
    inplanes = 64
    for width, blocks in zip((64, 128, 256, 512), (3, 4, 6, 3)):
        for b in range(blocks):
            out = width * 4
            sizes += [inplanes * width, width, width]
            sizes += [3 * 3 * width * width, width, width]
            sizes += [width * out, out, out]
            if b == 0:
                sizes += [inplanes * out, out, out]
            inplanes = out
    sizes += [2048 * 1000, 1000]
    assert len(sizes) == 161 and sum(sizes) == 25_557_032
    return sizes


@dataclasses.dataclass(frozen=True)
class Workload:
    """One synthetic workload.  ``schedule``:
    ``pull0``      every worker pulled at timestamp 0 (single round);
    ``uniform``    push at arrival position b carries j = b - min(s_b, b), s_b ~ U{0..max_staleness};
    ``rounds``     round 0 pulls at 0, later a worker pulls right after its own previous push
                   (Algorithm 1: Pull follows Push), so j = (timestamp of that push) + 1.
    """
    name: str
    index: int
    tensor_sizes: Tuple[int, ...]
    n_workers: int
    n_rounds: int
    keep_fractions: Tuple[Fraction, ...]
    distribution: str                      # "normal" | "student_t2_fp16" | "laplace"
    scales: Tuple[float, ...]              # one per tensor
    schedule: str
    seed: int = 0
    lr: float = 0.01
    max_staleness: int = 7

    @property
    def n_params(self) -> int:
        return int(sum(self.tensor_sizes))

    @property
    def offsets(self) -> List[int]:
        out, acc = [], 0
        for n in self.tensor_sizes:
            out.append(acc)
            acc += n
        return out

    def scaled(self, divisor: int, n_workers: Optional[int] = None, n_rounds: Optional[int] = None) -> "Workload":
        """Same structure with every tensor ``divisor`` times smaller (at least 1 entry):
        a case the CPU oracle finishes in seconds."""
        sizes = tuple(max(1, n // divisor) for n in self.tensor_sizes)
        return dataclasses.replace(
            self, name=f"{self.name}/div{divisor}", tensor_sizes=sizes,
            n_workers=n_workers or self.n_workers, n_rounds=n_rounds or self.n_rounds)


_CNN = (832, 51_264, 3_212_288, 10_250)
_CNN_SIGMA = (1e-2, 1e-3, 1e-4, 1e-3)


def _resnet_scales(seed: int) -> Tuple[float, ...]:
    rng = np.random.default_rng(seed + 4)
    return tuple(float(10.0 ** u) for u in rng.uniform(-5.0, -2.0, size=161))


def workload(index: int, seed: int = 0) -> Workload:
    """The five workloads (index 0..4)."""
    if index == 0:
        return Workload("small_cnn", 0, _CNN, 8, 1, ((1, 100),), "normal", _CNN_SIGMA, "pull0", seed)
    if index == 1:
        return Workload("many_workers", 1, _CNN, 200, 10, ((1, 100),), "normal", _CNN_SIGMA, "rounds", seed)
    if index == 2:
        return Workload("tie_stress", 2, _CNN, 64, 1, ((1, 1000), (1, 100), (1, 10)),
                        "student_t2_fp16", _CNN_SIGMA, "pull0", seed)
    if index == 3:
        return Workload("resnet50_shaped", 3, tuple(resnet50_tensor_sizes()), 32, 5, ((5, 1000),),
                        "laplace", _resnet_scales(seed), "rounds", seed)
    if index == 4:
        return Workload("large_flat", 4, (4_000_000,) * 25, 16, 1,
                        ((1, 1000), (1, 400), (1, 160), (1, 64), (1, 25), (1, 10)),
                        "normal", (1e-3,) * 25, "pull0", seed)
    raise ValueError("workload index must be 0..4")


def small_cnn_uniform_staleness(seed: int = 0) -> Workload:
    """Workload 0 with staleness drawn uniformly in [0, 7] per push."""
    return dataclasses.replace(workload(0, seed), name="small_cnn_uniform", schedule="uniform")


# --------------------------------------------------------------------------- gradients

def _worker_generator(wl: Workload, rnd: int, worker: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(((wl.seed * 1_000_003 + wl.index) * 10_007 + rnd) * 100_003 + worker)
    return g


def _scale_inplace(row: torch.Tensor, wl: Workload) -> None:
    if len(set(wl.scales)) == 1:
        row.mul_(wl.scales[0])
        return
    off = 0
    for n, s in zip(wl.tensor_sizes, wl.scales):
        row[off:off + n].mul_(s)
        off += n


def worker_gradient(wl: Workload, rnd: int, worker: int, device="cpu", out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Dense fp32 gradient vector of one worker in one round ([P]).  The same
    (workload, round, worker, device type) always yields the same bits."""
    P = wl.n_params
    gen = _worker_generator(wl, rnd, worker, device)
    row = out if out is not None else torch.empty(P, dtype=torch.float32, device=device)
    if wl.distribution == "normal":
        row.normal_(0.0, 1.0, generator=gen)
        _scale_inplace(row, wl)
    elif wl.distribution == "laplace":
        row.uniform_(-0.5, 0.5, generator=gen)
        sign = torch.sign(row)
        row.abs_().mul_(-2.0).add_(1.0).clamp_(min=1e-30).log_().mul_(sign).neg_()
        _scale_inplace(row, wl)
    elif wl.distribution == "student_t2_fp16":
        # t with 2 degrees of freedom: Z0 / sqrt((Z1^2 + Z2^2) / 2), then onto the fp16 grid
        row.normal_(0.0, 1.0, generator=gen)
        z1 = torch.empty_like(row).normal_(0.0, 1.0, generator=gen)
        z2 = torch.empty_like(row).normal_(0.0, 1.0, generator=gen)
        z1.mul_(z1).addcmul_(z2, z2).mul_(0.5).sqrt_().clamp_(min=1e-30)
        row.div_(z1)
        _scale_inplace(row, wl)
        row.copy_(row.half().float())
    else:
        raise ValueError(wl.distribution)
    return row


def round_gradients(wl: Workload, rnd: int, device="cpu", workers: Optional[Sequence[int]] = None) -> torch.Tensor:
    """[W, P] fp32: the gradients of ``workers`` (default: all) in round ``rnd``."""
    workers = list(range(wl.n_workers)) if workers is None else list(workers)
    out = torch.empty((len(workers), wl.n_params), dtype=torch.float32, device=device)
    for r, w in enumerate(workers):
        worker_gradient(wl, rnd, w, device, out=out[r])
    return out


def initial_parameters(wl: Workload, device="cpu") -> torch.Tensor:
    """Theta(0): N(0, 0.05^2) (Algorithm 2 starts from random parameters)."""
    g = torch.Generator(device=device)
    g.manual_seed(wl.seed * 7919 + 17 + wl.index)
    return torch.empty(wl.n_params, dtype=torch.float32, device=device).normal_(0.0, 0.05, generator=g)


# --------------------------------------------------------------------------- schedules

@dataclasses.dataclass
class Round:
    order: np.ndarray      # order[b] = worker whose push arrives b-th in this round
    pull_ts: np.ndarray    # pull_ts[b] = timestamp j carried by that push (uint64)
    first_ts: int          # server timestamp before the first push of the round


def arrival_schedule(wl: Workload) -> List[Round]:
    """Arrival order and pull timestamps of every push, round by round."""
    rng = np.random.default_rng(wl.seed * 1009 + 31 * wl.index + 5)
    W = wl.n_workers
    rounds: List[Round] = []
    last_push_ts = np.full(W, -1, dtype=np.int64)
    ts = 0
    for r in range(wl.n_rounds):
        order = rng.permutation(W)
        if wl.schedule == "pull0":
            pull = np.zeros(W, dtype=np.int64) + (0 if r == 0 else ts)
        elif wl.schedule == "uniform":
            s = rng.integers(0, wl.max_staleness + 1, size=W)
            b = np.arange(W) + ts
            pull = b - np.minimum(s, b)
        elif wl.schedule == "rounds":
            pull = np.where(last_push_ts[order] < 0, 0, last_push_ts[order] + 1)
        else:
            raise ValueError(wl.schedule)
        rounds.append(Round(order=order.astype(np.int64), pull_ts=pull.astype(np.uint64), first_ts=ts))
        last_push_ts[order] = ts + np.arange(W)
        ts += W
    return rounds


@dataclasses.dataclass
class ClosedLoop:
    """A sequence of pushes as an emulated platform would produce it: ``worker[u]`` pushes update u
    (u = the server's timestamp when it is applied) computed from the parameters it pulled at
    ``pull_ts[u]``.  ``klass[w]`` is the speed class of worker w, ``crashed_after[w]`` the number of
    pushes after which worker w stopped for good (-1: still alive at the end)."""
    worker: np.ndarray
    pull_ts: np.ndarray
    klass: np.ndarray
    crashed_after: np.ndarray


def closed_loop_schedule(n_workers: int, n_updates: int, seed: int = 0,
                         class_fractions: Sequence[float] = (1.0,), class_rates: Sequence[float] = (1.0,),
                         crash_probability: float = 0.0) -> ClosedLoop:
    """Event-driven emulation of the workers' loop (Algorithm 1: pull, compute, push, pull again at
    once).  A worker of class c needs an exponentially distributed time with mean 1 / class_rates[c]
    per update, so classes send updates in the ratio of their rates; the first
    round(class_fractions[0] * n_workers) workers are in class 0, and so on (the heterogeneity
    experiment: fractions 0.3 / 0.4 / 0.3 with rates 100 : 10 : 1).  After each of its pushes a worker
    stops for good with probability ``crash_probability`` (the fail-stop experiment: 0.004).  The
    sequence ends after ``n_updates`` pushes, or earlier if every worker has stopped."""
    import heapq
    if len(class_fractions) != len(class_rates) or abs(sum(class_fractions) - 1.0) > 1e-9:
        raise ValueError("one rate per class, fractions summing to 1")
    rng = np.random.default_rng(seed * 7919 + 13)
    bounds = np.round(np.cumsum(class_fractions) * n_workers).astype(np.int64)
    klass = np.searchsorted(bounds, np.arange(n_workers), side="right").astype(np.int64)
    klass = np.minimum(klass, len(class_rates) - 1)
    rate = np.asarray(class_rates, dtype=np.float64)[klass]
    heap = [(float(rng.exponential(1.0 / rate[w])), w) for w in range(n_workers)]
    heapq.heapify(heap)
    pulled_at = np.zeros(n_workers, dtype=np.int64)
    pushes = np.zeros(n_workers, dtype=np.int64)
    crashed_after = np.full(n_workers, -1, dtype=np.int64)
    worker, pull_ts = [], []
    while heap and len(worker) < n_updates:
        t, w = heapq.heappop(heap)
        worker.append(w)
        pull_ts.append(pulled_at[w])
        pushes[w] += 1
        pulled_at[w] = len(worker)                        # pulls again right after its own push
        if crash_probability > 0.0 and rng.random() < crash_probability:
            crashed_after[w] = pushes[w]
        else:
            heapq.heappush(heap, (t + float(rng.exponential(1.0 / rate[w])), w))
    return ClosedLoop(worker=np.asarray(worker, dtype=np.int64), pull_ts=np.asarray(pull_ts, dtype=np.uint64),
                      klass=klass, crashed_after=crashed_after)


def describe(wl: Workload) -> dict:
    return {"workload": wl.name, "tensors": len(wl.tensor_sizes), "params": wl.n_params,
            "workers": wl.n_workers, "rounds": wl.n_rounds,
            "keep_fractions": [f"{a}/{b}" for a, b in wl.keep_fractions],
            "distribution": wl.distribution, "schedule": wl.schedule, "seed": wl.seed}


# --------------------------------------------------------------------------- ready-made updates

def synthetic_updates(wl: Workload, keep_counts: Sequence[int], rnd: int, device="cpu",
                      zero_fraction: float = 0.0) -> Tuple[torch.Tensor, torch.Tensor]:
    """Updates for exercising the server alone: for every worker and tensor, ``keep_counts[l]``
    distinct ascending indices (one drawn uniformly from each of k equal strata of the tensor)
    with N(0, scale_l) values.  Returns (idx [W, K] int32 holding uint32 bit patterns,
    val [W, K] fp32).  Two workers name the same parameter with probability about k/n, as
    independent uniform choices would."""
    W, K = wl.n_workers, int(sum(keep_counts))
    idx = torch.empty((W, K), dtype=torch.int64, device=device)
    val = torch.empty((W, K), dtype=torch.float32, device=device)
    gen = torch.Generator(device=device)
    gen.manual_seed(((wl.seed * 1_000_003 + wl.index) * 10_007 + rnd) * 100_003 + 77_777)
    at = 0
    for off, n, k, s in zip(wl.offsets, wl.tensor_sizes, keep_counts, wl.scales):
        if k == 0:
            continue
        t = torch.arange(k, dtype=torch.int64, device=device)
        lo = (t * n) // k
        width = ((t + 1) * n) // k - lo
        u = torch.rand((W, k), dtype=torch.float64, device=device, generator=gen)
        pick = torch.minimum((u * width).to(torch.int64), width - 1)
        idx[:, at:at + k] = off + lo + pick
        val[:, at:at + k].normal_(0.0, 1.0, generator=gen).mul_(s)
        at += k
    if zero_fraction > 0:
        mask = torch.rand((W, K), device=device, generator=gen) < zero_fraction
        val[mask] = 0.0
    idx32 = (idx & 0xFFFFFFFF).to(torch.int64)
    idx32 = torch.where(idx32 >= 2**31, idx32 - 2**32, idx32).to(torch.int32)
    return idx32, val
