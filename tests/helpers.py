"""Shared test plumbing: run a workload through the CPU oracle and through the CUDA library."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_1702_04683_b200 import workloads as wlmod


def oracle_keep_counts(sizes, keep):
    return [oracle.keep_count(n, keep[0], keep[1]) for n in sizes]


def u32(t: torch.Tensor) -> np.ndarray:
    """int32 tensor (bit pattern of uint32) -> numpy uint32."""
    return t.detach().cpu().numpy().view(np.uint32)


def bits(a) -> np.ndarray:
    if isinstance(a, torch.Tensor):
        a = a.detach().cpu().numpy()
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def oracle_select_round(wl, grads_host: np.ndarray, ks, full_sort=False):
    """[W, P] host gradients -> (idx [W, K] uint32, val [W, K] float32) from the oracle."""
    W = grads_host.shape[0]
    K = int(sum(ks))
    idx = np.empty((W, K), dtype=np.uint32)
    val = np.empty((W, K), dtype=np.float32)
    for w in range(W):
        idx[w], val[w] = oracle.select_layers(grads_host[w], wl.offsets, wl.tensor_sizes, ks, full_sort=full_sort)
    return idx, val


def oracle_pipeline(wl, keep, device_for_inputs="cpu", literal=False):
    """Whole path on the CPU: per round select every worker's gradient, then apply the pushes in
    arrival order.  Returns dict(idx=[rounds][W,K], val=..., sigma=[rounds][W,K] (worker order),
    theta=final)."""
    ks = oracle_keep_counts(wl.tensor_sizes, keep)
    K = int(sum(ks))
    theta0 = wlmod.initial_parameters(wl, device_for_inputs).cpu().numpy()
    srv = oracle.Server(theta0, literal=literal)
    out = {"idx": [], "val": [], "sigma": [], "ks": ks}
    for r, rd in enumerate(wlmod.arrival_schedule(wl)):
        g = wlmod.round_gradients(wl, r, device_for_inputs).cpu().numpy()
        idx, val = oracle_select_round(wl, g, ks)
        sigma = np.empty((wl.n_workers, K), dtype=np.uint32)
        for b, w in enumerate(rd.order.tolist()):
            sigma[w] = srv.apply(idx[w], val[w], int(rd.pull_ts[b]), wl.lr)
        out["idx"].append(idx)
        out["val"].append(val)
        out["sigma"].append(sigma)
    out["theta"] = srv.theta()
    out["timestamp"] = srv.timestamp
    return out


def gpu_pipeline(wl, keep, mode=0, history_rounds=2):
    """Whole path through the C ABI on cuda:0, same inputs (generated on the GPU)."""
    from paper_1702_04683_b200 import binding
    dev = torch.device("cuda", 0)
    segs = binding.make_segments(wl.tensor_sizes, keep)
    sel = binding.Selector(segs, wl.n_workers, dev)
    K = sel.pairs_per_worker
    theta = wlmod.initial_parameters(wl, dev)
    srv = binding.Server(theta, history_pairs=max(1, history_rounds * wl.n_workers * K),
                         max_window_updates=max(2 * wl.n_workers, 8))
    srv.set_mode(mode)
    srv.set_validation(True)
    out = {"idx": [], "val": [], "sigma": []}
    for r, rd in enumerate(wlmod.arrival_schedule(wl)):
        g = wlmod.round_gradients(wl, r, dev)
        idx, val = sel.select(g)
        sigma = torch.empty_like(idx)
        begin = rd.order.astype(np.uint64) * np.uint64(K)
        count = np.full(wl.n_workers, K, dtype=np.uint32)
        srv.apply(idx.view(-1), val.view(-1), begin, count, rd.pull_ts, wl.lr, sigma_out=sigma.view(-1))
        out["idx"].append(u32(idx))
        out["val"].append(val.cpu().numpy())
        out["sigma"].append(u32(sigma))
    assert sel.last_error()[0] == 0
    assert srv.last_error() == 0
    out["theta"] = theta.cpu().numpy()
    out["timestamp"] = srv.timestamp
    return out


def gpu_inputs_to_host(wl, rnd):
    """Gradients generated on the GPU, copied to the host so both sides see the same bits."""
    return wlmod.round_gradients(wl, rnd, torch.device("cuda", 0))


def assert_same_pipeline(a, b):
    assert a["timestamp"] == b["timestamp"]
    for r in range(len(a["idx"])):
        assert np.array_equal(a["idx"][r], b["idx"][r]), f"round {r}: indices differ"
        assert np.array_equal(bits(a["val"][r]), bits(b["val"][r])), f"round {r}: values differ"
        assert np.array_equal(a["sigma"][r], b["sigma"][r]), f"round {r}: staleness differs"
    assert np.array_equal(bits(a["theta"]), bits(b["theta"])), "parameters differ"
