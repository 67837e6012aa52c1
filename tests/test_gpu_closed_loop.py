"""The workers' loop of Algorithm 1 closed over the server (pull, compute, select, push, pull again)
on emulated schedules with heterogeneous speeds and crashes: the CUDA path against the oracle, once
update by update with real pulls, once in batches of many updates per call."""
import numpy as np
import pytest
import torch

import oracle
from paper_1702_04683_b200 import workloads as wlmod

from helpers import bits, oracle_keep_counts, u32

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda", 0)


@pytest.fixture(scope="module")
def binding():
    from paper_1702_04683_b200 import binding as b
    return b


def schedule_case(kind):
    if kind == "heterogeneous":
        return wlmod.closed_loop_schedule(20, 360, seed=8, class_fractions=(0.3, 0.4, 0.3), class_rates=(100, 10, 1))
    return wlmod.closed_loop_schedule(24, 360, seed=9, crash_probability=0.03)


@pytest.mark.parametrize("kind", ["heterogeneous", "crashes"])
@pytest.mark.parametrize("batch", [1, 32])
def test_closed_loop_matches_the_oracle(binding, kind, batch):
    cl = schedule_case(kind)
    N = cl.worker.size
    wl = wlmod.workload(0).scaled(64, n_workers=int(cl.klass.size))       # 51 166 parameters, 4 tensors
    keep = (1, 100)
    ks = oracle_keep_counts(wl.tensor_sizes, keep)
    K = int(sum(ks))
    lag = np.arange(N) - cl.pull_ts.astype(np.int64)
    assert lag.max() >= 60                                               # slow or unlucky workers push very stale updates
    sel = binding.Selector(binding.make_segments(wl.tensor_sizes, keep), batch, DEV)
    theta = wlmod.initial_parameters(wl, DEV)
    ref = oracle.Server(theta.cpu().numpy())
    srv = binding.Server(theta, history_pairs=(int(lag.max()) + batch + 2) * K, max_window_updates=int(lag.max()) + batch + 2)
    srv.set_validation(True)
    pulled = {}                                                           # what each worker holds: the timestamp of its pull
    count_per_worker = {}
    for u0 in range(0, N, batch):
        us = list(range(u0, min(u0 + batch, N)))
        rows = []
        for u in us:                                                      # a worker's successive updates come from fresh gradients
            w = int(cl.worker[u])
            rows.append(wlmod.worker_gradient(wl, count_per_worker.get(w, 0), w, DEV))
            count_per_worker[w] = count_per_worker.get(w, 0) + 1
        grads = torch.stack(rows)
        idx, val = sel.select(grads)
        sigma = torch.empty_like(idx)
        if batch == 1:                                                    # the worker pushes with the timestamp it really pulled
            w = int(cl.worker[u0])
            j = pulled.get(w, 0)
            assert j == int(cl.pull_ts[u0])
            srv.apply(idx.view(-1), val.view(-1), [0], [K], [j], wl.lr, sigma_out=sigma.view(-1))
            pulled[w] = srv.pull()                                        # Pull follows Push
            assert pulled[w] == u0 + 1
        else:
            n = len(us)
            srv.apply(idx.view(-1), val.view(-1), np.arange(n, dtype=np.uint64) * np.uint64(K), np.full(n, K, np.uint32),
                      cl.pull_ts[u0:u0 + n], wl.lr, sigma_out=sigma.view(-1))
        g_host = grads.cpu().numpy()
        for b, u in enumerate(us):
            oi, ov = oracle.select_layers(g_host[b], wl.offsets, wl.tensor_sizes, ks)
            assert np.array_equal(u32(idx[b]), oi) and np.array_equal(bits(val[b]), bits(ov)), f"update {u}"
            want = ref.apply(oi, ov, int(cl.pull_ts[u]), wl.lr)
            assert np.array_equal(u32(sigma[b]), want), f"update {u}: staleness differs"
    assert sel.last_error()[0] == 0 and srv.last_error() == 0
    assert srv.timestamp == ref.timestamp == N
    assert np.array_equal(bits(theta), bits(ref.theta()))
    if kind == "crashes":
        assert (cl.crashed_after >= 0).sum() >= 3
