"""The synthetic input generators: shapes, determinism, schedule structure."""
import numpy as np
import pytest
import torch

from paper_1702_04683_b200 import workloads as wlmod


def test_tensor_tables():
    cnn = wlmod.workload(0)
    assert cnn.tensor_sizes == (832, 51_264, 3_212_288, 10_250) and cnn.n_params == 3_274_634
    rn = wlmod.workload(3)
    assert len(rn.tensor_sizes) == 161 and rn.n_params == 25_557_032
    assert min(rn.tensor_sizes) == 64 and max(rn.tensor_sizes) == 2_359_296
    assert sum(1 for n in rn.tensor_sizes if n <= 2048) == 107
    assert all(1e-5 <= b <= 1e-2 for b in rn.scales)
    big = wlmod.workload(4)
    assert big.n_params == 100_000_000 and len(big.keep_fractions) == 6
    assert [w.n_workers for w in map(wlmod.workload, range(5))] == [8, 200, 64, 32, 16]


def test_gradients_are_reproducible_and_distinct():
    wl = wlmod.workload(0).scaled(64)
    a = wlmod.round_gradients(wl, 0)
    b = wlmod.round_gradients(wl, 0)
    assert a.shape == (8, wl.n_params) and a.dtype == torch.float32
    assert torch.equal(a, b)
    assert torch.equal(a[3], wlmod.worker_gradient(wl, 0, 3))
    assert not torch.equal(a[0], a[1])
    assert not torch.equal(a, wlmod.round_gradients(wl, 1))
    # per-tensor standard deviations follow the table
    off = wl.offsets
    sd = a[:, off[2]:off[2] + wl.tensor_sizes[2]].std().item()
    assert 0.9e-4 < sd < 1.1e-4


def test_tie_stress_values_sit_on_the_fp16_grid():
    wl = wlmod.workload(2).scaled(64, n_workers=2)
    g = wlmod.round_gradients(wl, 0)
    assert torch.equal(g, g.half().float())
    big = g[:, wl.offsets[2]:]
    assert big.abs().unique().numel() < big.numel() // 2       # many exact ties
    assert not torch.isnan(g).any()


def test_laplace_scales():
    wl = wlmod.workload(3).scaled(16, n_workers=1)
    g = wlmod.round_gradients(wl, 0)[0]
    n, b = wl.tensor_sizes[-2], wl.scales[-2]
    seg = g[wl.offsets[-2]:wl.offsets[-2] + n]
    assert abs(seg.abs().mean().item() / b - 1.0) < 0.05       # E|x| = b for Laplace(0, b)


def test_schedule_rounds_structure():
    wl = wlmod.workload(1)
    rounds = wlmod.arrival_schedule(wl)
    assert len(rounds) == 10
    last = {}
    ts = 0
    for r, rd in enumerate(rounds):
        assert sorted(rd.order.tolist()) == list(range(200))
        assert rd.first_ts == ts
        for b, w in enumerate(rd.order.tolist()):
            j = int(rd.pull_ts[b])
            assert j == (last[w] + 1 if w in last else 0)       # Pull follows the worker's own Push
            assert j <= ts + b and (ts + b) - j <= 2 * 200 - 1
            last[w] = ts + b
        ts += 200
    again = wlmod.arrival_schedule(wl)
    assert all(np.array_equal(a.order, b.order) for a, b in zip(rounds, again))


def test_schedule_uniform_staleness():
    wl = wlmod.small_cnn_uniform_staleness()
    (rd,) = wlmod.arrival_schedule(wl)
    b = np.arange(8)
    lag = b - rd.pull_ts.astype(np.int64)
    assert np.all(lag >= 0) and np.all(lag <= 7) and np.all(rd.pull_ts.astype(np.int64) >= 0)
    (rd0,) = wlmod.arrival_schedule(wlmod.workload(0))
    assert not rd0.pull_ts.any()


def test_closed_loop_heterogeneous_classes():
    """Three classes in proportions 30 / 40 / 30 % whose workers send updates in the ratio 100 : 10 : 1
    (the heterogeneity experiment); pulls follow the worker's own push."""
    n, N = 200, 60_000
    cl = wlmod.closed_loop_schedule(n, N, seed=3, class_fractions=(0.3, 0.4, 0.3), class_rates=(100, 10, 1))
    assert np.bincount(cl.klass).tolist() == [60, 80, 60]
    assert cl.worker.size == N and (cl.crashed_after == -1).all()
    per_worker = np.bincount(cl.worker, minlength=n).astype(np.float64)
    mean = [per_worker[cl.klass == c].mean() for c in range(3)]
    assert 8.5 < mean[0] / mean[1] < 11.5 and 7.0 < mean[1] / mean[2] < 14.0
    last = {}
    for u, (w, j) in enumerate(zip(cl.worker.tolist(), cl.pull_ts.tolist())):
        assert j == (last[w] + 1 if w in last else 0) and j <= u
        last[w] = u
    lag = np.arange(N) - cl.pull_ts.astype(np.int64)
    slow = np.isin(cl.worker, np.where(cl.klass == 2)[0])
    assert lag[slow].mean() > 20 * lag[~slow].mean()            # slow workers' updates are far staler
    again = wlmod.closed_loop_schedule(n, N, seed=3, class_fractions=(0.3, 0.4, 0.3), class_rates=(100, 10, 1))
    assert np.array_equal(cl.worker, again.worker) and np.array_equal(cl.pull_ts, again.pull_ts)
    other = wlmod.closed_loop_schedule(n, N, seed=4, class_fractions=(0.3, 0.4, 0.3), class_rates=(100, 10, 1))
    assert not np.array_equal(cl.worker, other.worker)


def test_closed_loop_fail_stop_crashes():
    """After each push a worker stops for good with probability p: it never pushes again, and the number
    of pushes a worker manages is geometric with mean 1 / p."""
    n, p = 400, 0.02
    cl = wlmod.closed_loop_schedule(n, 10**6, seed=5, crash_probability=p)
    assert (cl.crashed_after >= 1).all() and cl.worker.size == int(cl.crashed_after.sum())   # everybody stops in the end
    per_worker = np.bincount(cl.worker, minlength=n)
    assert np.array_equal(per_worker, cl.crashed_after)
    assert abs(per_worker.mean() * p - 1.0) < 0.15                                          # mean of a geometric law
    assert abs((per_worker > 35).mean() - (1 - p) ** 35) < 0.08                             # its tail
    few = wlmod.closed_loop_schedule(200, 5000, seed=6, crash_probability=0.004)
    gone = few.crashed_after >= 0
    assert 5 <= gone.sum() <= 40                                                             # about 5000 * 0.004 = 20
    for w in np.where(gone)[0]:
        assert (few.worker == w).sum() == few.crashed_after[w]
    with pytest.raises(ValueError):
        wlmod.closed_loop_schedule(10, 10, class_fractions=(0.5, 0.4), class_rates=(1, 2))
