"""Parity of adacomp_apply and of the whole select -> apply path (CUDA, through the C ABI)
with the CPU oracle: indices, values, staleness counters and parameters bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_1702_04683_b200 import workloads as wlmod

from helpers import assert_same_pipeline, bits, gpu_pipeline, oracle_keep_counts, oracle_pipeline, u32

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda", 0)
MODES = [0, 1, 2, 3, 4]


@pytest.fixture(scope="module")
def binding():
    from paper_1702_04683_b200 import binding as b
    return b


def i32(a):
    """uint32 numpy -> int32 torch tensor with the same bits, on the GPU."""
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint32).view(np.int32)).to(DEV)


# ----------------------------------------------------------------------------- whole path

@pytest.mark.parametrize("mode", MODES)
def test_small_cnn_full_size_pipeline(mode):
    wl = wlmod.workload(0)
    assert_same_pipeline(gpu_pipeline(wl, (1, 100), mode), oracle_pipeline(wl, (1, 100), DEV))


@pytest.mark.parametrize("mode", MODES)
def test_small_cnn_uniform_staleness_pipeline(mode):
    wl = wlmod.small_cnn_uniform_staleness()
    assert_same_pipeline(gpu_pipeline(wl, (1, 100), mode), oracle_pipeline(wl, (1, 100), DEV))


@pytest.mark.parametrize("mode", MODES)
def test_many_workers_scaled_pipeline(mode):
    wl = wlmod.workload(1).scaled(64)                  # 200 workers x 10 rounds, 51 k parameters
    got, want = gpu_pipeline(wl, (1, 100), mode), oracle_pipeline(wl, (1, 100), DEV)
    assert_same_pipeline(got, want)
    assert max(int(s.max()) for s in want["sigma"]) >= 3      # the interleaving does produce staleness


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("keep", [(1, 1000), (1, 10)])
def test_tie_stress_scaled_pipeline(mode, keep):
    wl = wlmod.workload(2).scaled(8, n_workers=16)
    assert_same_pipeline(gpu_pipeline(wl, keep, mode), oracle_pipeline(wl, keep, DEV))


@pytest.mark.parametrize("mode", MODES)
def test_resnet_scaled_pipeline(mode):
    wl = wlmod.workload(3).scaled(8, n_workers=8, n_rounds=3)
    assert_same_pipeline(gpu_pipeline(wl, (5, 1000), mode), oracle_pipeline(wl, (5, 1000), DEV))


@pytest.mark.parametrize("mode", MODES)
def test_literal_form_agrees_on_a_small_case(mode):
    wl = wlmod.workload(1).scaled(512, n_workers=12, n_rounds=4)
    assert_same_pipeline(gpu_pipeline(wl, (1, 20), mode), oracle_pipeline(wl, (1, 20), DEV, literal=True))


# ----------------------------------------------------------------------------- server alone, full sizes

def run_server_both(binding, wl, ks, mode, zero_fraction=0.0, rounds=None, sample_only=False):
    K = int(sum(ks))
    theta = wlmod.initial_parameters(wl, DEV)
    theta0 = theta.cpu().numpy()
    srv = binding.Server(theta, history_pairs=2 * wl.n_workers * K, max_window_updates=2 * wl.n_workers)
    srv.set_mode(mode)
    ref = None if sample_only else oracle.Server(theta0)
    sched = wlmod.arrival_schedule(wl)[:rounds]
    all_idx, all_val, all_sig, begins, pulls = [], [], [], [], []
    for r, rd in enumerate(sched):
        idx, val = wlmod.synthetic_updates(wl, ks, r, DEV, zero_fraction)
        sigma = torch.empty_like(idx)
        begin = rd.order.astype(np.uint64) * np.uint64(K)
        srv.apply(idx.view(-1), val.view(-1), begin, np.full(wl.n_workers, K, np.uint32), rd.pull_ts, wl.lr,
                  sigma_out=sigma.view(-1))
        h_idx, h_val, h_sig = u32(idx), val.cpu().numpy(), u32(sigma)
        if ref is not None:
            for b, w in enumerate(rd.order.tolist()):
                want = ref.apply(h_idx[w], h_val[w], int(rd.pull_ts[b]), wl.lr)
                assert np.array_equal(h_sig[w], want), f"round {r} update {b}: staleness differs"
        else:
            for b, w in enumerate(rd.order.tolist()):     # arrival order, for the per-parameter trace
                all_idx.append(h_idx[w]); all_val.append(h_val[w]); all_sig.append(h_sig[w])
                pulls.append(int(rd.pull_ts[b]))
    assert srv.last_error() == 0
    got = theta.cpu().numpy()
    if ref is not None:
        assert np.array_equal(bits(got), bits(ref.theta()))
        assert srv.timestamp == ref.timestamp
        return
    # sampled parameters, each traced through every update by searching its index list
    idx_cat, val_cat = np.concatenate(all_idx), np.concatenate(all_val)
    pair_begin = (np.arange(len(all_idx) + 1, dtype=np.uint64) * np.uint64(K))
    rng = np.random.default_rng(5)
    named = np.unique(np.concatenate([a[rng.integers(0, K, 40)] for a in all_idx]))
    picks = np.concatenate([named[:400], rng.integers(0, wl.n_params, 50).astype(np.uint32)])
    for k in picks:
        sig_k, theta_k = oracle.parameter_trace(int(k), float(theta0[k]), idx_cat, val_cat, pair_begin,
                                                np.array(pulls, np.uint64), wl.lr)
        seen = [int(s[np.searchsorted(a, k)]) for a, s in zip(all_idx, all_sig)
                if np.searchsorted(a, k) < K and a[np.searchsorted(a, k)] == k]
        assert list(sig_k) == seen
        assert np.float32(theta_k).view(np.uint32) == got[k].view(np.uint32)
    # parameters no update named are untouched
    touched = np.zeros(wl.n_params, dtype=bool)
    touched[idx_cat] = True
    assert np.array_equal(bits(got[~touched]), bits(theta0[~touched]))


@pytest.mark.parametrize("mode", MODES)
def test_many_workers_full_size_server(binding, mode):
    wl = wlmod.workload(1)                               # 200 workers x 10 rounds x 32 748 pairs
    ks = oracle_keep_counts(wl.tensor_sizes, (1, 100))
    run_server_both(binding, wl, ks, mode, zero_fraction=0.01)


@pytest.mark.parametrize("mode", MODES)
def test_resnet_full_size_server(binding, mode):
    wl = wlmod.workload(3)
    ks = oracle_keep_counts(wl.tensor_sizes, (5, 1000))
    run_server_both(binding, wl, ks, mode)


# every keep fraction the benchmark times in the automatic mode (each picks another kernel or
# range size); the two ends of the sweep also in every forced mode
_LARGE_FLAT_CASES = [(0, k) for k in wlmod.workload(4).keep_fractions] + \
                    [(m, k) for m in MODES[1:] for k in ((1, 1000), (1, 10))]


@pytest.mark.parametrize("mode,keep", _LARGE_FLAT_CASES)
def test_large_flat_full_size_server_sampled(binding, mode, keep):
    wl = wlmod.workload(4)
    ks = oracle_keep_counts(wl.tensor_sizes, keep)
    run_server_both(binding, wl, ks, mode, sample_only=True)


# ----------------------------------------------------------------------------- whole path, full sizes

@pytest.mark.parametrize("index,keep,rounds", [(1, (1, 100), 2), (2, (1, 100), 1), (2, (1, 10), 1), (3, (5, 1000), 2)])
def test_full_size_selector_output_meets_the_server(index, keep, rounds):
    """The 200-worker, the tie-stress and the ResNet-50-shaped workloads at full tensor sizes and
    full worker counts: what the selector emits is what the server applies, round after round,
    against the oracle's select -> apply (two rounds where the workload has more: the second one
    carries windows that reach back over the first)."""
    import dataclasses
    wl = dataclasses.replace(wlmod.workload(index), n_rounds=rounds)
    got = gpu_pipeline(wl, keep, mode=0)
    want = oracle_pipeline(wl, keep, DEV)
    assert_same_pipeline(got, want)
    if rounds > 1:
        assert max(int(s.max()) for s in want["sigma"]) >= 1


# ----------------------------------------------------------------------------- semantics and errors

@pytest.mark.parametrize("mode", MODES)
def test_zero_values_empty_updates_and_scattered_slices(binding, mode):
    theta = torch.tensor([-0.0, 1.0, 2.0, -0.0, 5.0, 6.0], device=DEV)
    srv = binding.Server(theta, history_pairs=64, max_window_updates=8)
    srv.set_mode(mode)
    ref = oracle.Server(theta.cpu().numpy())
    # three updates stored out of arrival order inside one buffer, one of them empty
    idx = i32([9, 9, 0, 1, 3, 1, 4, 5])
    val = torch.tensor([0, 0, 0.0, 1.0, -0.0, 0.5, 0.25, 0.0], device=DEV)
    sigma = torch.full((8,), -1, dtype=torch.int32, device=DEV)
    begin, count, pull = [5, 0, 2, 5], [3, 0, 3, 3], [0, 0, 0, 1]
    srv.apply(idx, val, begin, count, pull, 0.5, sigma_out=sigma)
    want = []
    for b, c, j in zip(begin, count, pull):
        want.append(ref.apply(u32(idx)[b:b + c], val.cpu().numpy()[b:b + c], j, 0.5))
    assert srv.last_error() == 0 and srv.timestamp == 4 == ref.timestamp
    assert np.array_equal(bits(theta), bits(ref.theta()))
    s = u32(sigma)
    assert list(s[5:8]) == list(want[3]) and list(s[2:5]) == list(want[2])
    assert list(want[3]) == [1, 0, 0]      # the last update overwrote the first one's sigma slots
    assert torch.signbit(theta[0]) and torch.signbit(theta[3])


@pytest.mark.parametrize("mode", MODES)
def test_clustered_and_uneven_updates(binding, mode):
    """Updates whose indices crowd into a few stretches of the parameter vector (far more pairs per
    stretch than any kernel stages at once), next to thin and empty ones, over three calls."""
    P = 300_000
    rng = np.random.default_rng(11)
    theta = torch.from_numpy(rng.standard_normal(P).astype(np.float32)).to(DEV)
    ref = oracle.Server(theta.cpu().numpy())
    srv = binding.Server(theta, history_pairs=1 << 20, max_window_updates=32)
    srv.set_mode(mode)
    def updates():
        out = [np.arange(50_000, 60_000), np.arange(0, P, 7), np.sort(rng.choice(P, 3000, replace=False)),
               np.arange(55_000, 75_000), np.array([], dtype=np.int64), np.arange(P - 700, P),
               np.sort(rng.choice(np.arange(100_000, 101_000), 900, replace=False)), np.arange(58_000, 58_100)]
        return [a.astype(np.uint32) for a in out]
    ts = 0
    for call in range(3):
        ups = updates()
        vals = [rng.standard_normal(a.size).astype(np.float32) for a in ups]
        vals[3][::5] = 0.0                                   # present, but not a change
        begin = np.concatenate([[0], np.cumsum([a.size for a in ups])[:-1]]).astype(np.uint64)
        count = np.array([a.size for a in ups], np.uint32)
        pull = np.array([max(0, ts + b - int(rng.integers(0, 6))) for b in range(len(ups))], np.uint64)
        idx, val = i32(np.concatenate(ups)), torch.from_numpy(np.concatenate(vals)).to(DEV)
        sigma = torch.full_like(idx, -1)
        order = rng.permutation(len(ups))                    # arrival order differs from memory order
        srv.apply(idx, val, begin[order], count[order], pull, 0.05, sigma_out=sigma)
        s = u32(sigma)
        for b, w in enumerate(order.tolist()):
            want = ref.apply(ups[w], vals[w], int(pull[b]), 0.05)
            lo = int(begin[w])
            assert np.array_equal(s[lo:lo + ups[w].size], want), f"call {call} update {b}"
        ts += len(ups)
    assert srv.last_error() == 0 and srv.timestamp == ts == ref.timestamp
    assert np.array_equal(bits(theta), bits(ref.theta()))


@pytest.mark.parametrize("mode", [0, 3])
@pytest.mark.parametrize("crowded", [12, 3, 0])
def test_thin_updates_that_crowd_into_a_small_stretch(binding, mode, crowded):
    """Updates thin by their pair counts (1 % of the parameters each) of which `crowded` draw their pairs from
    one twentieth of the parameter vector and the rest from all of it: all, a few and none of them crowded,
    which is what decides the kernel on the device."""
    P, n_up, per = 2_000_000, 12, 20_000
    rng = np.random.default_rng(400 + crowded)
    theta = torch.from_numpy(rng.standard_normal(P).astype(np.float32)).to(DEV)
    ref = oracle.Server(theta.cpu().numpy())
    srv = binding.Server(theta, history_pairs=4 * n_up * per, max_window_updates=3 * n_up)
    srv.set_mode(mode)
    ts = 0
    for call in range(3):
        lo = int(rng.integers(0, P - P // 20))
        ups = [np.sort(rng.choice(np.arange(lo, lo + P // 20) if b < crowded else P, per, replace=False)).astype(np.uint32)
               for b in range(n_up)]
        vals = [rng.standard_normal(per).astype(np.float32) for _ in ups]
        begin = (np.arange(n_up) * per).astype(np.uint64)
        count = np.full(n_up, per, np.uint32)
        pull = np.array([max(0, ts + b - int(rng.integers(0, 2 * n_up))) for b in range(n_up)], np.uint64)
        idx, val = i32(np.concatenate(ups)), torch.from_numpy(np.concatenate(vals)).to(DEV)
        sigma = torch.full_like(idx, -1)
        srv.apply(idx, val, begin, count, pull, 0.05, sigma_out=sigma)
        s = u32(sigma)
        for b in range(n_up):
            want = ref.apply(ups[b], vals[b], int(pull[b]), 0.05)
            assert np.array_equal(s[b * per:(b + 1) * per], want), f"call {call} update {b}"
        ts += n_up
    assert srv.last_error() == 0 and srv.timestamp == ts == ref.timestamp
    assert np.array_equal(bits(theta), bits(ref.theta()))


@pytest.mark.parametrize("mode", MODES)
def test_parameters_on_an_odd_address_and_odd_count(binding, mode):
    """Theta as a view that starts 4 bytes past a 16-byte boundary, with a parameter count that is
    no multiple of 4: vector accesses must not be assumed."""
    P = 70_001
    rng = np.random.default_rng(3)
    buf = torch.from_numpy(rng.standard_normal(P + 8).astype(np.float32)).to(DEV)
    theta = buf[1:P + 1]
    assert theta.data_ptr() % 16 == 4
    guard_lo, guard_hi = buf[0].item(), buf[P + 1:].clone()
    ref = oracle.Server(theta.cpu().numpy())
    srv = binding.Server(theta, history_pairs=1 << 18, max_window_updates=16)
    srv.set_mode(mode)
    ts = 0
    for call in range(2):
        ups = [np.sort(rng.choice(P, size, replace=False)).astype(np.uint32) for size in (30_000, 9_000, 50_000, 700, P)]
        vals = [rng.standard_normal(a.size).astype(np.float32) for a in ups]
        begin = np.concatenate([[0], np.cumsum([a.size for a in ups])[:-1]]).astype(np.uint64)
        count = np.array([a.size for a in ups], np.uint32)
        pull = np.array([max(0, ts + b - 2) for b in range(len(ups))], np.uint64)
        idx, val = i32(np.concatenate(ups)), torch.from_numpy(np.concatenate(vals)).to(DEV)
        sigma = torch.full_like(idx, -1)
        srv.apply(idx, val, begin, count, pull, 0.1, sigma_out=sigma)
        s = u32(sigma)
        for b in range(len(ups)):
            want = ref.apply(ups[b], vals[b], int(pull[b]), 0.1)
            assert np.array_equal(s[int(begin[b]):int(begin[b]) + ups[b].size], want), f"call {call} update {b}"
        ts += len(ups)
    assert srv.last_error() == 0
    assert np.array_equal(bits(theta), bits(ref.theta()))
    assert buf[0].item() == guard_lo and torch.equal(buf[P + 1:], guard_hi)      # nothing written outside Theta


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("density", [0.002, 0.012, 0.03, 0.12, 0.3])
def test_forty_updates_without_staleness_counts(binding, mode, density):
    """More updates per call than one launch takes (32), windows that reach back before the call,
    no staleness output asked for (the kernels' plain variants): parameters bit for bit."""
    P = 200_003
    rng = np.random.default_rng(int(density * 1000))
    theta = torch.from_numpy(rng.standard_normal(P).astype(np.float32)).to(DEV)
    ref = oracle.Server(theta.cpu().numpy())
    srv = binding.Server(theta, history_pairs=1 << 23, max_window_updates=128)
    srv.set_mode(mode)
    ts = 0
    for call in range(2):
        n_up = 40
        ups = [np.sort(rng.choice(P, int(P * density * rng.uniform(0.5, 1.0)), replace=False)).astype(np.uint32)
               for _ in range(n_up)]
        vals = [rng.standard_normal(a.size).astype(np.float32) for a in ups]
        vals[7][::3] = 0.0
        begin = np.concatenate([[0], np.cumsum([a.size for a in ups])[:-1]]).astype(np.uint64)
        count = np.array([a.size for a in ups], np.uint32)
        pull = np.array([max(0, ts + b - int(rng.integers(0, 50))) for b in range(n_up)], np.uint64)
        idx, val = i32(np.concatenate(ups)), torch.from_numpy(np.concatenate(vals)).to(DEV)
        srv.apply(idx, val, begin, count, pull, 0.05)
        for b in range(n_up):
            ref.apply(ups[b], vals[b], int(pull[b]), 0.05)
        ts += n_up
    assert srv.last_error() == 0 and srv.timestamp == ts == ref.timestamp
    assert np.array_equal(bits(theta), bits(ref.theta()))


@pytest.mark.parametrize("mode", [0, 3])
@pytest.mark.parametrize("n_up", [6, 12])
@pytest.mark.parametrize("with_sigma", [False, True])
def test_updates_of_six_percent_density(binding, mode, n_up, with_sigma):
    """Updates whose densest one names 5.1 % - 6.8 % of the parameters: the dense kernel then works on
    ranges of 384 parameters, with two buffers of Theta and heads for up to 8 updates per launch and
    one buffer beyond.  Second call: windows that reach back before the launch."""
    P = 300_011
    rng = np.random.default_rng(384 + n_up)
    theta = torch.from_numpy(rng.standard_normal(P).astype(np.float32)).to(DEV)
    ref = oracle.Server(theta.cpu().numpy())
    srv = binding.Server(theta, history_pairs=1 << 21, max_window_updates=64)
    srv.set_mode(mode)
    ts = 0
    for call in range(2):
        sizes = [int(P * d) for d in rng.uniform(0.052, 0.066, n_up)]
        sizes[0] = int(P * 0.066)
        ups = [np.sort(rng.choice(P, sz, replace=False)).astype(np.uint32) for sz in sizes]
        vals = [rng.standard_normal(a.size).astype(np.float32) for a in ups]
        vals[1][::4] = 0.0
        begin = np.concatenate([[0], np.cumsum([a.size for a in ups])[:-1]]).astype(np.uint64)
        count = np.array([a.size for a in ups], np.uint32)
        pull = np.array([max(0, ts + b - int(rng.integers(0, 2 * n_up))) for b in range(n_up)], np.uint64)
        idx, val = i32(np.concatenate(ups)), torch.from_numpy(np.concatenate(vals)).to(DEV)
        sigma = torch.full_like(idx, -1) if with_sigma else None
        srv.apply(idx, val, begin, count, pull, 0.05, sigma_out=sigma)
        for b in range(n_up):
            want = ref.apply(ups[b], vals[b], int(pull[b]), 0.05)
            if with_sigma:
                lo = int(begin[b])
                assert np.array_equal(u32(sigma)[lo:lo + ups[b].size], want), f"call {call} update {b}"
        ts += n_up
    assert srv.last_error() == 0 and srv.timestamp == ts == ref.timestamp
    assert np.array_equal(bits(theta), bits(ref.theta()))


@pytest.mark.parametrize("mode", MODES)
def test_tight_history_ring_in_one_call(binding, mode):
    """A ring sized with no slack, several updates in one call: an old window on the first update,
    later updates of the same call that name parameters with history and whose pairs would wrap
    onto ring slots the first update's window still reaches.  Launches must be cut so that no such
    slot is overwritten while it can still be walked: staleness and parameters against the oracle."""
    P = 4096
    rng = np.random.default_rng(64)
    theta = torch.from_numpy(rng.standard_normal(P).astype(np.float32)).to(DEV)
    ref = oracle.Server(theta.cpu().numpy())
    srv = binding.Server(theta, history_pairs=40, max_window_updates=8)          # ring of 64 slots
    srv.set_mode(mode)
    def run(ups, pulls, lr=0.25):
        vals = [(1.0 + rng.random(len(a))).astype(np.float32) for a in ups]
        begin = np.concatenate([[0], np.cumsum([len(a) for a in ups])[:-1]]).astype(np.uint64)
        count = np.array([len(a) for a in ups], np.uint32)
        idx = i32(np.concatenate(ups).astype(np.uint32))
        val = torch.from_numpy(np.concatenate(vals)).to(DEV)
        sigma = torch.full_like(idx, -1)
        srv.apply(idx, val, begin, count, np.array(pulls, np.uint64), lr, sigma_out=sigma)
        s = u32(sigma)
        for b, a in enumerate(ups):
            want = ref.apply(np.asarray(a, np.uint32), vals[b], int(pulls[b]), lr)
            assert np.array_equal(s[int(begin[b]):int(begin[b]) + len(a)], want), f"update {b}"
    u0 = np.arange(0, 30) * 100                            # update 0: positions 0 .. 29
    run([u0], [0])
    # one call: b0 pulled at 0 (window = update 0), 10 pairs on update 0's parameters (positions 30 .. 39);
    # b1 fresh, 30 pairs on update 0's parameters (positions 40 .. 69: the last six wrap onto slots 0 .. 5)
    run([u0[:10], u0], [0, 2])
    # the same shape again, further along the ring, with three updates in the call
    ts = srv.timestamp
    run([u0[5:15], u0[:15], u0[10:25]], [ts - 1, ts, ts + 1])          # 40 pairs: all the history the server keeps
    assert srv.last_error() == 0 and srv.timestamp == ref.timestamp
    assert np.array_equal(bits(theta), bits(ref.theta()))


@pytest.mark.parametrize("mode", MODES)
def test_every_update_names_the_same_parameters(binding, mode):
    """Forty updates that all name the same 300 parameters (plus a few of their own): inside a launch
    every parameter is changed by every update, so the order of the updates per parameter is all
    that keeps the result right.  Staleness counts and parameters bit for bit."""
    P = 50_000
    rng = np.random.default_rng(77)
    theta = torch.from_numpy(rng.standard_normal(P).astype(np.float32)).to(DEV)
    ref = oracle.Server(theta.cpu().numpy())
    srv = binding.Server(theta, history_pairs=1 << 18, max_window_updates=64)
    srv.set_mode(mode)
    common = np.sort(rng.choice(P, 300, replace=False))
    ts = 0
    for call in range(2):
        ups = [np.unique(np.concatenate([common, rng.choice(P, 20, replace=False)])).astype(np.uint32) for _ in range(40)]
        vals = [rng.standard_normal(a.size).astype(np.float32) for a in ups]
        begin = np.concatenate([[0], np.cumsum([a.size for a in ups])[:-1]]).astype(np.uint64)
        count = np.array([a.size for a in ups], np.uint32)
        pull = np.array([max(0, ts + b - int(rng.integers(0, 45))) for b in range(40)], np.uint64)
        idx, val = i32(np.concatenate(ups)), torch.from_numpy(np.concatenate(vals)).to(DEV)
        sigma = torch.full_like(idx, -1)
        srv.apply(idx, val, begin, count, pull, 0.05, sigma_out=sigma)
        s = u32(sigma)
        for b in range(40):
            want = ref.apply(ups[b], vals[b], int(pull[b]), 0.05)
            assert np.array_equal(s[int(begin[b]):int(begin[b]) + ups[b].size], want), f"call {call} update {b}"
        ts += 40
    assert srv.last_error() == 0 and srv.timestamp == ts == ref.timestamp
    assert np.array_equal(bits(theta), bits(ref.theta()))


def test_window_and_capacity_errors_leave_the_server_unchanged(binding):
    theta = torch.zeros(100, device=DEV)
    srv = binding.Server(theta, history_pairs=40, max_window_updates=8)     # ring of 64 pairs
    idx = i32(np.arange(10))
    val = torch.ones(10, device=DEV)
    one = lambda j: srv.apply(idx, val, [0], [10], [j], 0.1)
    for _ in range(6):
        one(0)                                              # positions 0 .. 59
    assert srv.timestamp == 6
    for bad_j in (7, 99):                                   # j > i
        with pytest.raises(binding.AdacompError) as e:
            one(bad_j)
        assert e.value.status == binding.ERR_WINDOW
    with pytest.raises(binding.AdacompError) as e:          # 70 positions back: update 0 would be overwritten
        one(0)
    assert e.value.status == binding.ERR_WINDOW
    with pytest.raises(binding.AdacompError) as e:          # too many updates in one call
        srv.apply(idx, val, [0] * 9, [1] * 9, [6] * 9, 0.1)
    assert e.value.status == binding.ERR_CAPACITY
    big = i32(np.arange(50))
    with pytest.raises(binding.AdacompError) as e:          # one call's pairs exceed history_pairs
        srv.apply(big, torch.ones(50, device=DEV), [0], [50], [6], 0.1)
    assert e.value.status == binding.ERR_CAPACITY
    assert srv.timestamp == 6 and srv.last_error() == 0
    sig = torch.empty(10, dtype=torch.int32, device=DEV)
    srv.apply(idx, val, [0], [10], [1], 0.1, sigma_out=sig)  # still usable; window = updates 1..5
    assert srv.timestamp == 7 and sig.tolist() == [5] * 10
    assert np.allclose(theta[:10].cpu().numpy(), -0.1 * (1 + 1 + 1 / 2 + 1 / 3 + 1 / 4 + 1 / 5 + 1 / 5), rtol=1e-6)
    for far_j in (0,):                                      # window longer than max_window_updates
        for _ in range(2):
            one(srv.timestamp)
        with pytest.raises(binding.AdacompError) as e:
            one(0)
        assert e.value.status == binding.ERR_WINDOW


@pytest.mark.parametrize("mode", MODES)
def test_bad_indices_are_reported_not_followed(binding, mode):
    theta = torch.zeros(10, device=DEV)
    srv = binding.Server(theta, history_pairs=64, max_window_updates=8)
    srv.set_mode(mode)
    srv.apply(i32([1, 2, 4_000_000_000]), torch.ones(3, device=DEV), [0], [3], [0], 0.5)
    assert srv.last_error() == binding.ERR_UNSORTED         # index >= n_params: skipped and reported
    assert srv.last_error() == 0                            # reading clears it
    assert theta.cpu().tolist() == [0, -0.5, -0.5, 0, 0, 0, 0, 0, 0, 0]
    srv.set_validation(True)
    srv.apply(i32([3, 3]), torch.ones(2, device=DEV), [0], [2], [1], 0.5)
    assert srv.last_error() == binding.ERR_UNSORTED


@pytest.mark.parametrize("mode", MODES)
def test_position_rebasing(binding, mode):
    wl = wlmod.workload(1).scaled(256, n_workers=10, n_rounds=6)
    ks = oracle_keep_counts(wl.tensor_sizes, (1, 10))
    K = int(sum(ks))
    theta = wlmod.initial_parameters(wl, DEV)
    ref = oracle.Server(theta.cpu().numpy())
    srv = binding.Server(theta, history_pairs=2 * wl.n_workers * K, max_window_updates=2 * wl.n_workers)
    srv.set_mode(mode)
    srv.debug_skip_positions(2**32 - 16 - 2 * wl.n_workers * K - K // 2)   # re-base falls inside round 2
    for r, rd in enumerate(wlmod.arrival_schedule(wl)):
        idx, val = wlmod.synthetic_updates(wl, ks, r, DEV)
        sigma = torch.empty_like(idx)
        srv.apply(idx.view(-1), val.view(-1), rd.order.astype(np.uint64) * np.uint64(K),
                  np.full(wl.n_workers, K, np.uint32), rd.pull_ts, wl.lr, sigma_out=sigma.view(-1))
        for b, w in enumerate(rd.order.tolist()):
            want = ref.apply(u32(idx)[w], val[w].cpu().numpy(), int(rd.pull_ts[b]), wl.lr)
            assert np.array_equal(u32(sigma)[w], want), f"round {r}"
    assert srv.last_error() == 0
    assert np.array_equal(bits(theta), bits(ref.theta()))


def test_pull_returns_timestamp_and_copy(binding):
    theta = torch.arange(8, dtype=torch.float32, device=DEV)
    srv = binding.Server(theta, history_pairs=16, max_window_updates=4)
    assert srv.pull() == 0
    srv.apply(i32([2]), torch.ones(1, device=DEV), [0], [1], [0], 1.0)
    copy = torch.empty_like(theta)
    assert srv.pull(copy) == 1
    torch.cuda.synchronize()
    assert copy.tolist() == [0, 1, 1, 3, 4, 5, 6, 7]
    fresh = torch.zeros(8, device=DEV)
    srv.reset(fresh)
    assert srv.pull() == 0
    srv.apply(i32([2]), torch.ones(1, device=DEV), [0], [1], [0], 1.0, sigma_out=(s := torch.zeros(1, dtype=torch.int32, device=DEV)))
    assert int(s[0]) == 0 and fresh[2].item() == -1.0 and theta[2].item() == 1.0   # history was forgotten


@pytest.mark.parametrize("n_workers,pad", [(5, 0), (11, 12), (16, 4)])
def test_select_from_host_memory(binding, n_workers, pad):
    """adacomp_select_host with several worker counts and a worker stride longer than the layout: the pairs that arrive in
    host memory are the oracle's, and the device staging buffers hold the same."""
    wl = wlmod.workload(0).scaled(16, n_workers=n_workers)
    keep = (1, 100)
    sel = binding.Selector(binding.make_segments(wl.tensor_sizes, keep), n_workers, DEV)
    K, W, P = sel.pairs_per_worker, n_workers, wl.n_params
    g = wlmod.round_gradients(wl, 0, "cpu")
    h_g = torch.zeros((W, P + pad)).pin_memory()
    h_g[:, :P] = g
    d_g = torch.empty((W, P + pad), device=DEV)
    d_idx = torch.empty((W, K), dtype=torch.int32, device=DEV)
    d_val = torch.empty((W, K), device=DEV)
    h_idx = torch.full((W, K), -1, dtype=torch.int32).pin_memory()
    h_val = torch.zeros((W, K)).pin_memory()
    for _ in range(2):
        sel.select_host(h_g, d_g, d_idx, d_val, h_idx, h_val)
    torch.cuda.current_stream().synchronize()
    assert sel.last_error()[0] == 0
    ks = oracle_keep_counts(wl.tensor_sizes, keep)
    for w in range(W):
        oi, ov = oracle.select_layers(g[w].numpy(), wl.offsets, wl.tensor_sizes, ks)
        assert np.array_equal(h_idx[w].numpy().view(np.uint32), oi) and np.array_equal(bits(h_val[w]), bits(ov))
    assert torch.equal(d_idx.cpu(), h_idx) and torch.equal(d_val.cpu().view(torch.int32), h_val.view(torch.int32))


def test_host_entry_points(binding):
    wl = wlmod.workload(0).scaled(16)
    keep = (1, 100)
    segs = binding.make_segments(wl.tensor_sizes, keep)
    sel = binding.Selector(segs, wl.n_workers, DEV)
    K, W, P = sel.pairs_per_worker, wl.n_workers, wl.n_params
    h_g = wlmod.round_gradients(wl, 0, "cpu").pin_memory()
    d_g = torch.empty((W, P), device=DEV)
    d_idx = torch.empty((W, K), dtype=torch.int32, device=DEV)
    d_val = torch.empty((W, K), device=DEV)
    h_idx = torch.empty((W, K), dtype=torch.int32).pin_memory()
    h_val = torch.empty((W, K)).pin_memory()
    sel.select_host(h_g, d_g, d_idx, d_val, h_idx, h_val)
    torch.cuda.synchronize()
    ks = oracle_keep_counts(wl.tensor_sizes, keep)
    for w in range(W):
        oi, ov = oracle.select_layers(h_g[w].numpy(), wl.offsets, wl.tensor_sizes, ks)
        assert np.array_equal(h_idx[w].numpy().view(np.uint32), oi) and np.array_equal(bits(h_val[w]), bits(ov))
    theta = wlmod.initial_parameters(wl, DEV)
    ref = oracle.Server(theta.cpu().numpy())
    srv = binding.Server(theta, history_pairs=W * K, max_window_updates=W)
    (rd,) = wlmod.arrival_schedule(wl)
    d_sig = torch.empty((W, K), dtype=torch.int32, device=DEV)
    h_sig = torch.empty((W, K), dtype=torch.int32).pin_memory()
    srv.apply_host(h_idx.view(-1), h_val.view(-1), rd.order.astype(np.uint64) * np.uint64(K), np.full(W, K, np.uint32),
                   rd.pull_ts, wl.lr, d_idx.view(-1), d_val.view(-1), d_sig.view(-1), h_sig.view(-1))
    torch.cuda.synchronize()
    for b, w in enumerate(rd.order.tolist()):
        want = ref.apply(h_idx[w].numpy().view(np.uint32), h_val[w].numpy(), int(rd.pull_ts[b]), wl.lr)
        assert np.array_equal(h_sig[w].numpy().view(np.uint32), want)
    assert np.array_equal(bits(theta), bits(ref.theta()))
