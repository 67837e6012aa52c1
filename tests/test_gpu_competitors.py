"""Parity of the competitors' path (ASGD: dense updates; Comp-ASGD: whole-model top-k or a random
selection; both with the learning rate divided by the update's staleness) with the CPU oracle,
through the C ABI: indices, values, staleness and parameters bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_1702_04683_b200 import workloads as wlmod

from helpers import bits, u32

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda", 0)


@pytest.fixture(scope="module")
def binding():
    from paper_1702_04683_b200 import binding as b
    return b


def test_comp_asgd_whole_model_top_k_pipeline(binding):
    """One segment over the whole parameter vector (the selection of Comp-ASGD is not per tensor),
    updates applied in arrival order under the global-staleness rule."""
    wl = wlmod.workload(1).scaled(16, n_workers=24, n_rounds=4)       # 204 664 parameters
    P = wl.n_params
    k = oracle.keep_count(P, 1, 100)
    sel = binding.Selector(binding.segments_from([0], [P], [k]), wl.n_workers, DEV)
    theta = wlmod.initial_parameters(wl, DEV)
    ref = oracle.Server(theta.cpu().numpy(), rule="global")
    srv = binding.Server(theta, history_pairs=1, max_window_updates=4 * wl.n_workers)
    srv.set_rule(1)
    srv.set_validation(True)
    max_sigma = 0
    for r, rd in enumerate(wlmod.arrival_schedule(wl)):
        g = wlmod.round_gradients(wl, r, DEV)
        idx, val = sel.select(g)
        g_host = g.cpu().numpy()
        sigma = torch.empty_like(idx)
        srv.apply(idx.view(-1), val.view(-1), rd.order.astype(np.uint64) * np.uint64(k),
                  np.full(wl.n_workers, k, np.uint32), rd.pull_ts, wl.lr, sigma_out=sigma.view(-1))
        for b, w in enumerate(rd.order.tolist()):
            oi, ov = oracle.select(g_host[w], k)
            assert np.array_equal(u32(idx[w]), oi) and np.array_equal(bits(val[w]), bits(ov)), f"round {r} worker {w}"
            want = ref.apply(oi, ov, int(rd.pull_ts[b]), wl.lr)
            assert np.array_equal(u32(sigma[w]), want), f"round {r} update {b}"
            max_sigma = max(max_sigma, int(want.max()))
    assert max_sigma >= wl.n_workers // 2                             # the schedule does produce stale updates
    assert sel.last_error()[0] == 0 and srv.last_error() == 0
    assert srv.timestamp == ref.timestamp
    assert np.array_equal(bits(theta), bits(ref.theta()))


@pytest.mark.parametrize("shift", [0, 1])
def test_asgd_dense_updates(binding, shift):
    """Dense pushes; with shift = 1 Theta and the update start 4 bytes past a 16-byte boundary and the
    parameter count is odd, so the vector path must not be taken for granted."""
    P = 1_000_003
    g = torch.Generator(device=DEV)
    g.manual_seed(7 + shift)
    buf = torch.randn(P + 8, device=DEV, generator=g)
    theta = buf[shift:shift + P]
    guard = buf[shift + P:].clone()
    ref = oracle.Server(theta.cpu().numpy(), rule="global")
    srv = binding.Server(theta, history_pairs=1, max_window_updates=8)
    srv.set_rule(1)
    rng = np.random.default_rng(5)
    for i in range(9):
        j = int(rng.integers(max(0, i - 4), i + 1))
        dbuf = torch.randn(P + 4, device=DEV, generator=g)
        delta = dbuf[shift:shift + P]
        delta[::7] = 0.0
        srv.apply_dense(delta, j, 0.05)
        ref.apply_dense(delta.cpu().numpy(), j, 0.05)
    assert srv.timestamp == ref.timestamp == 9 and srv.last_error() == 0
    assert np.array_equal(bits(theta), bits(ref.theta()))
    assert torch.equal(buf[shift + P:], guard)


def test_comp_asgd_random_selection(binding):
    """The selection is drawn by the caller (here: the first k of a seeded permutation, ascending);
    the library gathers the values and applies the updates."""
    P, W, k = 300_007, 6, 3_000
    g = torch.Generator(device=DEV)
    g.manual_seed(11)
    grads = torch.randn(W, P + 5, device=DEV, generator=g)[:, 2:P + 2]            # rows on odd addresses
    idx = torch.stack([torch.sort(torch.randperm(P, device=DEV, generator=g)[:k])[0] for _ in range(W)]).to(torch.int32)
    sel = binding.Selector(binding.segments_from([0], [P], [k]), W, DEV)
    val = sel.gather(grads, idx)
    assert sel.last_error()[0] == 0
    g_host = grads.cpu().numpy()
    for w in range(W):
        assert np.array_equal(bits(val[w]), bits(oracle.gather(g_host[w], u32(idx[w]))))
    theta = torch.zeros(P, device=DEV)
    ref = oracle.Server(np.zeros(P, np.float32), rule="global")
    srv = binding.Server(theta, history_pairs=1, max_window_updates=8)
    srv.set_rule(1)
    sigma = torch.empty_like(idx)
    pulls = [0, 0, 1, 0, 3, 5]
    srv.apply(idx.view(-1), val.view(-1), np.arange(W, dtype=np.uint64) * np.uint64(k), np.full(W, k, np.uint32),
              pulls, 0.1, sigma_out=sigma.view(-1))
    for w in range(W):
        assert np.array_equal(u32(sigma[w]), ref.apply(u32(idx[w]), val[w].cpu().numpy(), pulls[w], 0.1))
    assert np.array_equal(bits(theta), bits(ref.theta()))
    # an index outside the layout is reported and reads as zero
    bad = idx.clone()
    bad[2, 5] = P
    out = sel.gather(grads, bad)
    assert sel.last_error()[0] == binding.ERR_INVALID
    assert out[2, 5].item() == 0.0 and torch.equal(out[3], val[3])


def test_rule_switch_and_errors(binding):
    theta = torch.zeros(16, device=DEV)
    srv = binding.Server(theta, history_pairs=64, max_window_updates=8)
    idx = torch.arange(4, dtype=torch.int32, device=DEV)
    val = torch.ones(4, device=DEV)
    with pytest.raises(binding.AdacompError) as e:               # dense updates belong to rule 1
        srv.apply_dense(torch.ones(16, device=DEV), 0, 0.5)
    assert e.value.status == binding.ERR_INVALID
    srv.set_rule(1)
    srv.apply(idx, val, [0], [4], [0], 0.5)
    with pytest.raises(binding.AdacompError) as e:               # the other rule's history is missing by now
        srv.set_rule(0)
    assert e.value.status == binding.ERR_INVALID
    with pytest.raises(binding.AdacompError) as e:               # j > i
        srv.apply(idx, val, [0], [4], [2], 0.5)
    assert e.value.status == binding.ERR_WINDOW
    with pytest.raises(binding.AdacompError) as e:
        srv.apply_dense(torch.ones(16, device=DEV), 5, 0.5)
    assert e.value.status == binding.ERR_WINDOW
    assert srv.timestamp == 1
    sig = torch.empty(4, dtype=torch.int32, device=DEV)
    srv.apply(idx, val, [0, 0], [4, 0], [0, 0], 0.5, sigma_out=sig)        # staleness 1, then an empty update
    srv.apply_dense(torch.full((16,), 2.0, device=DEV), 1, 0.5)            # staleness 2
    assert srv.timestamp == 4 and sig.tolist() == [1, 1, 1, 1] and srv.last_error() == 0
    assert theta.cpu().tolist() == [-1.5] * 4 + [-0.5] * 12
    fresh = torch.zeros(16, device=DEV)
    srv.reset(fresh)
    srv.set_rule(0)                                                         # allowed again at timestamp 0
    srv.apply(idx, val, [0, 0], [4, 4], [0, 0], 0.5, sigma_out=(s2 := torch.empty(4, dtype=torch.int32, device=DEV)))
    assert s2.tolist() == [1, 1, 1, 1] and fresh[:4].cpu().tolist() == [-1.0] * 4
