"""Parity of adacomp_select (CUDA, through the C ABI) with the CPU oracle: indices and values
must match bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_1702_04683_b200 import workloads as wlmod

from helpers import bits, oracle_keep_counts, oracle_select_round, u32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_1702_04683_b200 import binding as b
    return b


def gpu_select(binding, grads, offsets, ns, ks, max_workers=None):
    segs = binding.segments_from(offsets, ns, ks)
    sel = binding.Selector(segs, max_workers or (grads.shape[0] if grads.dim() == 2 else 1), grads.device)
    idx, val = sel.select(grads)
    status, _ = sel.last_error()
    assert status == 0
    return u32(idx), val.cpu().numpy(), sel


def check_against_oracle(binding, grads, offsets, ns, ks):
    idx, val, _ = gpu_select(binding, grads, offsets, ns, ks)
    g_host = grads.cpu().numpy()
    if g_host.ndim == 1:
        g_host = g_host[None]
    for w in range(g_host.shape[0]):
        oi, ov = oracle.select_layers(g_host[w], offsets, ns, ks)
        assert np.array_equal(idx[w], oi), f"worker {w}: indices differ"
        assert np.array_equal(bits(val[w]), bits(ov)), f"worker {w}: values differ"


# ----------------------------------------------------------------------------- edge cases

def test_tiny_and_degenerate_segments(binding):
    dev = torch.device("cuda", 0)
    ns = [1, 2, 0, 7, 13, 64, 1001, 4096, 5, 3]
    ks = [1, 2, 0, 0, 13, 1, 17, 4096, 5, 1]
    offsets = np.concatenate([[0], np.cumsum(ns)[:-1]]).tolist()
    g = torch.randn(3, sum(ns), device=dev)
    check_against_oracle(binding, g, offsets, ns, ks)


def test_ties_zeros_and_inf(binding):
    dev = torch.device("cuda", 0)
    n = 300_000                              # three chunks with a ragged tail
    cases = {
        "all_equal": torch.full((n,), 0.5),
        "all_zero_mixed_sign": torch.where(torch.arange(n) % 3 == 0, torch.tensor(-0.0), torch.tensor(0.0)),
        "two_values": torch.where(torch.rand(n) < 0.5, torch.tensor(1.0), torch.tensor(-2.0)),
        "coarse_grid": torch.round(torch.randn(n) * 3) / 3,
        "with_inf": torch.cat([torch.randn(n - 4), torch.tensor([float("inf"), -float("inf"), 0.0, -0.0])]),
        "denormals": torch.randn(n) * 1e-42,
    }
    for name, g in cases.items():
        g = g.to(torch.float32).to(dev)
        for k in (1, 2, 1000, n // 2, n - 1, n):
            check_against_oracle(binding, g, [0], [n], [k])


def test_gaps_strides_and_unaligned_views(binding):
    dev = torch.device("cuda", 0)
    # segments with gaps between them, odd sizes, a worker stride larger than the extent and a
    # base pointer that is only 4-byte aligned
    offsets = [3, 1000, 140_001, 400_000]
    ns = [990, 139_000, 131_073, 262_145]
    ks = [10, 1390, 1311, 2622]
    extent = offsets[-1] + ns[-1]
    buf = torch.randn(4 * (extent + 37) + 3, device=dev)
    for shift in (0, 1, 2, 3):
        g = buf[shift:shift + 4 * (extent + 37)].view(4, extent + 37)
        assert g.data_ptr() % 16 == (buf.data_ptr() + 4 * shift) % 16
        check_against_oracle(binding, g, offsets, ns, ks)


def test_deterministic_and_input_untouched(binding):
    dev = torch.device("cuda", 0)
    wl = wlmod.workload(0)
    g = wlmod.round_gradients(wl, 0, dev)
    before = g.clone()
    ks = oracle_keep_counts(wl.tensor_sizes, (1, 100))
    a_idx, a_val, sel = gpu_select(binding, g, wl.offsets, wl.tensor_sizes, ks)
    idx2, val2 = sel.select(g)
    assert np.array_equal(a_idx, u32(idx2)) and np.array_equal(bits(a_val), bits(val2))
    assert torch.equal(g, before)


def test_fewer_workers_than_the_handle_allows(binding):
    dev = torch.device("cuda", 0)
    g = torch.randn(5, 50_000, device=dev)
    segs = binding.segments_from([0, 20_000], [20_000, 30_000], [200, 3000])
    sel = binding.Selector(segs, 8, dev)
    idx, val = sel.select(g[:2])
    for w in range(2):
        oi, ov = oracle.select_layers(g[w].cpu().numpy(), [0, 20_000], [20_000, 30_000], [200, 3000])
        assert np.array_equal(u32(idx)[w], oi) and np.array_equal(bits(val[w]), bits(ov))
    with pytest.raises(binding.AdacompError):
        sel.select(torch.randn(9, 50_000, device=dev))


def test_routes_agree_and_are_taken(binding):
    dev = torch.device("cuda", 0)
    wl = wlmod.workload(0)
    g = wlmod.round_gradients(wl, 0, dev)
    ks = oracle_keep_counts(wl.tensor_sizes, (1, 100))
    segs = binding.segments_from(wl.offsets, wl.tensor_sizes, ks)
    sel = binding.Selector(segs, wl.n_workers, dev)
    idx_a, val_a = sel.select(g)
    status, general = sel.last_error()
    assert status == 0 and general == 0            # the 832- and 10 250-entry tensors are selected on chip, the others bracketed
    sel.set_route(1)
    idx_g, val_g = sel.select(g)
    status, general = sel.last_error()
    assert status == 0 and general == 8 * 4
    assert torch.equal(idx_a, idx_g) and torch.equal(val_a.view(torch.int32), val_g.view(torch.int32))
    sel.set_route(0)
    idx_b, _ = sel.select(g)
    assert torch.equal(idx_a, idx_b) and sel.last_error() == (0, 0)


def test_three_routes_by_size_and_keep_fraction(binding):
    """Tensors shorter than 32 768 entries are selected whole in shared memory, longer tensors that
    keep more than a quarter take the general route, the rest the single-pass route: all against
    the oracle, with ties and every keep count at the edges."""
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(21)
    sizes = [1, 2, 31, 32, 33, 1000, 1024, 4097, 16_383, 16_384, 16_385, 20_000, 32_767, 40_000, 70_000]
    ks = [1, 2, 31, 1, 33, 999, 7, 4097, 5, 16_384, 100, 19_999, 300, 30_000, 700]
    offsets = np.concatenate([[0], np.cumsum(np.array(sizes) + 3)[:-1]]).tolist()   # odd gaps: unaligned tensors
    W = 3
    stride = offsets[-1] + sizes[-1] + 5
    g = rng.standard_normal((W, stride)).astype(np.float32)
    g[:, ::7] = np.round(g[:, ::7], 1)                     # ties
    g[1, ::5] = 0.0
    gt = torch.from_numpy(g).to(dev)
    sel = binding.Selector(binding.segments_from(offsets, sizes, ks), W, dev)
    idx, val = sel.select(gt)
    status, general = sel.last_error()
    assert status == 0 and general == W                    # 30 000 of 40 000 (fraction); every shorter tensor is on chip, whatever it keeps
    h_idx, h_val = idx.cpu().numpy().view(np.uint32), val.cpu().numpy()
    for w in range(W):
        oi, ov = oracle.select_layers(g[w], offsets, sizes, ks)
        assert np.array_equal(h_idx[w], oi) and np.array_equal(h_val[w].view(np.uint32), ov.view(np.uint32))


def test_awkward_value_layouts_stay_exact_and_ties_fall_back(binding):
    dev = torch.device("cuda", 0)
    n, k = 1_000_000, 10_000
    g = torch.randn(3, n, device=dev) * 1e-6
    # worker 0: every large entry sits in one contiguous block
    g[0, 500_000:510_000] = (1.0 + torch.rand(10_000, device=dev)) * torch.where(torch.rand(10_000, device=dev) < 0.5, -1.0, 1.0)
    # worker 1: sorted by magnitude
    g[1] = torch.sort(g[1].abs())[0]
    # worker 2: two magnitudes only, so the threshold value is shared by half a million entries and
    # no bracket can isolate it: the instance must be handed to the general route
    g[2] = torch.where(torch.rand(n, device=dev) < 0.5, 1.0, -2.0)
    idx, val, sel = gpu_select(binding, g, [0], [n], [k])
    for w in range(3):
        oi, ov = oracle.select(g[w].cpu().numpy(), k)
        assert np.array_equal(idx[w], oi) and np.array_equal(bits(val[w]), bits(ov))
    sel.select(g)
    assert sel.last_error() == (0, 1)


def test_dense_candidates_crowded_and_spread(binding):
    """Keep fractions of 5-20 %: spread-out data, data concentrated near zero, a stretch in which
    every entry is large (its pieces do not fit the scan kernel's stage and go to the lists
    directly) and a coarse grid with ties at every level (which may overflow the lists and fall
    back to the general route).  Either way the answer is exact."""
    dev = torch.device("cuda", 0)
    n = 1_500_001
    g = torch.randn(4, n + 3, device=dev)[:, 1:n + 1]
    g[1] = g[1] * torch.rand(n, device=dev) ** 4                       # heavy concentration near zero
    g[2, 200_000:420_000] *= 1000.0                                    # 220 000 large entries in one stretch
    g[3] = torch.round(g[3] * 8) / 8                                   # coarse grid: many ties at every level
    for k, general_expected in ((75_000, None), (150_000, None), (300_000, None)):
        segs = binding.segments_from([0], [n], [k])
        sel = binding.Selector(segs, 4, dev)
        idx, val = sel.select(g)
        status, general = sel.last_error()
        assert status == 0
        for w in range(4):
            oi, ov = oracle.select(g[w].cpu().numpy(), k)
            assert np.array_equal(u32(idx[w]), oi), (k, w)
            assert np.array_equal(bits(val[w]), bits(ov)), (k, w)
        assert general <= 1                                            # at most the tied worker fell back


@pytest.mark.parametrize("k", [40, 1_500, 6_000])
def test_low_keep_fractions_with_candidates_crowded_into_a_few_pieces(binding, k):
    """Keep fractions of 1/37 500 to 1/250 pick the form of the ordered write in which a lane takes a piece: evenly
    spread data (a few candidates per piece), a burst of large entries inside two pieces (far more than 32 candidates
    in a piece), data concentrated near zero, a coarse grid with ties at every level, two tensors of different
    lengths side by side, odd alignment."""
    dev = torch.device("cuda", 0)
    n, n2 = 1_500_001, 70_000
    gen = torch.Generator(device=dev)
    gen.manual_seed(100 + k)
    g = torch.randn((4, n + n2 + 5), device=dev, generator=gen)[:, 1:n + n2 + 1]
    g[1, 300_100:301_900] *= 50.0                                      # 1800 large entries in a row
    g[2, :n] *= torch.rand(n, device=dev, generator=gen) ** 4          # heavy concentration near zero
    g[3, :n] = torch.round(g[3, :n] * 4) / 4                           # coarse grid: many ties at every level
    k2 = max(1, k // 20)
    sel = binding.Selector(binding.segments_from([0, n], [n, n2], [k, k2]), 4, dev)
    for _ in range(2):
        idx, val = sel.select(g)
    status, general = sel.last_error()
    assert status == 0 and general <= 2                                 # at most the tied row's tensors fell back
    for w in range(4):
        oi, ov = oracle.select_layers(g[w].cpu().numpy(), [0, n], [n, n2], [k, k2])
        assert np.array_equal(u32(idx[w]), oi), (k, w)
        assert np.array_equal(bits(val[w]), bits(ov)), (k, w)


@pytest.mark.parametrize("k", [1, 1_500, 75_000, 300_000])
def test_cluster_route_on_large_tensors(binding, k):
    """Route 2: tensors of a million entries or more are selected by one thread-block cluster each, which
    keeps masks and candidate values on chip between the single pass and the ordered write.  Rows at odd
    alignments, a crowded stretch (its block's store overflows: handed to the general route), a coarse grid
    with thousands of ties at the threshold, a NaN (handed over), a shorter tensor beside the large one."""
    dev = torch.device("cuda", 0)
    n, n2 = 1_300_003, 200_000
    gen = torch.Generator(device=dev)
    gen.manual_seed(k)
    g = torch.randn((5, n + n2 + 7), device=dev, generator=gen)[:, 3:n + n2 + 3]
    g[1, :n] = torch.round(g[1, :n] * 8) / 8
    g[2, 100_000:400_000] *= 1000.0
    g[3, 777_777] = float("nan")
    g[4, :n] *= torch.rand(n, device=dev, generator=gen) ** 4
    k2 = 2_000
    sel = binding.Selector(binding.segments_from([0, n], [n, n2], [k, k2]), 5, dev)
    assert sel.route_info()["cluster_tensors"] == 1
    sel.set_route(2)
    idx, val = sel.select(g)
    status, general = sel.last_error()
    assert status == 0 and 1 <= general <= 3             # the NaN for sure; the crowded and the tied worker may join it
    g_host = g.cpu().numpy()
    for w in range(5):
        oi, ov = oracle.select_layers(g_host[w], [0, n], [n, n2], [k, k2])
        assert np.array_equal(u32(idx)[w], oi), w
        assert np.array_equal(bits(val[w]), bits(ov)), w
    sel.set_route(0)                                       # the same handle on the default route: same answer
    idx0, val0 = sel.select(g)
    assert sel.last_error()[0] == 0
    assert torch.equal(idx, idx0) and torch.equal(val.view(torch.int32), val0.view(torch.int32))


@pytest.mark.parametrize("n,k", [(32_768, 1), (32_768, 8192), (40_000, 400), (65_537, 700), (1 << 20, 1), (3_000_001, 30_001)])
def test_bracket_route_sizes(binding, n, k):
    dev = torch.device("cuda", 0)
    g = torch.randn(3, n + 5, device=dev)[:, 2:n + 2]          # rows start at odd alignments
    segs = binding.segments_from([0], [n], [k])
    sel = binding.Selector(segs, 3, dev)
    idx, val = sel.select(g)
    assert sel.last_error()[0] == 0
    for w in range(3):
        oi, ov = oracle.select(g[w].cpu().numpy(), k)
        assert np.array_equal(u32(idx[w]), oi) and np.array_equal(bits(val[w]), bits(ov))


def test_one_segment_over_a_hundred_million_entries(binding):
    """A tensor far longer than the resolve kernel's shared-memory span table (whole-model selection, an
    embedding table): still the single-pass route, still exact."""
    dev = torch.device("cuda", 0)
    n, k = 100_000_003, 1_000_001
    g = torch.randn(2, n + 3, device=dev)[:, 1:n + 1]
    g[1] *= torch.rand(n, device=dev)
    sel = binding.Selector(binding.segments_from([0], [n], [k]), 2, dev)
    idx, val = sel.select(g)
    assert sel.last_error() == (0, 0)                                  # nobody fell back to the general route
    idx64 = idx.to(torch.int64) & 0xFFFFFFFF
    assert bool((idx64[:, 1:] > idx64[:, :-1]).all()) and int(idx64.max()) < n
    assert torch.equal(torch.gather(g, 1, idx64).view(torch.int32), val.view(torch.int32))
    for w in range(2):
        oi, ov = oracle.select(g[w].cpu().numpy(), k)
        assert np.array_equal(u32(idx[w]), oi) and np.array_equal(bits(val[w]), bits(ov))


# ----------------------------------------------------------------------------- the workloads

def test_small_cnn_full_size(binding):
    wl = wlmod.workload(0)
    g = wlmod.round_gradients(wl, 0, torch.device("cuda", 0))
    ks = oracle_keep_counts(wl.tensor_sizes, wl.keep_fractions[0])
    assert sum(ks) == 32_748
    check_against_oracle(binding, g, wl.offsets, wl.tensor_sizes, ks)


@pytest.mark.parametrize("keep", [(1, 1000), (1, 100), (1, 10)])
def test_tie_stress_full_tensors(binding, keep):
    wl = wlmod.workload(2)
    g = wlmod.round_gradients(wl, 0, torch.device("cuda", 0), workers=range(6))
    ks = oracle_keep_counts(wl.tensor_sizes, keep)
    # the data really has ties at the threshold in the big tensor
    check_against_oracle(binding, g, wl.offsets, wl.tensor_sizes, ks)


def test_resnet50_shaped_full_tensors(binding):
    wl = wlmod.workload(3)
    g = wlmod.round_gradients(wl, 0, torch.device("cuda", 0), workers=range(3))
    ks = oracle_keep_counts(wl.tensor_sizes, wl.keep_fractions[0])
    assert sum(ks) == 127_874
    check_against_oracle(binding, g, wl.offsets, wl.tensor_sizes, ks)


@pytest.fixture(scope="module")
def large_flat_gradients():
    """Workload 4's 16 x 100 M gradients, generated once for the six keep fractions."""
    wl = wlmod.workload(4)
    g = wlmod.round_gradients(wl, 0, torch.device("cuda", 0))
    yield wl, g
    del g
    torch.cuda.empty_cache()


@pytest.mark.parametrize("keep", wlmod.workload(4).keep_fractions)
def test_large_flat_full_size_sampled(binding, large_flat_gradients, keep):
    """100 M parameters x 16 workers in the launch configuration the benchmark times, at every keep
    fraction it times; the oracle checks sampled (worker, tensor) selections one by one, and cheap
    invariants cover the rest."""
    dev = torch.device("cuda", 0)
    wl, g = large_flat_gradients
    ks = oracle_keep_counts(wl.tensor_sizes, keep)
    K = sum(ks)
    segs = binding.segments_from(wl.offsets, wl.tensor_sizes, ks)
    sel = binding.Selector(segs, wl.n_workers, dev)
    idx, val = sel.select(g)
    assert sel.last_error() == (0, 0)              # every selection stayed on the single-pass route
    # invariants at full size, on the GPU: ascending inside each tensor's slice, values are the
    # entries they name, indices stay inside their tensor
    idx64 = idx.view(wl.n_workers, len(ks), ks[0]).to(torch.int64) & 0xFFFFFFFF
    assert bool((idx64[:, :, 1:] > idx64[:, :, :-1]).all())
    lo = torch.tensor(wl.offsets, device=dev).view(1, -1, 1)
    assert bool(((idx64 >= lo) & (idx64 < lo + wl.tensor_sizes[0])).all())
    gathered = torch.gather(g, 1, idx64.view(wl.n_workers, K))
    assert torch.equal(gathered.view(torch.int32), val.view(torch.int32))
    del idx64, gathered
    # the oracle on sampled selections: 26 distinct (worker, tensor) pairs, the first and the last included
    rng = np.random.default_rng(keep[1])
    n_inst = wl.n_workers * len(ks)
    picks = set(rng.choice(n_inst, 24, replace=False).tolist()) | {0, n_inst - 1}
    for inst in sorted(picks):
        w, l = divmod(inst, len(ks))
        off, n = wl.offsets[l], wl.tensor_sizes[l]
        oi, ov = oracle.select(g[w, off:off + n].cpu().numpy(), ks[l], offset=off)
        lo_k = sum(ks[:l])
        assert np.array_equal(u32(idx[w, lo_k:lo_k + ks[l]]), oi), (w, l)
        assert np.array_equal(bits(val[w, lo_k:lo_k + ks[l]]), bits(ov)), (w, l)


# ----------------------------------------------------------------------------- NaN

def _nan_patterns():
    """Quiet, signalling and payload-carrying NaNs of both signs, as fp32 bit patterns."""
    return np.array([0x7FC00000, 0xFFC00000, 0x7FA00001, 0xFF800001, 0x7FC12345, 0x7FFFFFFF, 0xFFFFFFFF, 0x7F800001],
                    dtype=np.uint32)


def test_nan_orders_above_inf_on_every_route(binding):
    """The contract for NaN inputs: a NaN orders above +Inf by its bit pattern (sign dropped), the
    same on every route, values bit for bit.  One bracketed tensor (the single pass detects the NaN
    and hands the tensor to the general route), one tensor small enough for the on-chip route, one
    tensor that keeps more than a quarter (general route by plan)."""
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(404)
    sizes = [200_000, 9_000, 50_000]
    ks = [2_000, 90, 20_000]
    offsets = [0, 200_003, 209_010]
    stride = offsets[-1] + sizes[-1] + 1
    W = 4
    g = rng.standard_normal((W, stride)).astype(np.float32)
    nan = _nan_patterns()
    gb = g.view(np.uint32)
    # worker 0: no NaN anywhere; worker 1: NaNs in every tensor (fewer than k); worker 2: NaNs and
    # infinities together in the bracketed tensor; worker 3: more NaNs than k in the small tensor
    for off, n in zip(offsets, sizes):
        gb[1, off + rng.choice(n, nan.size, replace=False)] = nan
    pos = rng.choice(sizes[0], nan.size + 4, replace=False)
    gb[2, pos[:nan.size]] = nan
    g[2, pos[nan.size:]] = [np.inf, -np.inf, np.inf, -np.inf]
    many = rng.choice(sizes[1], 200, replace=False)
    gb[3, offsets[1] + many] = nan[rng.integers(0, nan.size, 200)]
    gt = torch.from_numpy(g).to(dev)
    assert np.array_equal(gt.cpu().numpy().view(np.uint32), gb)          # the copy kept every payload
    sel = binding.Selector(binding.segments_from(offsets, sizes, ks), W, dev)
    idx, val = sel.select(gt)
    status, general = sel.last_error()
    assert status == 0
    # general route: the third tensor of every worker (by plan) and the bracketed tensor of the two
    # workers whose single pass met a NaN
    assert general == W + 2
    h_idx, h_val = u32(idx), val.cpu().numpy()
    for w in range(W):
        oi, ov = oracle.select_layers(g[w], offsets, sizes, ks)
        assert np.array_equal(h_idx[w], oi), f"worker {w}: indices differ"
        assert np.array_equal(bits(h_val[w]), bits(ov)), f"worker {w}: values differ"
    # every NaN of worker 1 is among the kept entries of its tensor (it orders above everything finite)
    kept = set(h_idx[1].tolist())
    assert all(int(i) in kept for i in np.flatnonzero(np.isnan(g[1])))


def test_stage_timing_modes_leave_the_result_alone(binding):
    """Events around every kernel (1), around the pass over the gradient only (2), or none (0): the same pairs come
    out, the call count is the number of calls since the switch, and mode 2 reports that one stage only."""
    dev = torch.device("cuda", 0)
    n, k = 600_000, 3_000
    gen = torch.Generator(device=dev)
    gen.manual_seed(31)
    g = torch.randn((3, n), device=dev, generator=gen)
    sel = binding.Selector(binding.segments_from([0], [n], [k]), 3, dev)
    want_idx, want_val = sel.select(g)
    want_idx, want_val = want_idx.clone(), want_val.clone()
    for mode, calls in ((1, 3), (2, 2), (0, 1)):
        sel.set_profiling(mode)
        for _ in range(calls):
            idx, val = sel.select(g)
        assert torch.equal(idx, want_idx) and torch.equal(val.view(torch.int32), want_val.view(torch.int32))
        if mode:
            prof = sel.profile()
            assert prof.pop("calls") == calls
            timed = {name for name, ms in prof.items() if ms > 0}
            assert "bracket_scan" in timed
            assert (timed == {"bracket_scan"}) == (mode == 2)
    assert sel.last_error() == (0, 0)
    oi, ov = oracle.select(g[1].cpu().numpy(), k)
    assert np.array_equal(u32(want_idx[1]), oi) and np.array_equal(bits(want_val[1]), bits(ov))
