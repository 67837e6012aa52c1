"""adacomp_select_static: the selection entry point for callers that cannot allocate.

Some users of this library run where device memory cannot be requested: a plug-in inside another
framework's training step has no access to that framework's memory pool, a service that sized
its memory at start-up must not grow, and under memory pressure an allocation may stall the
device or fail.  For them the library carries a small fixed scratch array of its own, and
adacomp_select_static uses it instead of a caller-provided workspace.  This test checks, through
the C ABI, that it returns exactly what the regular entry point returns and what the CPU oracle
returns (indices and values bit for bit, the tolerance all selection tests use), twice in a row
with different inputs, since the second call finds the array as the first one left it; that
further calls leave the amount of free device memory where it was; and the edges of its own
geometry (a base that is only 4-byte aligned, the largest size it takes).  It is collected last
on purpose.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_1702_04683_b200 import binding as b
    return b


def regular_select(binding, g, k):
    segs = binding.segments_from([0], [g.numel()], [k])
    sel = binding.Selector(segs, 1, g.device)
    idx, val = sel.select(g)
    assert sel.last_error()[0] == 0
    return idx[0].clone(), val[0].clone()


def assert_is_oracle_selection(g, k, idx, val):
    want_idx, want_val = oracle.select(g.cpu().numpy(), k)
    assert np.array_equal(idx.cpu().numpy().view(np.uint32), want_idx)
    assert np.array_equal(val.cpu().numpy().view(np.uint32), want_val.view(np.uint32))


def test_static_entry_point_matches_regular_one_twice_in_a_row(binding):
    dev = torch.device("cuda", 0)
    gen = torch.Generator(device=dev)
    gen.manual_seed(20260)
    cases = [(300_001, 2_999), (1_000_000, 10_000)]              # ragged tail; several chunks
    inputs = [torch.randn(n, device=dev, generator=gen) for n, _ in cases]
    inputs[1] = torch.round(inputs[1] * 8) / 8                    # second call: heavy ties at the threshold
    # outputs are allocated before the calls: the entry point itself allocates nothing
    outs = [(torch.full((k,), -1, dtype=torch.int32, device=dev), torch.zeros(k, device=dev)) for _, k in cases]
    launches = binding.adacomp_kernel_launches()
    for g, (n, k), (idx, val) in zip(inputs, cases, outs):       # two calls back to back on one stream
        binding.adacomp_select_static(g, k, idx, val)
    assert binding.adacomp_select_static_last_error(0) == 0      # waits for the stream
    assert binding.adacomp_kernel_launches() == launches + 2 * 8
    for g, (n, k), (idx, val) in zip(inputs, cases, outs):
        want_idx, want_val = regular_select(binding, g, k)
        assert torch.equal(idx, want_idx)
        assert torch.equal(val.view(torch.int32), want_val.view(torch.int32))
        assert bool((idx[1:] > idx[:-1]).all())
        assert_is_oracle_selection(g, k, idx, val)


def test_static_entry_point_allocates_nothing_and_takes_awkward_geometry(binding):
    dev = torch.device("cuda", 0)
    gen = torch.Generator(device=dev)
    gen.manual_seed(777)
    n_max = 1 << 24                                              # the most the built-in scratch covers
    buf = torch.randn(n_max + 8, device=dev, generator=gen)
    odd = buf[1:200_002]                                         # 4 bytes past a 16-byte boundary, odd length
    assert odd.data_ptr() % 16 == 4
    big = buf[1:n_max + 1]                                       # with the odd base this needs every chunk slot of the scratch
    cases = [(odd, 1_234), (big, 5_000), (big[:n_max - 3], 1)]
    outs = [(torch.full((k,), -1, dtype=torch.int32, device=dev), torch.zeros(k, device=dev)) for _, k in cases]
    binding.adacomp_select_static(odd, 7, outs[0][0][:7], outs[0][1][:7])        # first call on the device: address look-up
    torch.cuda.synchronize()
    allocated, reserved = torch.cuda.memory_allocated(dev), torch.cuda.memory_reserved(dev)
    free_before, _ = torch.cuda.mem_get_info(dev)
    for (g, k), (idx, val) in zip(cases, outs):
        binding.adacomp_select_static(g, k, idx, val)
    assert binding.adacomp_select_static_last_error(0) == 0
    free_after, _ = torch.cuda.mem_get_info(dev)
    assert torch.cuda.memory_allocated(dev) == allocated and torch.cuda.memory_reserved(dev) == reserved
    assert free_after >= free_before                             # nothing was taken from the device behind torch's back
    for (g, k), (idx, val) in zip(cases, outs):
        assert_is_oracle_selection(g, k, idx, val)


def test_static_entry_point_limits(binding):
    dev = torch.device("cuda", 0)
    lib = binding.raw()
    g = torch.zeros(16, device=dev)
    idx = torch.zeros(16, dtype=torch.int32, device=dev)
    val = torch.zeros(16, device=dev)
    # one entry more than the built-in scratch covers: refused before anything is read or enqueued
    rc = lib.adacomp_select_static(g.data_ptr(), (1 << 24) + 1, 4, idx.data_ptr(), val.data_ptr(), 0, None)
    assert rc == binding.ERR_CAPACITY
    assert lib.adacomp_select_static(g.data_ptr(), 16, 17, idx.data_ptr(), val.data_ptr(), 0, None) == binding.ERR_INVALID
    assert lib.adacomp_select_static(None, 16, 4, idx.data_ptr(), val.data_ptr(), 0, None) == binding.ERR_INVALID
    # all of a tensor, and a single entry
    g = torch.tensor([0.5, -2.0, 0.0, 2.0, -0.0], device=dev)
    binding.adacomp_select_static(g, 5, idx[:5], val[:5])
    assert idx[:5].tolist() == [0, 1, 2, 3, 4] and torch.equal(val[:5], g)
    binding.adacomp_select_static(g, 1, idx[:1], val[:1])
    assert idx[:1].tolist() == [1] and val[:1].tolist() == [-2.0]
