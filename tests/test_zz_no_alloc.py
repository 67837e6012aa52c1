"""adacomp_select_static: the selection entry point for callers that cannot allocate.

Some users of this library run where device memory cannot be requested: a plug-in inside another
framework's training step has no access to that framework's memory pool, a service that sized
its memory at start-up must not grow, and under memory pressure an allocation may stall the
device or fail.  For them the library carries a small fixed scratch array of its own, and
adacomp_select_static uses it instead of a caller-provided workspace.  This test checks, through
the C ABI, that it returns exactly what the regular entry point returns (indices and values bit
for bit, the tolerance all selection tests use), twice in a row with different inputs, since
the second call finds the array as the first one left it.  It is collected last on purpose.
"""
import ctypes

import numpy as np
import pytest
import torch

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
    torch.cuda.synchronize()
    assert binding.adacomp_kernel_launches() == launches + 2 * 8
    for g, (n, k), (idx, val) in zip(inputs, cases, outs):
        want_idx, want_val = regular_select(binding, g, k)
        assert torch.equal(idx, want_idx)
        assert torch.equal(val.view(torch.int32), want_val.view(torch.int32))
        assert bool((idx[1:] > idx[:-1]).all())


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
