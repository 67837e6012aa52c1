"""The C-ABI boundary without a GPU: the library loads, exports every symbol the header
declares, and its host-side argument checks answer before any CUDA call is made."""
import ctypes
import math
import os
import re
from fractions import Fraction

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_1702_04683_b200 import build
    build.build()                       # nvcc cross-compiles without a GPU
    from paper_1702_04683_b200 import binding as b
    return b


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "adacomp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(adacomp_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(binding):
    names = declared_symbols()
    assert len(names) >= 20
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in adacomp.h but not exported"
    assert sorted(binding.EXPORTS) == names, "binding and header disagree on the entry points"


def test_status_strings_and_version(binding):
    assert binding.adacomp_version() >= 100
    assert binding.adacomp_status_string(0) == "ok"
    seen = {binding.adacomp_status_string(c) for c in range(0, -9, -1)}
    assert len(seen) == 9 and "unknown status" not in seen
    assert binding.adacomp_status_string(-99) == "unknown status"


def test_keep_count_rule(binding):
    # hand-computed values (the same ones the oracle is pinned to)
    assert [binding.adacomp_keep_count(n, 1, 100) for n in (832, 51_264, 3_212_288, 10_250)] == [9, 513, 32_123, 103]
    assert binding.adacomp_keep_count(64, 5, 1000) == 1
    assert binding.adacomp_keep_count(2_359_296, 5, 1000) == 11_797
    assert binding.adacomp_keep_count(0, 1, 10) == 0
    assert binding.adacomp_keep_count(10, 1, 1) == 10
    rng = np.random.default_rng(0)
    for _ in range(500):
        n = int(rng.integers(1, 2**32 - 1))
        den = int(rng.integers(1, 2**31))
        num = int(rng.integers(0, den + 1))
        assert binding.adacomp_keep_count(n, num, den) == min(n, max(1, math.ceil(Fraction(n * num, den))))
    for bad in ((10, 1, 0), (10, 3, 2), (2**32, 1, 2)):
        with pytest.raises(binding.AdacompError) as e:
            binding.adacomp_keep_count(*bad)
        assert e.value.status == binding.ERR_INVALID


def _ws_bytes(binding, segs, workers):
    n = ctypes.c_size_t(0)
    rc = binding.raw().adacomp_select_workspace_bytes(segs, len(segs), workers, ctypes.byref(n))
    return rc, n.value


def test_select_layout_checks(binding):
    ok = binding.segments_from([0, 100], [100, 50], [10, 5])
    rc, nbytes = _ws_bytes(binding, ok, 4)
    assert rc == 0 and nbytes > 0 and nbytes % 256 == 0
    assert _ws_bytes(binding, ok, 8)[1] > nbytes                       # grows with the worker count
    assert _ws_bytes(binding, binding.segments_from([0], [10], [11]), 1)[0] == binding.ERR_INVALID   # k > n
    assert _ws_bytes(binding, binding.segments_from([0, 50], [100, 50], [1, 1]), 1)[0] == binding.ERR_INVALID  # overlap
    assert _ws_bytes(binding, binding.segments_from([100, 0], [10, 10], [1, 1]), 1)[0] == binding.ERR_INVALID  # order
    assert _ws_bytes(binding, ok, 0)[0] == binding.ERR_INVALID
    assert _ws_bytes(binding, binding.segments_from([2**32 - 10], [100], [1]), 1)[0] == binding.ERR_INVALID
    # empty tensors and k = 0 are legal
    assert _ws_bytes(binding, binding.segments_from([0, 0, 7], [0, 7, 3], [0, 0, 3]), 2)[0] == 0


def test_create_rejects_bad_workspace_before_touching_cuda(binding):
    lib = binding.raw()
    segs = binding.segments_from([0], [100], [10])
    h = ctypes.c_void_p()
    assert lib.adacomp_select_create(ctypes.byref(h), segs, 1, 1, None, 1 << 20, 0) == binding.ERR_INVALID
    assert lib.adacomp_select_create(ctypes.byref(h), segs, 1, 1, ctypes.c_void_p(0x1001), 1 << 20, 0) == binding.ERR_INVALID
    assert h.value is None
    s = ctypes.c_void_p()
    assert lib.adacomp_server_create(ctypes.byref(s), 100, 100, 8, None, 1 << 20, 0) == binding.ERR_INVALID
    assert lib.adacomp_server_create(ctypes.byref(s), 0, 100, 8, ctypes.c_void_p(0x1000), 1 << 20, 0) == binding.ERR_INVALID
    assert lib.adacomp_server_create(ctypes.byref(s), 100, 2**31, 8, ctypes.c_void_p(0x1000), 1 << 20, 0) == binding.ERR_INVALID
    assert lib.adacomp_server_create(ctypes.byref(s), 100, 100, 2**24, ctypes.c_void_p(0x1000), 1 << 20, 0) == binding.ERR_INVALID
    assert lib.adacomp_server_create(ctypes.byref(s), 100, 100, 8, ctypes.c_void_p(0x1000), 16, 0) == binding.ERR_ALLOC
    n = ctypes.c_size_t(0)
    assert lib.adacomp_server_workspace_bytes(1000, 5000, ctypes.byref(n)) == 0
    assert n.value >= 1000 * 4 + 8192 * 4
    assert lib.adacomp_server_workspace_bytes(2**32, 5000, ctypes.byref(n)) == binding.ERR_INVALID


def test_null_handles_are_refused(binding):
    lib = binding.raw()
    ts = ctypes.c_uint64(0)
    assert lib.adacomp_select(None, None, 0, 1, None, None, None) == binding.ERR_INVALID
    assert lib.adacomp_apply(None, None, None, None, None, None, 1, 0.1, None, None) == binding.ERR_INVALID
    assert lib.adacomp_server_timestamp(None, ctypes.byref(ts)) == binding.ERR_INVALID
    assert lib.adacomp_server_reset(None, None, None) == binding.ERR_INVALID
    assert lib.adacomp_select_destroy(None) == 0 and lib.adacomp_server_destroy(None) == 0


def test_binding_has_no_cpu_path():
    # the binding must not import the oracle or fall back to anything on the CPU
    src = open(os.path.join(ROOT, "paper_1702_04683_b200", "binding.py")).read()
    assert "import oracle" not in src and "from oracle" not in src
    for f in os.listdir(os.path.join(ROOT, "paper_1702_04683_b200", "csrc")):
        assert "oracle" not in open(os.path.join(ROOT, "paper_1702_04683_b200", "csrc", f)).read()
