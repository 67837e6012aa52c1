"""Do the pins bite?  Each case plants one plausible mistake in a COPY of the oracle's source (on
the CPU, never in the CUDA path), builds it, and checks that at least one pin-style check fails
on it, while the untouched oracle passes them all."""
import ctypes
import itertools
import os
import subprocess
import sys
import tempfile

import numpy as np
import pytest

import oracle

SRC = os.path.join(os.path.dirname(oracle.__file__), "adacomp_oracle.cpp")

MUTATIONS = {
    "smaller magnitude first": ("if (ka != kb) return ka > kb;", "if (ka != kb) return ka < kb;"),
    "higher index wins ties": ("return a < b;\n    }\n};", "return a > b;\n    }\n};"),
    "sign bit kept in the key": ("return bits & 0x7FFFFFFFu;", "return bits;"),
    "floor instead of ceiling": ("(prod + c_den - 1) / c_den", "prod / c_den"),
    "window misses update j": ("for (uint64_t u = j; u < i; ++u)", "for (uint64_t u = j + 1; u < i; ++u)"),
    "list window misses update j": ("ts[t - 1] >= j", "ts[t - 1] > j"),
    "multiply by sigma": ("alpha / static_cast<float>(sigma_k)", "alpha * static_cast<float>(sigma_k)"),
    "gradient ascent": ("return theta_k - step;", "return theta_k + step;"),
    "zero values recorded": ("if (val[e] != 0.0f) {\n            s->theta[k] = updated_parameter(s->theta[k], alpha, sigma_k, val[e]);\n            changed.push_back(k);\n        }",
                             "s->theta[k] = updated_parameter(s->theta[k], alpha, sigma_k, val[e]);\n        changed.push_back(k);"),
    "no tick on empty update": ("    s->nonzero_idx.push_back(std::move(changed));\n    s->timestamp = i + 1;",
                                "    s->nonzero_idx.push_back(std::move(changed));\n    if (n_pairs) s->timestamp = i + 1;"),
}


def build_variant(text, tmpdir, name):
    src = os.path.join(tmpdir, name + ".cpp")
    lib = os.path.join(tmpdir, name + ".so")
    open(src, "w").write(text)
    subprocess.run(["g++", "-std=c++17", "-O1", "-ffp-contract=off", "-shared", "-fPIC", "-o", lib, src], check=True)
    L = ctypes.CDLL(lib)
    u32p, f32p = ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(ctypes.c_float)
    L.oracle_keep_count.restype = ctypes.c_uint32
    L.oracle_keep_count.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32]
    L.oracle_select.argtypes = [f32p, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint64, u32p, f32p]
    for kind in ("literal", "server"):
        getattr(L, f"oracle_{kind}_create").restype = ctypes.c_void_p
        getattr(L, f"oracle_{kind}_create").argtypes = [ctypes.c_uint64, f32p]
        getattr(L, f"oracle_{kind}_apply").argtypes = [ctypes.c_void_p, u32p, f32p, ctypes.c_uint64, ctypes.c_uint64,
                                                        ctypes.c_float, u32p]
        getattr(L, f"oracle_{kind}_theta").argtypes = [ctypes.c_void_p, f32p]
        getattr(L, f"oracle_{kind}_timestamp").restype = ctypes.c_uint64
        getattr(L, f"oracle_{kind}_timestamp").argtypes = [ctypes.c_void_p]
    return L


def p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def pins_hold(L) -> bool:
    """A compact version of the pins of test_oracle_select / test_oracle_apply, on a raw library."""
    # selection: unique valid subset on tiny tensors with ties and signs
    for g in ([1.0, -3.0, 3.0, 0.5, -0.0, 0.0], [2.0, 2.0, -2.0, 1.0], [-5.0, 4.0, 0.25]):
        g = np.array(g, dtype=np.float32)
        keys = (g.view(np.uint32) & 0x7FFFFFFF).astype(np.int64)
        for k in range(1, g.size):
            idx = np.zeros(k, np.uint32); val = np.zeros(k, np.float32)
            L.oracle_select(p(g, ctypes.c_float), g.size, k, 0, p(idx, ctypes.c_uint32), p(val, ctypes.c_float))
            valid = [s for s in itertools.combinations(range(g.size), k)
                     if all(keys[a] > keys[b] or (keys[a] == keys[b] and a < b) for a in s for b in range(g.size) if b not in s)]
            if tuple(int(i) for i in idx) != valid[0]:
                return False
    if [L.oracle_keep_count(n, 1, 100) for n in (832, 51_264)] != [9, 513]:
        return False
    for kind in ("literal", "server"):
        create, apply = getattr(L, f"oracle_{kind}_create"), getattr(L, f"oracle_{kind}_apply")
        theta_of, ts_of = getattr(L, f"oracle_{kind}_theta"), getattr(L, f"oracle_{kind}_timestamp")
        # Figure 2: pull, two foreign updates, own update -> staleness 2; with warm-up before the pull
        th = np.zeros(4, np.float32)
        h = create(4, p(th, ctypes.c_float))
        idx = np.array([1, 3], np.uint32); val = np.array([0.5, -1.0], np.float32); sig = np.zeros(2, np.uint32)
        for u in range(3):
            apply(h, p(idx, ctypes.c_uint32), p(val, ctypes.c_float), 2, u, 0.5, p(sig, ctypes.c_uint32))
        j = 3
        for u in range(2):
            apply(h, p(idx, ctypes.c_uint32), p(val, ctypes.c_float), 2, 3 + u, 0.5, p(sig, ctypes.c_uint32))
        apply(h, p(idx, ctypes.c_uint32), p(val, ctypes.c_float), 2, j, 0.5, p(sig, ctypes.c_uint32))
        if list(sig) != [2, 2]:
            return False
        # closed form with dyadic numbers: 5 updates at sigma 0 and one at sigma 2
        out = np.zeros(4, np.float32)
        theta_of(h, p(out, ctypes.c_float))
        if out[1] != np.float32(-(5 * 0.25 + 0.125)) or out[3] != np.float32(5 * 0.5 + 0.25) or out[0] != 0:
            return False
        # zero-valued pair: not a change; empty update still ticks
        z = np.array([0.0, 1.0], np.float32)
        apply(h, p(idx, ctypes.c_uint32), p(z, ctypes.c_float), 2, 6, 0.5, p(sig, ctypes.c_uint32))
        apply(h, p(idx, ctypes.c_uint32), p(val, ctypes.c_float), 0, 7, 0.5, p(sig, ctypes.c_uint32))
        apply(h, p(idx, ctypes.c_uint32), p(val, ctypes.c_float), 2, 6, 0.5, p(sig, ctypes.c_uint32))
        if list(sig) != [0, 1] or ts_of(h) != 9:
            return False
    return True


def test_untouched_oracle_passes_the_compact_pins():
    assert pins_hold(ctypes.CDLL(oracle.build()) and build_variant(open(SRC).read(), tempfile.mkdtemp(), "pristine"))


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(name):
    old, new = MUTATIONS[name]
    text = open(SRC).read()
    assert text.count(old) >= 1, "the mutation no longer matches the oracle's source"
    L = build_variant(text.replace(old, new), tempfile.mkdtemp(), "mutant")
    assert not pins_hold(L), f"no pin noticed: {name}"
