"""Pins for the oracle's statement of the competitors' rule (ASGD, Comp-ASGD: "the learning rate is
divided by staleness and is global to each update") and of the gather that serves a selection made
elsewhere.  None of the expectations below is produced by the function under test."""
import ctypes
import os
import tempfile
from fractions import Fraction

import numpy as np
import pytest

import oracle
from test_oracle_mutations import SRC, build_variant, p

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "fig2_staleness.txt")


def f32(x):
    return np.asarray(x, dtype=np.float32)


def bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def test_paper_worked_example_gives_update_staleness_two():
    idx, val = np.array([0, 3, 5], dtype=np.uint32), f32([1.0, 2.0, -4.0])
    srv = oracle.Server(np.zeros(6, dtype=np.float32), rule="global")
    pulled, seen, expect = {}, {}, {}
    for line in open(GOLDEN):
        line = line.split("#")[0].split()
        if not line:
            continue
        if line[0] == "warmup_pushes":
            for _ in range(int(line[1])):
                srv.apply(idx, val, srv.timestamp, 0.5)
        elif line[0] == "pull":
            pulled[line[1]] = srv.timestamp
        elif line[0] == "push":
            seen[line[1]] = srv.apply(idx, val, pulled.pop(line[1], srv.timestamp), 0.5)
        elif line[0] == "expect":
            expect[line[1]] = int(line[2])
    assert expect == {"w2": 2}
    assert list(seen["w2"]) == [2, 2, 2] and list(seen["w1"]) == [0, 0, 0] and list(seen["w3"]) == [0, 0, 0]
    # 7 updates at staleness 0 and one at staleness 2, all dyadic: exact
    assert list(srv.theta()) == [-(7 * 0.5 + 0.25), 0, 0, -(7 * 1.0 + 0.5), 0, 7 * 2.0 + 1.0]


@pytest.mark.parametrize("literal", [False, True])
def test_full_updates_agree_with_the_per_parameter_rule(literal):
    """When every update names every parameter with a non-zero value, Eq. 3 counts every update of the
    window for every parameter: sigma_k = i - j, and the two rules are the same function."""
    rng = np.random.default_rng(21)
    P = 40
    theta0 = rng.standard_normal(P).astype(np.float32)
    a, b = oracle.Server(theta0, literal=literal), oracle.Server(theta0, rule="global")
    idx = np.arange(P, dtype=np.uint32)
    for i in range(15):
        j = int(rng.integers(max(0, i - 5), i + 1))
        g = rng.standard_normal(P).astype(np.float32)
        g[g == 0] = 1.0
        sa, sb = a.apply(idx, g, j, 0.05), b.apply(idx, g, j, 0.05)
        assert list(sa) == list(sb) == [i - j] * P
    assert np.array_equal(bits(a.theta()), bits(b.theta()))


def test_single_worker_is_plain_sgd_exact():
    rng = np.random.default_rng(22)
    P = 30
    theta0 = (rng.integers(-64, 64, P) / 16).astype(np.float32)
    srv = oracle.Server(theta0, rule="global")
    want = [Fraction(float(t)) for t in theta0]
    for _ in range(6):                                     # pulls right before each push: staleness 0
        idx = np.sort(rng.choice(P, 7, replace=False)).astype(np.uint32)
        val = (rng.integers(-32, 32, 7) / 8).astype(np.float32)
        assert list(srv.apply(idx, val, srv.timestamp, 0.25)) == [0] * 7
        for k, v in zip(idx, val):
            want[int(k)] -= Fraction(1, 4) * Fraction(float(v))
    assert [Fraction(float(t)) for t in srv.theta()] == want          # every intermediate is exact in fp32


def test_disjoint_sets_pulled_at_zero_are_divided_by_their_position():
    """Where the per-parameter rule sees no staleness at all (disjoint supports), the global rule
    divides update b's learning rate by b."""
    B, per = 9, 4
    theta0 = np.zeros(B * per, dtype=np.float32)
    glob, ada = oracle.Server(theta0, rule="global"), oracle.Server(theta0)
    vals = f32([3.0, -1.5, 0.75, 6.0])
    for b in range(B):
        idx = np.arange(b * per, (b + 1) * per, dtype=np.uint32)
        assert list(glob.apply(idx, vals, 0, 0.5)) == [b] * per
        assert list(ada.apply(idx, vals, 0, 0.5)) == [0] * per
    got = glob.theta()
    for b in range(B):
        for e, v in enumerate(vals):
            want = -Fraction(1, 2) / max(b, 1) * Fraction(float(v))
            assert abs(Fraction(float(got[b * per + e])) - want) <= abs(want) * Fraction(1, 2**22)
    assert np.array_equal(ada.theta(), np.tile(-0.5 * vals, B))


def test_dense_push_is_the_sparse_push_of_every_parameter():
    rng = np.random.default_rng(23)
    P = 257
    theta0 = rng.standard_normal(P).astype(np.float32)
    a, b = oracle.Server(theta0, rule="global"), oracle.Server(theta0, rule="global")
    for i in range(7):
        j = int(rng.integers(0, i + 1))
        g = rng.standard_normal(P).astype(np.float32)
        g[::5] = 0.0
        a.apply_dense(g, j, 0.1)
        b.apply(np.arange(P, dtype=np.uint32), g, j, 0.1)
    assert a.timestamp == b.timestamp == 7
    assert np.array_equal(bits(a.theta()), bits(b.theta()))
    # and against a dense fp32 axpy written with array operations, one rounding per operation
    th = theta0.copy()
    rng = np.random.default_rng(23)
    rng.standard_normal(P)
    for i in range(7):
        j = int(rng.integers(0, i + 1))
        g = rng.standard_normal(P).astype(np.float32)
        g[::5] = 0.0
        alpha = np.float32(0.1) / np.float32(i - j) if i != j else np.float32(0.1)
        th = (th - (alpha * g).astype(np.float32)).astype(np.float32)
    assert np.array_equal(bits(a.theta()), bits(th))


def test_every_entry_is_applied_as_written_and_every_update_ticks():
    theta0 = f32([-0.0, 1.0, -0.0, 2.0])
    srv = oracle.Server(theta0, rule="global")
    srv.apply(np.array([0, 1], np.uint32), f32([0.0, 0.0]), 0, 0.5)       # -0 - (+0) = -0 ; 1 - 0 = 1
    srv.apply(np.array([], np.uint32), f32([]), 0, 0.5)                  # empty: still an update
    srv.apply(np.array([2], np.uint32), f32([-0.0]), 1, 0.5)             # -0 - (-0) = +0 (IEEE subtraction)
    got = srv.theta()
    assert srv.timestamp == 3
    assert list(got) == [0.0, 1.0, 0.0, 2.0]
    assert list(np.signbit(got)) == [True, False, False, False]
    with pytest.raises(ValueError):
        srv.apply(np.array([1], np.uint32), f32([1.0]), 4, 0.5)          # j > i
    with pytest.raises(ValueError):
        srv.apply(np.array([2, 1], np.uint32), f32([1.0, 1.0]), 0, 0.5)  # not ascending
    with pytest.raises(ValueError):
        srv.apply(np.array([4], np.uint32), f32([1.0]), 0, 0.5)          # out of range
    assert srv.timestamp == 3 and np.array_equal(bits(srv.theta()), bits(got))
    with pytest.raises(ValueError):
        oracle.Server(theta0).apply_dense(theta0, 0, 0.5)                # dense pushes belong to the global rule


def test_gather_is_plain_indexing():
    rng = np.random.default_rng(24)
    g = rng.standard_normal(1000).astype(np.float32)
    g[[3, 7]] = [-0.0, np.float32("nan")]
    g.view(np.uint32)[9] = 0x7FC12345                                      # a NaN with a payload
    idx = np.concatenate([[3, 7, 9, 999, 0, 0], rng.integers(0, 1000, 500)]).astype(np.uint32)
    assert np.array_equal(bits(oracle.gather(g, idx)), bits(g[idx]))
    assert oracle.gather(g, np.array([], np.uint32)).size == 0
    with pytest.raises(ValueError):
        oracle.gather(g, np.array([1000], np.uint32))


# --------------------------------------------------------------------------- do these pins bite?

GLOBAL_MUTATIONS = {
    "staleness counts the update itself": ("const uint32_t sigma = static_cast<uint32_t>(i - j);\n    for (uint64_t e = 0; e < n_pairs; ++e) {",
                                           "const uint32_t sigma = static_cast<uint32_t>(i - j + 1);\n    for (uint64_t e = 0; e < n_pairs; ++e) {"),
    "dense push ignores staleness": ("for (size_t k = 0; k < s->theta.size(); ++k) s->theta[k] = updated_parameter(s->theta[k], alpha, sigma, delta[k]);",
                                     "for (size_t k = 0; k < s->theta.size(); ++k) s->theta[k] = updated_parameter(s->theta[k], alpha, 0, delta[k]);"),
    "no tick": ("        s->theta[idx[e]] = updated_parameter(s->theta[idx[e]], alpha, sigma, val[e]);\n    }\n    s->timestamp = i + 1;",
                "        s->theta[idx[e]] = updated_parameter(s->theta[idx[e]], alpha, sigma, val[e]);\n    }\n    if (n_pairs) s->timestamp = i + 1;"),
    "zero entries skipped": ("        s->theta[idx[e]] = updated_parameter(s->theta[idx[e]], alpha, sigma, val[e]);\n    }\n    s->timestamp = i + 1;",
                             "        if (val[e] != 0.0f) s->theta[idx[e]] = updated_parameter(s->theta[idx[e]], alpha, sigma, val[e]);\n    }\n    s->timestamp = i + 1;"),
    "gather off by one": ("val_out[e] = g[idx[e]];", "val_out[e] = g[idx[e] ? idx[e] - 1 : 0];"),
}


def global_pins_hold(L) -> bool:
    u32p, f32p = ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(ctypes.c_float)
    L.oracle_global_create.restype = ctypes.c_void_p
    L.oracle_global_create.argtypes = [ctypes.c_uint64, f32p]
    L.oracle_global_apply.argtypes = [ctypes.c_void_p, u32p, f32p, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_float, u32p]
    L.oracle_global_apply_dense.argtypes = [ctypes.c_void_p, f32p, ctypes.c_uint64, ctypes.c_float]
    L.oracle_global_theta.argtypes = [ctypes.c_void_p, f32p]
    L.oracle_global_timestamp.restype = ctypes.c_uint64
    L.oracle_global_timestamp.argtypes = [ctypes.c_void_p]
    L.oracle_gather.argtypes = [f32p, ctypes.c_uint64, u32p, ctypes.c_uint64, f32p]
    th = f32([0.0, -0.0, 0.0, 0.0])
    h = L.oracle_global_create(4, p(th, ctypes.c_float))
    idx, val, sig = np.array([0, 3], np.uint32), f32([1.0, -2.0]), np.zeros(2, np.uint32)
    for u in range(3):                                       # warm-up at staleness 0
        L.oracle_global_apply(h, p(idx, ctypes.c_uint32), p(val, ctypes.c_float), 2, u, 0.5, p(sig, ctypes.c_uint32))
    for u in range(2):                                       # Figure 2: two foreign updates after the pull at 3
        L.oracle_global_apply(h, p(idx, ctypes.c_uint32), p(val, ctypes.c_float), 2, 3 + u, 0.5, p(sig, ctypes.c_uint32))
    L.oracle_global_apply(h, p(idx, ctypes.c_uint32), p(val, ctypes.c_float), 2, 3, 0.5, p(sig, ctypes.c_uint32))
    if list(sig) != [2, 2]:
        return False
    dense = f32([4.0, 0.0, 0.0, 8.0])
    L.oracle_global_apply_dense(h, p(dense, ctypes.c_float), 2, 0.5)          # staleness 4
    L.oracle_global_apply(h, p(idx, ctypes.c_uint32), p(val, ctypes.c_float), 0, 7, 0.5, p(sig, ctypes.c_uint32))   # empty
    zero = f32([0.0, 0.0])
    one = np.array([1, 2], np.uint32)
    L.oracle_global_apply(h, p(one, ctypes.c_uint32), p(-zero, ctypes.c_float), 2, 8, 0.5, p(sig, ctypes.c_uint32))
    out = np.zeros(4, np.float32)
    L.oracle_global_theta(h, p(out, ctypes.c_float))
    if L.oracle_global_timestamp(h) != 9:
        return False
    if list(out) != [-(5 * 0.5 + 0.25 + 0.5), 0.0, 0.0, 5 * 1.0 + 0.5 - 1.0] or np.signbit(out[1]):
        return False
    g = f32([10.0, 11.0, 12.0, 13.0])
    got = np.zeros(3, np.float32)
    L.oracle_gather(p(g, ctypes.c_float), 4, p(np.array([3, 0, 2], np.uint32), ctypes.c_uint32), 3, p(got, ctypes.c_float))
    return list(got) == [13.0, 10.0, 12.0]


def test_untouched_oracle_passes_the_compact_global_pins():
    assert global_pins_hold(build_variant(open(SRC).read(), tempfile.mkdtemp(), "same"))


@pytest.mark.parametrize("name", sorted(GLOBAL_MUTATIONS))
def test_planted_mistake_in_the_global_rule_is_caught(name):
    old, new = GLOBAL_MUTATIONS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, "the mutation no longer matches the source"
    assert not global_pins_hold(build_variant(text.replace(old, new), tempfile.mkdtemp(), "mutant"))
