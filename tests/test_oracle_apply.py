"""Pins for the oracle's parameter server (Algorithm 2, Eq. 3-5): the paper's worked
staleness example, brute-force set counting, closed forms in exact rational
arithmetic, invariants and degenerate cases."""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "fig2_staleness.txt")
KINDS = [True, False]   # literal membership form, per-parameter list form


def f32(x):
    return np.asarray(x, dtype=np.float32)


# --------------------------------------------------------------------------- worked example

def replay_golden(literal):
    """Replays the event list of the fixture; every push names the same three parameters, so
    the per-parameter staleness of each entry equals the update's global staleness."""
    idx = np.array([1, 4, 6], dtype=np.uint32)
    val = f32([0.5, -0.25, 1.0])
    srv = oracle.Server(np.zeros(8, dtype=np.float32), literal=literal)
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
            j = pulled.pop(line[1], srv.timestamp)   # a worker with no recorded pull pulled just now
            seen[line[1]] = srv.apply(idx, val, j, 0.5)
        elif line[0] == "expect":
            expect[line[1]] = int(line[2])
    return seen, expect


@pytest.mark.parametrize("literal", KINDS)
def test_paper_worked_example(literal):
    seen, expect = replay_golden(literal)
    assert expect == {"w2": 2}
    assert list(seen["w2"]) == [2, 2, 2]
    assert list(seen["w1"]) == [0, 0, 0] and list(seen["w3"]) == [0, 0, 0]


# --------------------------------------------------------------------------- brute force on sets

def random_pushes(rng, P, n_pushes, max_pairs, zero_frac=0.0, max_lag=6):
    pushes = []
    for i in range(n_pushes):
        m = int(rng.integers(0, max_pairs + 1))
        idx = np.sort(rng.choice(P, size=min(m, P), replace=False)).astype(np.uint32)
        val = rng.standard_normal(idx.size).astype(np.float32)
        val[rng.random(idx.size) < zero_frac] = 0.0
        j = i - int(rng.integers(0, min(i, max_lag) + 1))
        pushes.append((idx, val, j))
    return pushes


def brute_force_sigmas(pushes):
    """Eq. 3 with Python sets: S_u = parameters changed by update u with a non-zero value."""
    S, out = [], []
    for i, (idx, val, j) in enumerate(pushes):
        out.append([sum(1 for u in range(j, i) if int(k) in S[u]) for k in idx])
        S.append({int(k) for k, v in zip(idx, val) if v != 0.0})
    return out, S


@pytest.mark.parametrize("literal", KINDS)
@pytest.mark.parametrize("zero_frac", [0.0, 0.3])
def test_sigma_equals_set_counting(literal, zero_frac):
    rng = np.random.default_rng(11)
    for trial in range(30):
        P = int(rng.integers(4, 40))
        pushes = random_pushes(rng, P, int(rng.integers(1, 25)), P, zero_frac)
        want, S = brute_force_sigmas(pushes)
        srv = oracle.Server(np.zeros(P, dtype=np.float32), literal=literal)
        for i, (idx, val, j) in enumerate(pushes):
            got = srv.apply(idx, val, j, 0.01)
            assert list(got) == want[i]
            assert all(0 <= s <= i - j for s in got)                       # sigma_k <= global staleness
            # sum of sigma = sum over the window of the overlap with the update's index set
            assert int(got.sum()) == sum(len(S[u] & {int(k) for k in idx}) for u in range(j, i))
        assert srv.timestamp == len(pushes)


@pytest.mark.parametrize("literal", KINDS)
def test_identical_sets_give_global_staleness_and_disjoint_sets_give_zero(literal):
    rng = np.random.default_rng(12)
    P, B = 64, 9
    idx = np.sort(rng.choice(P, 10, replace=False)).astype(np.uint32)
    srv = oracle.Server(np.zeros(P, dtype=np.float32), literal=literal)
    for i in range(B):
        j = int(rng.integers(0, i + 1))
        assert list(srv.apply(idx, f32(np.ones(10)), j, 0.1)) == [i - j] * 10
    srv = oracle.Server(np.zeros(P, dtype=np.float32), literal=literal)
    for i in range(8):
        part = np.arange(i * 8, i * 8 + 8, dtype=np.uint32)
        assert list(srv.apply(part, f32(np.ones(8)), 0, 0.1)) == [0] * 8


# --------------------------------------------------------------------------- closed forms

@pytest.mark.parametrize("literal", KINDS)
def test_single_worker_is_plain_sparse_sgd_exact(literal):
    # one worker pulls right before each push (j = i): Eq. 4 reduces to Theta - alpha * sum(v)
    # (Eq. 2).  Dyadic values keep every fp32 operation exact, so the pin is exact.
    rng = np.random.default_rng(13)
    P = 32
    theta0 = (rng.integers(-64, 65, size=P) / 8.0).astype(np.float32)
    srv = oracle.Server(theta0, literal=literal)
    want = [Fraction(float(t)) for t in theta0]
    alpha = 0.5
    for i in range(40):
        idx = np.sort(rng.choice(P, 5, replace=False)).astype(np.uint32)
        val = (rng.integers(-32, 33, size=5) / 16.0).astype(np.float32)
        sig = srv.apply(idx, val, i, alpha)
        assert not sig.any()
        for k, v in zip(idx, val):
            want[int(k)] -= Fraction(alpha) * Fraction(float(v))
    got = srv.theta()
    assert [Fraction(float(t)) for t in got] == want


@pytest.mark.parametrize("literal", KINDS)
def test_same_set_all_pulled_at_zero_harmonic_closed_form(literal):
    # B updates naming the same parameters with the same values, all pulled at 0: update b has
    # sigma = b, so Theta = Theta0 - alpha * v * (1 + sum_{s=1}^{B-1} 1/s).
    P, B, alpha = 16, 12, 0.01
    rng = np.random.default_rng(14)
    theta0 = rng.standard_normal(P).astype(np.float32)
    idx = np.arange(0, P, 2, dtype=np.uint32)
    val = rng.standard_normal(idx.size).astype(np.float32)
    srv = oracle.Server(theta0, literal=literal)
    for b in range(B):
        assert list(srv.apply(idx, val, 0, alpha)) == [b] * idx.size
    h = 1 + sum(Fraction(1, s) for s in range(1, B))
    got = srv.theta()
    for t, (k, v) in enumerate(zip(idx, val)):
        want = Fraction(float(theta0[k])) - Fraction(float(np.float32(alpha))) * Fraction(float(v)) * h
        assert abs(Fraction(float(got[k])) - want) <= abs(want) * Fraction(1, 10**6)
    odd = np.arange(1, P, 2)
    assert np.array_equal(got[odd].view(np.uint32), theta0[odd].view(np.uint32))
    # with B = 3 and dyadic data the factor is 1 + 1 + 1/2 and everything is exact
    srv = oracle.Server(np.zeros(4, dtype=np.float32), literal=literal)
    for _ in range(3):
        srv.apply(np.array([2], dtype=np.uint32), f32([0.75]), 0, 0.5)
    assert Fraction(float(srv.theta()[2])) == -Fraction(1, 2) * Fraction(3, 4) * Fraction(5, 2)


@pytest.mark.parametrize("literal", KINDS)
def test_full_updates_reduce_to_global_staleness_rule(literal):
    # c = 1: every update names every parameter, so sigma_k is the update's global staleness and
    # Algorithm 2 is the dense rule "learning rate divided by staleness" the paper compares with.
    rng = np.random.default_rng(15)
    P, alpha = 50, np.float32(0.01)
    theta = rng.standard_normal(P).astype(np.float32)
    srv = oracle.Server(theta, literal=literal)
    idx = np.arange(P, dtype=np.uint32)
    for i in range(12):
        j = int(rng.integers(0, i + 1))
        g = rng.standard_normal(P).astype(np.float32)
        g[g == 0] = 1.0
        srv.apply(idx, g, j, float(alpha))
        a = alpha / np.float32(i - j) if i != j else alpha
        theta = (theta - (np.float32(a) * g).astype(np.float32)).astype(np.float32)   # dense axpy, fp32
    assert np.array_equal(srv.theta().view(np.uint32), theta.view(np.uint32))


@pytest.mark.parametrize("literal", KINDS)
def test_disjoint_updates_commute_bit_exactly(literal):
    rng = np.random.default_rng(16)
    P = 90
    theta0 = rng.standard_normal(P).astype(np.float32)
    parts = [np.arange(s, s + 10, dtype=np.uint32) for s in range(0, 90, 10)]
    vals = [rng.standard_normal(10).astype(np.float32) for _ in parts]
    results = []
    for perm in (np.arange(9), rng.permutation(9), rng.permutation(9)):
        srv = oracle.Server(theta0, literal=literal)
        for p in perm:
            assert not srv.apply(parts[p], vals[p], 0, 0.01).any()
        results.append(srv.theta().view(np.uint32))
    assert np.array_equal(results[0], results[1]) and np.array_equal(results[0], results[2])


@pytest.mark.parametrize("literal", KINDS)
def test_double_precision_reevaluation_per_update(literal):
    rng = np.random.default_rng(17)
    P = 40
    pushes = random_pushes(rng, P, 30, 20)
    theta = rng.standard_normal(P).astype(np.float32)
    srv = oracle.Server(theta, literal=literal)
    for idx, val, j in pushes:
        before = srv.theta().astype(np.float64)
        sig = srv.apply(idx, val, j, 0.01)
        after = srv.theta().astype(np.float64)
        a = np.where(sig == 0, 0.01, 0.01 / np.maximum(sig, 1))
        want = before.copy()
        want[idx] -= a * val.astype(np.float64)
        scale = np.maximum(np.abs(want), np.abs(before))       # one update: error relative to operands
        assert np.all(np.abs(after - want) <= 1e-6 * np.maximum(scale, 1e-30))


# --------------------------------------------------------------------------- degenerate cases

@pytest.mark.parametrize("literal", KINDS)
def test_zero_valued_entries_are_not_changes(literal):
    theta0 = f32([-0.0, 1.0, 2.0, -0.0])
    srv = oracle.Server(theta0, literal=literal)
    idx = np.array([0, 1, 3], dtype=np.uint32)
    assert list(srv.apply(idx, f32([0.0, 1.0, -0.0]), 0, 0.5)) == [0, 0, 0]
    # parameter 0 and 3 keep their sign bit: they were not rewritten
    assert np.array_equal(srv.theta().view(np.uint32), f32([-0.0, 0.5, 2.0, -0.0]).view(np.uint32))
    # a second update pulled at 0 sees one change on parameter 1 only
    assert list(srv.apply(idx, f32([1.0, 1.0, 1.0]), 0, 0.5)) == [0, 1, 0]
    assert srv.timestamp == 2


@pytest.mark.parametrize("literal", KINDS)
def test_empty_update_still_ticks_and_counts_in_no_window(literal):
    srv = oracle.Server(np.zeros(4, dtype=np.float32), literal=literal)
    e = np.array([], dtype=np.uint32)
    srv.apply(e, f32([]), 0, 0.1)
    srv.apply(np.array([1], dtype=np.uint32), f32([1.0]), 0, 0.1)
    srv.apply(e, f32([]), 2, 0.1)
    assert srv.timestamp == 3
    assert list(srv.apply(np.array([1], dtype=np.uint32), f32([1.0]), 0, 0.1)) == [1]


@pytest.mark.parametrize("literal", KINDS)
def test_untouched_parameters_keep_their_bits(literal):
    rng = np.random.default_rng(18)
    P = 200
    theta0 = rng.standard_normal(P).astype(np.float32)
    pushes = random_pushes(rng, 100, 20, 30)          # only parameters < 100 are ever named
    srv = oracle.Server(theta0, literal=literal)
    named = set()
    for idx, val, j in pushes:
        srv.apply(idx, val, j, 0.01)
        named |= {int(k) for k in idx}
    rest = np.array(sorted(set(range(P)) - named))
    assert np.array_equal(srv.theta()[rest].view(np.uint32), theta0[rest].view(np.uint32))


@pytest.mark.parametrize("literal", KINDS)
def test_bad_pushes_are_refused(literal):
    srv = oracle.Server(np.zeros(4, dtype=np.float32), literal=literal)
    with pytest.raises(ValueError):
        srv.apply(np.array([0], dtype=np.uint32), f32([1.0]), 1, 0.1)      # j > i
    with pytest.raises(ValueError):
        srv.apply(np.array([2, 1], dtype=np.uint32), f32([1.0, 1.0]), 0, 0.1)
    with pytest.raises(ValueError):
        srv.apply(np.array([4], dtype=np.uint32), f32([1.0]), 0, 0.1)
    assert srv.timestamp == 0


# --------------------------------------------------------------------------- the forms agree

def test_three_forms_agree_on_random_sequences():
    rng = np.random.default_rng(19)
    for trial in range(25):
        P = int(rng.integers(8, 120))
        pushes = random_pushes(rng, P, int(rng.integers(1, 40)), P // 2, zero_frac=0.1, max_lag=12)
        theta0 = rng.standard_normal(P).astype(np.float32)
        a = oracle.Server(theta0, literal=True)
        b = oracle.Server(theta0, literal=False)
        sig_all = []
        for idx, val, j in pushes:
            sa, sb = a.apply(idx, val, j, 0.01), b.apply(idx, val, j, 0.01)
            assert np.array_equal(sa, sb)
            sig_all.append(sa)
        ta, tb = a.theta(), b.theta()
        assert np.array_equal(ta.view(np.uint32), tb.view(np.uint32))
        # one parameter at a time, by searching each update's sorted index list
        idx_cat = np.concatenate([p[0] for p in pushes]) if pushes else np.zeros(0, np.uint32)
        val_cat = np.concatenate([p[1] for p in pushes]) if pushes else np.zeros(0, np.float32)
        begin = np.concatenate([[0], np.cumsum([p[0].size for p in pushes])]).astype(np.uint64)
        pull = np.array([p[2] for p in pushes], dtype=np.uint64)
        for k in rng.choice(P, size=min(P, 10), replace=False):
            sig_k, theta_k = oracle.parameter_trace(int(k), float(theta0[k]), idx_cat, val_cat, begin, pull, 0.01)
            want = [int(s[np.nonzero(p[0] == k)[0][0]]) for s, p in zip(sig_all, pushes) if (p[0] == k).any()]
            assert list(sig_k) == want
            assert np.float32(theta_k).view(np.uint32) == ta[k].view(np.uint32)
