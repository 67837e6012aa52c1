"""Pins for the oracle's SELECT_GRAD (Algorithm 1).  None of these expectations is
produced by the oracle itself: they come from enumerating subsets, from the
pairwise form of the definition, from library routines on special cases and from
hand-computed keep counts."""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle


def key_of(g):
    return np.asarray(g, dtype=np.float32).view(np.uint32) & np.uint32(0x7FFFFFFF)


def check_is_the_selection(g, k, idx, val, offset=0):
    """Pairwise statement of the rule: every kept entry beats every dropped entry under
    (larger magnitude, then lower index).  With a strict total order exactly one k-subset
    passes, so this identifies the answer without sorting anything."""
    g = np.asarray(g, dtype=np.float32)
    n = g.size
    assert idx.dtype == np.uint32 and val.dtype == np.float32
    assert idx.size == k and val.size == k
    loc = idx.astype(np.int64) - offset
    assert np.all(loc >= 0) and np.all(loc < n)
    assert np.all(np.diff(loc) > 0), "indices must be strictly ascending"
    assert np.array_equal(val.view(np.uint32), g[loc].view(np.uint32)), "values must be the raw entries"
    keys = key_of(g).astype(np.int64)
    kept = np.zeros(n, dtype=bool)
    kept[loc] = True
    if k == 0 or k == n:
        return
    ks, ku = keys[kept], keys[~kept]
    i_s, i_u = np.nonzero(kept)[0], np.nonzero(~kept)[0]
    # weakest kept entry: smallest key, and among those the highest index
    wk = ks.min()
    wi = i_s[ks == wk].max()
    # strongest dropped entry: largest key, and among those the lowest index
    sk = ku.max()
    si = i_u[ku == sk].min()
    assert wk > sk or (wk == sk and wi < si), "a dropped entry outranks a kept one"


def unique_valid_subset(g, k):
    """Brute force over all k-subsets of a tiny tensor."""
    keys = [int(x) for x in key_of(g)]
    n = len(keys)
    valid = []
    for sub in itertools.combinations(range(n), k):
        s = set(sub)
        ok = all((keys[a] > keys[b]) or (keys[a] == keys[b] and a < b)
                 for a in sub for b in range(n) if b not in s)
        if ok:
            valid.append(sub)
    assert len(valid) == 1
    return valid[0]


ALPHABET = [0.0, -0.0, 1.0, -1.0, 2.5, -2.5, float("inf"), 1e-45]


@pytest.mark.parametrize("full_sort", [True, False])
def test_exhaustive_tiny_alphabet(full_sort):
    # every tensor of length <= 4 over an alphabet full of ties, signed zeros, a denormal and Inf
    for n in range(1, 5):
        for combo in itertools.product(ALPHABET, repeat=n):
            g = np.array(combo, dtype=np.float32)
            for k in range(0, n + 1):
                idx, val = oracle.select(g, k, full_sort=full_sort)
                assert tuple(int(i) for i in idx) == unique_valid_subset(g, k)
                assert np.array_equal(val.view(np.uint32), g[idx.astype(np.int64)].view(np.uint32))


@pytest.mark.parametrize("full_sort", [True, False])
def test_subset_enumeration_random(full_sort):
    rng = np.random.default_rng(1)
    for _ in range(200):
        n = int(rng.integers(1, 11))
        g = rng.choice(np.array([0.5, -0.5, 1.0, 3.0, -3.0, 0.0, 7.0], dtype=np.float32), size=n)
        g = np.where(rng.random(n) < 0.4, rng.standard_normal(n).astype(np.float32), g).astype(np.float32)
        k = int(rng.integers(0, n + 1))
        idx, _ = oracle.select(g, k, full_sort=full_sort)
        assert tuple(int(i) for i in idx) == unique_valid_subset(g, k)


@pytest.mark.parametrize("full_sort", [True, False])
def test_pairwise_rule_medium(full_sort):
    rng = np.random.default_rng(2)
    for trial in range(60):
        n = int(rng.integers(1, 3000))
        if trial % 3 == 0:      # heavy ties: values on a coarse grid
            g = np.round(rng.standard_normal(n) * 4).astype(np.float32) / 4
        elif trial % 3 == 1:
            g = rng.standard_normal(n).astype(np.float32)
        else:                   # all equal magnitude, mixed sign
            g = (np.where(rng.random(n) < 0.5, -1, 1) * 0.25).astype(np.float32)
        for k in {0, 1, n // 100 + 1, n // 2, n - 1 if n > 1 else 1, n}:
            if k > n:
                continue
            idx, val = oracle.select(g, k, offset=1000, full_sort=full_sort)
            check_is_the_selection(g, k, idx, val, offset=1000)


def test_partial_sort_variant_equals_definition():
    rng = np.random.default_rng(3)
    for _ in range(10_000):
        n = int(rng.integers(1, 65))
        g = (rng.integers(-6, 7, size=n) * 0.5).astype(np.float32)
        k = int(rng.integers(0, n + 1))
        a = oracle.select(g, k, full_sort=True)
        b = oracle.select(g, k, full_sort=False)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1].view(np.uint32), b[1].view(np.uint32))


def test_keep_everything_is_identity():
    g = np.random.default_rng(4).standard_normal(777).astype(np.float32)
    idx, val = oracle.select(g, 777, offset=5)
    assert np.array_equal(idx, np.arange(5, 782, dtype=np.uint32))
    assert np.array_equal(val, g)


def test_keep_one_is_first_argmax():
    rng = np.random.default_rng(5)
    for _ in range(200):
        g = (rng.integers(-9, 10, size=50)).astype(np.float32)
        idx, val = oracle.select(g, 1)
        assert int(idx[0]) == int(np.argmax(np.abs(g)))      # numpy returns the first maximum
        assert val[0] == g[idx[0]]


def test_magnitudes_match_library_sort():
    rng = np.random.default_rng(6)
    g = rng.standard_normal(50_000).astype(np.float32)
    # the multiset of kept magnitudes is unique even when a few magnitudes collide
    k = 500
    idx, val = oracle.select(g, k)
    assert np.array_equal(np.sort(np.abs(val)), np.sort(np.abs(g))[-k:])


def test_signed_zero_and_inf():
    g = np.array([0.0, -0.0, np.inf, -np.inf, 1.0, -0.0], dtype=np.float32)
    idx, val = oracle.select(g, 2)
    assert list(idx) == [2, 3]
    idx, val = oracle.select(g, 4)
    assert list(idx) == [0, 2, 3, 4]            # the first zero wins among the zeros
    assert np.signbit(val[0]) == False
    idx, val = oracle.select(g, 5)
    assert list(idx) == [0, 1, 2, 3, 4] and np.signbit(val[1])   # -0 is emitted as -0


def test_k_larger_than_n_is_an_error():
    with pytest.raises(ValueError):
        oracle.select(np.zeros(3, dtype=np.float32), 4)


def test_layers_are_selected_independently():
    # a tensor of tiny values next to a tensor of huge values: per-tensor selection keeps
    # entries of both, selection "across the whole model" would keep none of the first
    rng = np.random.default_rng(7)
    a = (rng.standard_normal(100) * 1e-6).astype(np.float32)
    b = (rng.standard_normal(300) * 1e3).astype(np.float32)
    grad = np.concatenate([a, b])
    idx, val = oracle.select_layers(grad, [0, 100], [100, 300], [3, 9])
    assert idx.size == 12 and np.all(idx[:3] < 100) and np.all(idx[3:] >= 100)
    check_is_the_selection(a, 3, idx[:3], val[:3], 0)
    check_is_the_selection(b, 9, idx[3:], val[3:], 100)


# --------------------------------------------------------------------------- keep count

def test_keep_count_against_exact_rationals():
    rng = np.random.default_rng(8)
    for _ in range(2000):
        n = int(rng.integers(1, 2**31))
        den = int(rng.integers(1, 100_000))
        num = int(rng.integers(0, den + 1))
        want = min(n, max(1, math.ceil(Fraction(n * num, den))))
        assert oracle.keep_count(n, num, den) == want
    assert oracle.keep_count(0, 1, 100) == 0


def test_keep_count_of_the_workloads():
    # hand-computed: ceil(832/100)=9, ceil(51264/100)=513, ceil(3212288/100)=32123, ceil(10250/100)=103
    assert [oracle.keep_count(n, 1, 100) for n in (832, 51_264, 3_212_288, 10_250)] == [9, 513, 32_123, 103]
    assert [oracle.keep_count(4_000_000, 1, d) for d in (1000, 400, 160, 64, 25, 10)] == \
        [4_000, 10_000, 25_000, 62_500, 160_000, 400_000]
    # a 64-entry tensor at 0.5 % still sends one entry
    assert oracle.keep_count(64, 5, 1000) == 1
    assert oracle.keep_count(2_359_296, 5, 1000) == 11_797     # 11796.48 rounded up


def test_nan_orders_above_inf_by_bit_pattern():
    """The reading for NaN inputs: the key is the bit pattern without the sign, so every NaN
    outranks +-Inf and NaNs rank among themselves by payload; values keep their bits (signalling
    NaNs are not quieted).  Checked with the pairwise form of the rule and by subset enumeration."""
    pats = np.array([0x7FC00000, 0xFFC00000, 0x7FA00001, 0xFF800001, 0x7FC12345, 0x7FFFFFFF], dtype=np.uint32)
    tiny = np.array([1.0, np.inf, 0.0, -np.inf, 2.0, -3.0, 0.5], dtype=np.float32)
    tiny = np.concatenate([tiny, pats[:3].view(np.float32)])
    rng = np.random.default_rng(9)
    tiny = tiny[rng.permutation(tiny.size)]
    for k in range(1, tiny.size + 1):
        idx, val = oracle.select(tiny, k)
        assert tuple(int(i) for i in idx) == unique_valid_subset(tiny, k)
        assert np.array_equal(val.view(np.uint32), tiny.view(np.uint32)[idx])
        idx2, _ = oracle.select(tiny, k, full_sort=True)
        assert np.array_equal(idx, idx2)
    # with 3 NaNs and 2 infinities, k = 3 keeps exactly the NaNs and k = 5 adds both infinities
    nan_at = set(np.flatnonzero(np.isnan(tiny)).tolist())
    assert set(oracle.select(tiny, 3)[0].tolist()) == nan_at
    assert set(oracle.select(tiny, 5)[0].tolist()) == nan_at | set(np.flatnonzero(np.isinf(tiny)).tolist())
    g = rng.standard_normal(5000).astype(np.float32)
    g.view(np.uint32)[rng.choice(5000, pats.size, replace=False)] = pats
    for k in (1, 3, 6, 7, 50):
        idx, val = oracle.select(g, k)
        check_is_the_selection(g, k, idx, val)
