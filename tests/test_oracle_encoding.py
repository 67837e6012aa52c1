"""Pins for the oracle's statement of the index coding (blocks of 256 entries: first index, gap
width, bit-packed gaps) and of the lossless value packing (blocks of 256 entries: smallest exponent,
exponent width, bit-packed sign / relative exponent / mantissa).  Expectations come from streams
worked out by hand, from Python's arbitrary-precision integers used as bit strings, and from the
round trip."""
import tempfile

import numpy as np
import pytest

import oracle
from test_oracle_mutations import SRC, build_variant, p

import ctypes


def bigint_encode(idx):
    """The format again, with one Python integer per block as the bit string."""
    idx = [int(i) for i in idx]
    words, off = [], []
    for first in range(0, len(idx), 256):
        blk = idx[first:first + 256]
        off.append(len(words))
        gaps = [(b - a - 1) % 2**32 for a, b in zip(blk, blk[1:])]
        w = max((g.bit_length() for g in gaps), default=0)
        bitstring = sum(g << (e * w) for e, g in enumerate(gaps))
        n_words = (len(gaps) * w + 31) // 32
        words += [blk[0], w] + [(bitstring >> (32 * i)) & 0xFFFFFFFF for i in range(n_words)]
    off.append(len(words))
    return np.array(words, dtype=np.uint32), np.array(off, dtype=np.uint64)


def test_stream_worked_out_by_hand():
    # gaps of [5, 6, 9, 300]: 0, 2, 290 -> 9 bits each; 0 | 2 << 9 | 290 << 18 = 1024 + 76 021 760
    words, off = oracle.encode_indices([5, 6, 9, 300])
    assert words.tolist() == [5, 9, 76_022_784] and off.tolist() == [0, 3]
    # consecutive indices have gap 0: no payload at all
    words, off = oracle.encode_indices(list(range(40, 300)))               # 260 entries: two blocks
    assert words.tolist() == [40, 0, 296, 0] and off.tolist() == [0, 2, 4]
    # a 5-bit gap straddles the first word boundary: entries 1 .. 7 of gap 21 = 0b10101
    words, _ = oracle.encode_indices([22 * e for e in range(8)])
    assert words.tolist()[:2] == [0, 5]
    assert words[2] == sum(21 << (5 * e) for e in range(7)) & 0xFFFFFFFF and words[3] == (sum(21 << (5 * e) for e in range(7)) >> 32)
    assert oracle.encode_indices([])[0].size == 0 and oracle.encode_indices([7])[0].tolist() == [7, 0]


@pytest.mark.parametrize("n", [0, 1, 2, 255, 256, 257, 513, 5000])
@pytest.mark.parametrize("density", [0.5, 0.01, 0.0001])
def test_matches_the_bit_string_form_and_round_trips(n, density):
    rng = np.random.default_rng(n * 7 + int(density * 1e4))
    span = max(n, int(n / density)) + 1
    idx = np.sort(rng.choice(span, n, replace=False)).astype(np.uint32)
    words, off = oracle.encode_indices(idx)
    want_words, want_off = bigint_encode(idx)
    assert np.array_equal(words, want_words) and np.array_equal(off, want_off)
    assert np.array_equal(oracle.decode_indices(words, off, n), idx)
    # size: two header words per block, then the packed gaps
    sizes = np.diff(off.astype(np.int64))
    for b, size in enumerate(sizes.tolist()):
        n_b = min(256, n - 256 * b)
        assert size == 2 + ((n_b - 1) * int(words[int(off[b]) + 1]) + 31) // 32


def test_extreme_gaps_and_lists_that_are_not_ascending():
    for idx in ([0, 2**32 - 2], [2**32 - 2], [0, 1, 2**31, 2**31 + 1], [9, 3, 3, 2**32 - 2, 0]):
        idx = np.array(idx, dtype=np.uint32)
        words, off = oracle.encode_indices(idx)
        assert np.array_equal(words, bigint_encode(idx)[0])
        assert np.array_equal(oracle.decode_indices(words, off, idx.size), idx)      # gaps are taken modulo 2^32
    assert oracle.encode_indices([0, 2**32 - 2])[0].tolist() == [0, 32, 2**32 - 3]
    with pytest.raises(ValueError):
        oracle.decode_indices(np.array([0, 33, 0], np.uint32), np.array([0, 3], np.uint64), 2)


def test_bytes_per_index_at_the_paper_densities():
    rng = np.random.default_rng(1)
    for inv_c, most in ((10, 1.1), (100, 1.6), (1000, 2.0)):          # gaps of about 1 / c: ~log2(8 / c) bits with the tail
        idx = np.sort(rng.choice(10**6, 10**6 // inv_c, replace=False)).astype(np.uint32)
        words, _ = oracle.encode_indices(idx)
        assert np.log2(inv_c) / 8 < 4.0 * words.size / idx.size < most


CODING_MUTATIONS = {
    "gap keeps the 1": ("const uint64_t gap = idx[first + e] - idx[first + e - 1] - 1u;", "const uint64_t gap = idx[first + e] - idx[first + e - 1];"),
    "bits most significant first": ("if ((gap >> bit) & 1u) words_out[at + pos / 32] |= 1u << (pos % 32);",
                                    "if ((gap >> bit) & 1u) words_out[at + pos / 32] |= 0x80000000u >> (pos % 32);"),
    "width one short": ("words_out[at++] = widest;", "words_out[at++] = widest ? widest - 1 : 0;"),
    "entry 1 skipped": ("const uint64_t pos = (e - 1) * widest + bit;\n                if ((gap >> bit) & 1u) words_out",
                        "const uint64_t pos = e * widest + bit;\n                if ((gap >> bit) & 1u) words_out"),
}


def coding_pins_hold(L) -> bool:
    u32p, u64p = ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(ctypes.c_uint64)
    L.oracle_encode_indices.restype = ctypes.c_uint64
    L.oracle_encode_indices.argtypes = [u32p, ctypes.c_uint64, u32p, u64p]
    for idx, want in (([5, 6, 9, 300], [5, 9, 76_022_784]), ([22 * e for e in range(8)], None)):
        idx = np.array(idx, np.uint32)
        words = np.zeros(idx.size + 8, np.uint32)
        off = np.zeros(2, np.uint64)
        total = L.oracle_encode_indices(p(idx, ctypes.c_uint32), idx.size, p(words, ctypes.c_uint32), p(off, ctypes.c_uint64))
        ref = want if want is not None else bigint_encode(idx)[0].tolist()
        if words[:int(total)].tolist() != ref:
            return False
    return True


def test_untouched_oracle_passes_the_compact_coding_pins():
    assert coding_pins_hold(build_variant(open(SRC).read(), tempfile.mkdtemp(), "same"))


@pytest.mark.parametrize("name", sorted(CODING_MUTATIONS))
def test_planted_mistake_in_the_coding_is_caught(name):
    old, new = CODING_MUTATIONS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, "the mutation no longer matches the source"
    assert not coding_pins_hold(build_variant(text.replace(old, new), tempfile.mkdtemp(), "mutant"))


# ----------------------------------------------------------------------------- value packing

def bigint_encode_values(val):
    """The value format again, with one Python integer per block as the bit string."""
    bits = [int(b) for b in np.asarray(val, dtype=np.float32).view(np.uint32)]
    words, off = [], []
    for first in range(0, len(bits), 256):
        blk = bits[first:first + 256]
        off.append(len(words))
        exps = [(b >> 23) & 0xFF for b in blk]
        e_min, w_e = min(exps), (max(exps) - min(exps)).bit_length()
        width = 24 + w_e
        entries = [(b & 0x7FFFFF) | ((e - e_min) << 23) | ((b >> 31) << (23 + w_e)) for b, e in zip(blk, exps)]
        bitstring = sum(x << (t * width) for t, x in enumerate(entries))
        n_words = (len(blk) * width + 31) // 32
        words += [e_min | (w_e << 8)] + [(bitstring >> (32 * i)) & 0xFFFFFFFF for i in range(n_words)]
    off.append(len(words))
    return np.array(words, dtype=np.uint32), np.array(off, dtype=np.uint64)


def test_value_stream_worked_out_by_hand():
    # 1.0 = exponent 127, -2.0 = sign, exponent 128, 1.5 = exponent 127 and the top mantissa bit: e_min 127, one
    # exponent bit, 25 bits an entry.  Entries 0, 2^23 + 2^24, 2^22 at bits 0, 25, 50: bits 48, 49 and 72 are set.
    words, off = oracle.encode_values(np.array([1.0, -2.0, 1.5], np.float32))
    assert words.tolist() == [127 | 1 << 8, 0, (1 << 16) | (1 << 17), 1 << 8] and off.tolist() == [0, 4]
    # equal exponents: 24 bits an entry (sign + mantissa); 0.75 = exponent 126, mantissa 2^22
    words, off = oracle.encode_values(np.array([0.75, -0.75], np.float32))
    # entries 2^22 and 2^22 + 2^23 (the sign) at bits 0 and 24: bits 22, 46 and 47 are set
    assert words.tolist() == [126, 1 << 22, (1 << 14) | (1 << 15)] and off.tolist() == [0, 3]
    assert oracle.encode_values(np.array([], np.float32))[0].size == 0


@pytest.mark.parametrize("n", [0, 1, 2, 255, 256, 257, 513, 5000])
@pytest.mark.parametrize("spread", [0.0, 1.0, 30.0])
def test_values_match_the_bit_string_form_and_round_trip(n, spread):
    rng = np.random.default_rng(n * 11 + int(spread))
    val = (rng.standard_normal(n) * np.exp2(rng.uniform(-spread, spread, n))).astype(np.float32)
    words, off = oracle.encode_values(val)
    want_words, want_off = bigint_encode_values(val)
    assert np.array_equal(words, want_words) and np.array_equal(off, want_off)
    assert np.array_equal(oracle.decode_values(words, off, n).view(np.uint32), val.view(np.uint32))
    for b, size in enumerate(np.diff(off.astype(np.int64)).tolist()):
        n_b = min(256, n - 256 * b)
        assert size == 1 + (n_b * (24 + (int(words[int(off[b])]) >> 8)) + 31) // 32


def test_every_kind_of_bit_pattern_comes_back():
    # zeros of both signs, denormals, the extremes, infinities, NaNs with payloads: all 8 exponent bits are needed
    pats = np.array([0x00000000, 0x80000000, 0x00000001, 0x807FFFFF, 0x00800000, 0x7F7FFFFF, 0xFF7FFFFF, 0x7F800000,
                     0xFF800000, 0x7FC00000, 0xFFC12345, 0x7F800001, 0x3F800000, 0xBF800000], dtype=np.uint32)
    words, off = oracle.encode_values(pats.view(np.float32))
    assert int(words[0]) == (0 | 8 << 8) and words.size == 1 + pats.size          # 32 bits an entry
    assert np.array_equal(oracle.decode_values(words, off, pats.size).view(np.uint32), pats)
    assert np.array_equal(words, bigint_encode_values(pats.view(np.float32))[0])
    rng = np.random.default_rng(3)
    anything = rng.integers(0, 2**32, 3000, dtype=np.uint64).astype(np.uint32)
    words, off = oracle.encode_values(anything.view(np.float32))
    assert np.array_equal(oracle.decode_values(words, off, anything.size).view(np.uint32), anything)
    with pytest.raises(ValueError):                                               # an exponent width no block can have
        oracle.decode_values(np.array([9 << 8, 0, 0], np.uint32), np.array([0, 3], np.uint64), 1)


def test_bytes_per_value_of_the_largest_entries_of_gaussian_data():
    rng = np.random.default_rng(2)
    g = rng.standard_normal(10**6).astype(np.float32) * 1e-3
    for inv_c, most in ((10, 3.4), (100, 3.3), (1000, 3.3)):          # the kept values span two to three binades
        kept = g[np.sort(np.argsort(-np.abs(g))[:10**6 // inv_c])]
        words, _ = oracle.encode_values(kept)
        assert 3.0 < 4.0 * words.size / kept.size < most


VALUE_MUTATIONS = {
    "exponent not relative": ("e_rel = ((bits >> 23) & 0xFFu) - e_min, sign", "e_rel = ((bits >> 23) & 0xFFu), sign"),
    "sign below the exponent": ("const uint64_t entry = mantissa | (e_rel << 23) | (sign << (23 + w_e));",
                                "const uint64_t entry = mantissa | (sign << 23) | (e_rel << 24);"),
    "width one short": ("const uint32_t w_e = bits_needed(e_max - e_min), width = 24 + w_e;",
                        "const uint32_t w_e = bits_needed(e_max - e_min), width = 23 + w_e;"),
    "header fields swapped": ("words_out[at++] = e_min | (w_e << 8);", "words_out[at++] = w_e | (e_min << 8);"),
}


def value_pins_hold(L) -> bool:
    u32p, u64p, f32p = ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_float)
    L.oracle_encode_values.restype = ctypes.c_uint64
    L.oracle_encode_values.argtypes = [f32p, ctypes.c_uint64, u32p, u64p]
    for val, want in (([1.0, -2.0, 1.5], [127 | 1 << 8, 0, (1 << 16) | (1 << 17), 1 << 8]), ([0.1 * (t - 3.5) for t in range(9)], None)):
        val = np.array(val, np.float32)
        words = np.zeros(val.size + 8, np.uint32)
        off = np.zeros(2, np.uint64)
        total = L.oracle_encode_values(p(val, ctypes.c_float), val.size, p(words, ctypes.c_uint32), p(off, ctypes.c_uint64))
        ref = want if want is not None else bigint_encode_values(val)[0].tolist()
        if words[:int(total)].tolist() != ref:
            return False
    return True


def test_untouched_oracle_passes_the_value_packing_pins():
    assert value_pins_hold(build_variant(open(SRC).read(), tempfile.mkdtemp(), "same"))


@pytest.mark.parametrize("name", sorted(VALUE_MUTATIONS))
def test_planted_mistake_in_the_value_packing_is_caught(name):
    old, new = VALUE_MUTATIONS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, "the mutation no longer matches the source"
    assert not value_pins_hold(build_variant(text.replace(old, new), tempfile.mkdtemp(), "mutant"))
