"""Pins for the oracle's statement of the index coding (blocks of 256 entries: first index, gap
width, bit-packed gaps).  Expectations come from a stream worked out by hand, from Python's
arbitrary-precision integers used as bit strings, and from the round trip."""
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
