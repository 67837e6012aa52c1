"""Parity of the index coding and of the value packing (CUDA, through the C ABI) with the CPU oracle: the
streams and the block offsets word for word, and the round trip."""
import numpy as np
import pytest
import torch

import oracle
from paper_1702_04683_b200 import workloads as wlmod

from helpers import oracle_keep_counts, u32

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda", 0)


@pytest.fixture(scope="module")
def binding():
    from paper_1702_04683_b200 import binding as b
    return b


def check(binding, idx_rows):
    """idx_rows: [W, K] uint32 numpy.  Encodes on the GPU, compares with the oracle, decodes again."""
    idx = torch.from_numpy(np.ascontiguousarray(idx_rows, dtype=np.uint32).view(np.int32)).to(DEV)
    W, K = idx.shape
    words, off = binding.adacomp_encode_indices(idx)
    torch.cuda.synchronize()
    h_words, h_off = words.cpu().numpy().view(np.uint32), off.cpu().numpy().astype(np.uint64)
    total = 0
    for w in range(W):
        ow, oo = oracle.encode_indices(idx_rows[w])
        assert np.array_equal(h_off[w], oo), f"worker {w}: block offsets differ"
        assert np.array_equal(h_words[w, :ow.size], ow), f"worker {w}: stream differs"
        total += ow.size
    back = binding.adacomp_decode_indices(words, off, K)
    assert np.array_equal(u32(back), np.ascontiguousarray(idx_rows, dtype=np.uint32))
    return 4.0 * total / max(1, W * K)


@pytest.mark.parametrize("K", [0, 1, 2, 255, 256, 257, 512, 70_001])
def test_sizes_around_the_block_boundaries(binding, K):
    rng = np.random.default_rng(K)
    rows = np.stack([np.sort(rng.choice(max(K, 1) * 37 + 5, K, replace=False)).astype(np.uint32) for _ in range(3)])
    check(binding, rows)


def test_extreme_gaps_and_lists_that_are_not_ascending(binding):
    rows = np.array([[0, 2**32 - 2, 2**32 - 1, 5], [9, 3, 3, 0], [0, 1, 2, 3], [2**31, 2**31 + 1, 7, 2**32 - 1]], dtype=np.uint32)
    check(binding, rows)
    long_row = np.concatenate([np.arange(300, dtype=np.uint32) * np.uint32(14_000_000), [5, 5, 2**32 - 1]]).astype(np.uint32)
    check(binding, long_row[None])
    with pytest.raises(binding.AdacompError) as e:            # stream capacity too small
        idx = torch.zeros((1, 1000), dtype=torch.int32, device=DEV)
        small = torch.empty((1, 1000), dtype=torch.int32, device=DEV)
        off = torch.empty((1, 5), dtype=torch.int64, device=DEV)
        binding._check(binding.raw().adacomp_encode_indices(idx.data_ptr(), 1000, 1, small.data_ptr(), 1000, off.data_ptr(), 0, 0), "enc")
    assert e.value.status == binding.ERR_CAPACITY


@pytest.mark.parametrize("keep", [(1, 1000), (1, 100), (1, 10)])
def test_selected_updates_of_a_workload(binding, keep):
    """What adacomp_select emits, coded: bytes per index against the 4 of the plain list."""
    wl = wlmod.workload(2)                                      # tie_stress: 3.27 M parameters
    g = wlmod.round_gradients(wl, 0, DEV, workers=range(5))
    sel = binding.Selector(binding.make_segments(wl.tensor_sizes, keep), 5, DEV)
    idx, _ = sel.select(g)
    per_index = check(binding, u32(idx))
    assert per_index < {1000: 2.0, 100: 1.6, 10: 1.1}[keep[1]]


def test_full_size_update_round_trip_and_sampled_blocks(binding):
    """10^7 indices per worker (the largest update of the benchmark): round trip on the GPU, the oracle
    on sampled blocks."""
    wl = wlmod.workload(4)
    ks = oracle_keep_counts(wl.tensor_sizes, (1, 10))
    idx, _ = wlmod.synthetic_updates(wl, ks, 0, DEV)
    idx = idx[:4].contiguous()
    K = idx.shape[1]
    words, off = binding.adacomp_encode_indices(idx)
    back = binding.adacomp_decode_indices(words, off, K)
    assert torch.equal(back, idx)
    h_off = off.cpu().numpy()
    rng = np.random.default_rng(2)
    for _ in range(40):
        w, b = int(rng.integers(4)), int(rng.integers((K + 255) // 256))
        blk = u32(idx[w, 256 * b:256 * b + 256])
        ow, _ = oracle.encode_indices(blk)
        lo = int(h_off[w, b])
        assert int(h_off[w, b + 1]) - lo == ow.size
        assert np.array_equal(u32(words[w, lo:lo + ow.size]), ow)
    assert 4.0 * float(h_off[:, -1].sum()) / (4 * K) < 1.0      # under a byte per index at keep 1/10


def test_corrupt_streams_are_not_followed(binding):
    """A decoder at the server's ingress cannot trust what arrives: block offsets that point outside
    the stream, a width above 32 bits, or a payload that would run past the end must not be read;
    the block decodes to 0xFFFFFFFF (an index every server refuses) and the other blocks are intact."""
    rng = np.random.default_rng(5)
    K = 1000                                                    # four blocks
    rows = np.stack([np.sort(rng.choice(10**6, K, replace=False)).astype(np.uint32) for _ in range(2)])
    idx = torch.from_numpy(rows.view(np.int32)).to(DEV)
    words, off = binding.adacomp_encode_indices(idx)
    cap = words.shape[1]
    bad_off = off.clone()
    bad_off[0, 1] = 10**12                                      # block 1 of worker 0: far outside the stream
    bad_off[1, 3] = cap - 1                                     # block 3 of worker 1: header would straddle the end
    bad_words = words.clone()
    bad_words[0, int(off[0, 2]) + 1] = 77                       # block 2 of worker 0: a width of 77 bits
    back = u32(binding.adacomp_decode_indices(bad_words, bad_off, K))
    want = rows.copy()
    want[0, 256:512] = want[0, 512:768] = 0xFFFFFFFF
    want[1, 768:] = 0xFFFFFFFF
    assert np.array_equal(back, want)


# ----------------------------------------------------------------------------- value packing

def check_values(binding, val_rows):
    """val_rows: [W, K] float32 numpy (any bit patterns).  Packs on the GPU, compares the stream and the block
    offsets with the oracle word for word, unpacks again: every bit pattern must come back."""
    rows = np.ascontiguousarray(val_rows, dtype=np.float32)
    val = torch.from_numpy(rows.view(np.int32)).to(DEV).view(torch.float32)
    W, K = val.shape
    words, off = binding.adacomp_encode_values(val)
    torch.cuda.synchronize()
    h_words, h_off = words.cpu().numpy().view(np.uint32), off.cpu().numpy().astype(np.uint64)
    total = 0
    for w in range(W):
        ow, oo = oracle.encode_values(rows[w])
        assert np.array_equal(h_off[w], oo), f"worker {w}: block offsets differ"
        assert np.array_equal(h_words[w, :ow.size], ow), f"worker {w}: stream differs"
        total += ow.size
    back = binding.adacomp_decode_values(words, off, K)
    assert np.array_equal(back.view(torch.int32).cpu().numpy().view(np.uint32), rows.view(np.uint32))
    return 4.0 * total / max(1, W * K)


@pytest.mark.parametrize("K", [0, 1, 2, 255, 256, 257, 512, 70_001])
@pytest.mark.parametrize("spread", [0.0, 2.0, 40.0])
def test_values_around_the_block_boundaries(binding, K, spread):
    rng = np.random.default_rng(K + int(spread))
    rows = (rng.standard_normal((3, K)) * np.exp2(rng.uniform(-spread, spread, (3, K)))).astype(np.float32)
    check_values(binding, rows)


def test_every_kind_of_bit_pattern_is_packed_and_comes_back(binding):
    pats = np.array([0x00000000, 0x80000000, 0x00000001, 0x807FFFFF, 0x00800000, 0x7F7FFFFF, 0xFF7FFFFF, 0x7F800000,
                     0xFF800000, 0x7FC00000, 0xFFC12345, 0x7F800001, 0x3F800000, 0xBF800000], dtype=np.uint32)
    assert check_values(binding, pats.view(np.float32)[None]) > 4.0          # all 8 exponent bits: 32 bits an entry + the header
    rng = np.random.default_rng(9)
    anything = rng.integers(0, 2**32, (2, 5000), dtype=np.uint64).astype(np.uint32)
    check_values(binding, anything.view(np.float32))
    same = np.full((1, 600), -0.375, np.float32)                              # one exponent: 24 bits an entry
    assert check_values(binding, same) < 3.03
    with pytest.raises(binding.AdacompError) as e:                            # stream capacity too small
        v = torch.zeros((1, 1000), device=DEV)
        small = torch.empty((1, 1000), dtype=torch.int32, device=DEV)
        off = torch.empty((1, 5), dtype=torch.int64, device=DEV)
        binding._check(binding.raw().adacomp_encode_values(v.data_ptr(), 1000, 1, small.data_ptr(), 1000, off.data_ptr(), 0, 0), "enc")
    assert e.value.status == binding.ERR_CAPACITY


@pytest.mark.parametrize("keep", [(1, 1000), (1, 100), (1, 10)])
def test_selected_values_of_a_workload(binding, keep):
    """What adacomp_select emits, packed: bytes per value against the 4 of the plain list, on Gaussian gradients
    (the large flat workload, scaled down) and on the heavy-tailed tie-stress workload."""
    wl = wlmod.workload(4).scaled(16, n_workers=3)
    sel = binding.Selector(binding.make_segments(wl.tensor_sizes, keep), 3, DEV)
    _, val = sel.select(wlmod.round_gradients(wl, 0, DEV))
    assert check_values(binding, val.cpu().numpy()) < 3.4
    wl = wlmod.workload(2)
    sel = binding.Selector(binding.make_segments(wl.tensor_sizes, keep), 5, DEV)
    _, val = sel.select(wlmod.round_gradients(wl, 0, DEV, workers=range(5)))
    assert check_values(binding, val.cpu().numpy()) < 4.0


def test_corrupt_value_streams_are_not_followed(binding):
    """Block offsets that point outside the stream, a header no encoder writes, or a payload that would run past the
    end must not be read: the block unpacks to +0.0 (a value that changes no parameter), the other blocks are intact."""
    rng = np.random.default_rng(6)
    K = 1000                                                    # four blocks
    rows = rng.standard_normal((2, K)).astype(np.float32)
    val = torch.from_numpy(rows).to(DEV)
    words, off = binding.adacomp_encode_values(val)
    cap = words.shape[1]
    bad_off = off.clone()
    bad_off[0, 1] = 10**12                                      # block 1 of worker 0: far outside the stream
    bad_off[1, 3] = cap - 3                                     # block 3 of worker 1: its payload would run past the end
    bad_words = words.clone()
    bad_words[0, int(off[0, 2])] = 9 << 8                       # block 2 of worker 0: an exponent width of 9 bits
    back = binding.adacomp_decode_values(bad_words, bad_off, K).cpu().numpy()
    want = rows.copy()
    want[0, 256:768] = 0.0
    want[1, 768:] = 0.0
    assert np.array_equal(back.view(np.uint32), want.view(np.uint32))


def test_full_size_values_round_trip_and_sampled_blocks(binding):
    """10^7 values per worker (the largest update of the benchmark, as the selector emits it for 4 workers): round
    trip on the GPU bit for bit, the oracle on sampled blocks."""
    wl = wlmod.workload(4)
    import dataclasses
    wl4 = dataclasses.replace(wl, n_workers=4)
    sel = binding.Selector(binding.make_segments(wl.tensor_sizes, (1, 10)), 4, DEV)
    _, val = sel.select(wlmod.round_gradients(wl4, 0, DEV))
    K = val.shape[1]
    words, off = binding.adacomp_encode_values(val)
    back = binding.adacomp_decode_values(words, off, K)
    assert torch.equal(back.view(torch.int32), val.view(torch.int32))
    h_off = off.cpu().numpy()
    rng = np.random.default_rng(4)
    for _ in range(40):
        w, b = int(rng.integers(4)), int(rng.integers((K + 255) // 256))
        blk = val[w, 256 * b:256 * b + 256].cpu().numpy()
        ow, _ = oracle.encode_values(blk)
        lo = int(h_off[w, b])
        assert int(h_off[w, b + 1]) - lo == ow.size
        assert np.array_equal(u32(words[w, lo:lo + ow.size]), ow)
    assert 4.0 * float(h_off[:, -1].sum()) / (4 * K) < 3.3      # 26 to 27 bits a value
