"""Parity of the index coding (CUDA, through the C ABI) with the CPU oracle: the streams and the
block offsets word for word, and the round trip."""
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
