"""The sharded server's glue on a GPU: one rank (a process group of size 1, so the exchange is a local
copy) drives ShardedServer with the CUDA library as the local server; staleness counts and parameters
against the oracle.  The routing between ranks is covered on CPU ranks in test_sharding_gloo.py."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist

import oracle
from paper_1702_04683_b200 import sharding, workloads as wlmod

from helpers import bits, oracle_keep_counts, u32

pytestmark = pytest.mark.gpu


def test_one_rank_sharded_server_on_the_gpu():
    dev = torch.device("cuda", 0)
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=0, world_size=1)
    try:
        wl = wlmod.workload(1).scaled(16, n_workers=12, n_rounds=3)
        ks = oracle_keep_counts(wl.tensor_sizes, (1, 50))
        K = int(sum(ks))
        theta = wlmod.initial_parameters(wl, dev)
        ref = oracle.Server(theta.cpu().numpy())
        srv = sharding.ShardedServer(theta, wl.n_params, wl.n_workers, history_pairs=4 * wl.n_workers * K,
                                     max_window_updates=2 * wl.n_workers)
        assert (srv.lo, srv.hi) == (0, wl.n_params)
        for r, rd in enumerate(wlmod.arrival_schedule(wl)):
            idx, val = wlmod.synthetic_updates(wl, ks, r, dev, zero_fraction=0.02)
            sigma, begin, count = srv.step(idx, val, rd.order, rd.pull_ts, wl.lr, want_sigma=True)
            h_idx, h_val, h_sig = u32(idx), val.cpu().numpy(), u32(sigma)
            for b, w in enumerate(rd.order.tolist()):
                want = ref.apply(h_idx[w], h_val[w], int(rd.pull_ts[b]), wl.lr)
                assert int(count[w]) == K
                assert np.array_equal(h_sig[int(begin[w]):int(begin[w]) + K], want), (r, b)
        assert srv.applier.last_error() == 0 and srv.timestamp == ref.timestamp
        assert np.array_equal(bits(theta), bits(ref.theta()))
    finally:
        dist.destroy_process_group()
