"""The multi-GPU plan on CPU: two gloo ranks each own half of the parameters; routing every
update's slices to their owners and applying them there gives the same staleness counters and
the same parameters as one server that sees everything."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_1702_04683_b200 import sharding, workloads as wlmod


def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def scenario():
    wl = wlmod.workload(1).scaled(256, n_workers=6, n_rounds=3)          # 12.8 k parameters, 6 workers, 3 rounds
    ks = [oracle.keep_count(n, 1, 20) for n in wl.tensor_sizes]
    return wl, ks


def worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl, ks = scenario()
        K = sum(ks)
        ranges = sharding.parameter_ranges(wl.n_params, world)
        lo, hi = ranges[rank]
        theta0 = wlmod.initial_parameters(wl, "cpu").numpy()
        shard = oracle.Server(theta0[lo:hi])
        per_rank = wl.n_workers // world                                   # workers rank r hosts: r*per_rank ...
        sig_log = []
        for r, rd in enumerate(wlmod.arrival_schedule(wl)):
            idx_all, val_all = wlmod.synthetic_updates(wl, ks, r, "cpu", zero_fraction=0.05)
            mine = slice(rank * per_rank, (rank + 1) * per_rank)
            got = sharding.exchange_updates(idx_all[mine].to(torch.int64), val_all[mine], ranges)
            # slices of worker w (global id) for my range
            per_worker = {}
            for src, (li, v, counts) in enumerate(got):
                off = 0
                for wloc, c in enumerate(counts.tolist()):
                    per_worker[src * per_rank + wloc] = (li[off:off + c].numpy().astype(np.uint32), v[off:off + c].numpy())
                    off += c
            for b, w in enumerate(rd.order.tolist()):                      # global arrival order
                li, v = per_worker[w]
                sig_log.append((r, w, shard.apply(li, v, int(rd.pull_ts[b]), wl.lr)))
        q.put((rank, lo, hi, shard.theta(), shard.timestamp, sig_log))
    finally:
        dist.destroy_process_group()


def test_two_rank_parameter_sharding_matches_one_server():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = free_port()
    procs = [ctx.Process(target=worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # one server that sees everything
    wl, ks = scenario()
    theta0 = wlmod.initial_parameters(wl, "cpu").numpy()
    ref = oracle.Server(theta0)
    ref_sig = {}
    for r, rd in enumerate(wlmod.arrival_schedule(wl)):
        idx_all, val_all = wlmod.synthetic_updates(wl, ks, r, "cpu", zero_fraction=0.05)
        for b, w in enumerate(rd.order.tolist()):
            i32 = idx_all[w].numpy().view(np.uint32)
            ref_sig[(r, w)] = (i32, ref.apply(i32, val_all[w].numpy(), int(rd.pull_ts[b]), wl.lr))
    want = ref.theta()
    assert results[0][1] == 0 and results[-1][2] == wl.n_params and results[0][2] == results[1][1]
    for rank, lo, hi, theta, ts, sig_log in results:
        assert ts == ref.timestamp                                   # every shard ticks once per update
        assert np.array_equal(theta.view(np.uint32), want[lo:hi].view(np.uint32))
        for r, w, sig in sig_log:
            i32, full = ref_sig[(r, w)]
            sel = (i32 >= lo) & (i32 < hi)
            assert np.array_equal(sig, full[sel])


class OracleApplier:
    """The oracle behind the interface of the library's server: lets ShardedServer run on CPU ranks."""

    def __init__(self, theta):
        self.srv = oracle.Server(theta)

    @property
    def timestamp(self):
        return self.srv.timestamp

    def apply(self, idx, val, begin, count, pull_ts, lr, sigma_out=None):
        i, v = idx.numpy().view(np.uint32), val.numpy()
        for b in range(len(begin)):
            lo, n = int(begin[b]), int(count[b])
            sig = self.srv.apply(i[lo:lo + n], v[lo:lo + n], int(pull_ts[b]), lr)
            if sigma_out is not None:
                sigma_out.numpy().view(np.uint32)[lo:lo + n] = sig


def sharded_worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl, ks = scenario()
        per_rank = wl.n_workers // world
        ranges = sharding.parameter_ranges(wl.n_params, world)
        lo, hi = ranges[rank]
        theta0 = wlmod.initial_parameters(wl, "cpu")
        shard = theta0[lo:hi].clone()
        srv = sharding.ShardedServer(shard, wl.n_params, per_rank, history_pairs=1 << 16, max_window_updates=64,
                                     applier=OracleApplier(shard.numpy()))
        log = []
        for r, rd in enumerate(wlmod.arrival_schedule(wl)):
            idx_all, val_all = wlmod.synthetic_updates(wl, ks, r, "cpu", zero_fraction=0.05)    # int32 holding uint32 bits
            mine = slice(rank * per_rank, (rank + 1) * per_rank)
            sigma, begin, count = srv.step(idx_all[mine], val_all[mine], rd.order, rd.pull_ts, wl.lr, want_sigma=True)
            for w in range(wl.n_workers):
                log.append((r, w, sigma.numpy().view(np.uint32)[int(begin[w]):int(begin[w]) + int(count[w])].copy()))
        q.put((rank, lo, hi, srv.applier.srv.theta(), srv.timestamp, log))
    finally:
        dist.destroy_process_group()


def test_sharded_server_class_matches_one_server():
    """The class a multi-GPU job uses (exchange, then the local apply in global arrival order), driven on
    two CPU ranks with the oracle as the local applier: staleness counts and parameters of the shards
    are those of one server that sees everything."""
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = free_port()
    procs = [ctx.Process(target=sharded_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    wl, ks = scenario()
    ref = oracle.Server(wlmod.initial_parameters(wl, "cpu").numpy())
    ref_sig = {}
    for r, rd in enumerate(wlmod.arrival_schedule(wl)):
        idx_all, val_all = wlmod.synthetic_updates(wl, ks, r, "cpu", zero_fraction=0.05)
        for b, w in enumerate(rd.order.tolist()):
            i32 = idx_all[w].numpy().view(np.uint32)
            ref_sig[(r, w)] = (i32, ref.apply(i32, val_all[w].numpy(), int(rd.pull_ts[b]), wl.lr))
    want = ref.theta()
    for rank, lo, hi, theta, ts, log in results:
        assert ts == ref.timestamp
        assert np.array_equal(theta.view(np.uint32), want[lo:hi].view(np.uint32))
        for r, w, sig in log:
            i32, full = ref_sig[(r, w)]
            assert np.array_equal(sig, full[(i32 >= lo) & (i32 < hi)])


def test_ranges_and_slice_points():
    ranges = sharding.parameter_ranges(10_000, 4)
    assert ranges[0][0] == 0 and ranges[-1][1] == 10_000
    assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
    assert all(lo % sharding.RANGE_ALIGN == 0 for lo, _ in ranges)
    idx = torch.tensor([0, 5, 2047, 2048, 9_999], dtype=torch.int64)
    cuts = sharding.slice_points(idx, ranges)
    assert cuts[0] == 0 and cuts[-1] == 5
    for r, (lo, hi) in enumerate(ranges):
        part = idx[cuts[r]:cuts[r + 1]]
        assert bool(((part >= lo) & (part < hi)).all())
