#!/usr/bin/env python
"""Benchmark of the AdaComp hot path on B200: SELECT_GRAD (select + compact) over resident dense
gradients, then the parameter-server update of the selected pairs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 0..4] [--keep a/b] [--impl reference]

One step = one pass of the whole hot path over one batch of synthetic input: for every keep
fraction of the workload, select the gradients of all workers, then apply the resulting updates in
a seeded arrival order.  Default workload: the 100 M-parameter one (25 tensors x 4 M, 16 workers,
six keep fractions from 0.1 % to 10 %).  Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1702_04683_b200 import workloads as wlmod  # noqa: E402

METRIC = "dense-gradient GB/s scanned (select+compact, with the selected pairs applied)"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM bytes (read + write) of ONE launch of the scan kernel and of the apply kernel that does the work, from ncu
# captures of workload 4, MB per keep fraction.  The scan kernel was captured with 4 of the 16 workers: a launch over W
# workers moves W / 4 times as much (every worker's tensors are independent).  The apply kernel was captured with all 16
# updates in the launch on tensors four times smaller: parameters and pairs, hence the traffic, are a quarter of a
# full-size launch's.  Only valid while the kernel sources are the ones that were profiled (guarded by their hashes).
SCAN_TRAFFIC_W4_MB = {'1/1000': 1617.2, '1/400': 1627.7, '1/160': 1648.3, '1/64': 1691.3, '1/25': 1789.2, '1/10': 2010.6}
APPLY_TRAFFIC_DIV4_MB = {'1/1000': 91.3, '1/400': 190.1, '1/160': 327.4, '1/64': 463.5, '1/25': 632.0, '1/10': 924.8}
SCAN_SOURCE_SHA256_16 = "fa86615eff0206da"
APPLY_SOURCE_SHA256_16 = "6dff16245f48ee38"


def _source_hash(name):
    import hashlib
    try:
        src = open(os.path.join(ROOT, "paper_1702_04683_b200", "csrc", name), "rb").read()
    except OSError:
        return None
    return hashlib.sha256(src).hexdigest()[:16]


def scan_traffic_bytes(workload_index, keeps, workers):
    """Mean DRAM bytes per scan launch over the given keep fractions, or None if unknown."""
    if not SCAN_SOURCE_SHA256_16 or _source_hash("select_bracket.cuh") != SCAN_SOURCE_SHA256_16 or workload_index != 4:
        return None
    try:
        per = [SCAN_TRAFFIC_W4_MB["%d/%d" % k] * 1e6 * workers / 4.0 for k in keeps]
    except KeyError:
        return None
    return sum(per) / len(per)


def apply_traffic_mb(workload_index, keep):
    """DRAM MB of a full-size apply launch at this keep fraction: 4 x the ncu capture of the 16-update launch on tensors
    four times smaller (--divide 4; parameters and pairs, hence the traffic, scale together), or None if unknown."""
    if not APPLY_SOURCE_SHA256_16 or _source_hash("apply.cu") != APPLY_SOURCE_SHA256_16 or workload_index != 4:
        return None
    mb = APPLY_TRAFFIC_DIV4_MB.get("%d/%d" % keep)
    return None if mb is None else round(4.0 * mb, 1)


def run_apply_variants(binding, wl, dev, peak, keep=(1, 100), reps=5, warmup=3):
    """adacomp_apply on index sets and windows the main sweep does not show, at one keep fraction, W updates per call:
    'uniform' (one index per stratum, all pulled at the round's start: what top-k of iid data gives), 'clustered' (all
    pairs of an update inside a random twentieth of each tensor, as real gradients crowd into rows and layers) and
    'stale' (uniform index sets, every update pulled 2 W updates before it is applied: windows that reach back over two
    earlier rounds)."""
    W, P = wl.n_workers, wl.n_params
    ks = [binding.adacomp_keep_count(n, *keep) for n in wl.tensor_sizes]
    K = int(sum(ks))
    stream = torch.cuda.current_stream()
    idx_u, val = wlmod.synthetic_updates(wl, ks, 0, dev)
    # clustered: squeeze every tensor's strata into a window of n / 20 entries at a seeded offset per (worker, tensor)
    gen = torch.Generator(device=dev)
    gen.manual_seed(4242)
    idx_c = torch.empty_like(idx_u)
    at = 0
    for off, n, k in zip(wl.offsets, wl.tensor_sizes, ks):
        width = max(k, n // 20)
        start = (torch.rand((W, 1), device=dev, generator=gen) * (n - width)).to(torch.int64)
        t = torch.arange(k, dtype=torch.int64, device=dev).view(1, k)
        idx_c[:, at:at + k] = (off + start + (t * width) // k).to(torch.int32)
        at += k
    begin = np.arange(W, dtype=np.uint64) * np.uint64(K)
    count = np.full(W, K, np.uint32)
    out = {"keep": "%d/%d" % keep, "updates_per_call": W, "pairs_per_update": K}

    def timed(srv, idx, stale):
        def call(fresh=False):
            ts = srv.timestamp
            pull = np.full(W, ts, np.uint64) if fresh or not stale else (ts + np.arange(W, dtype=np.uint64) - np.uint64(2 * W))
            srv.apply(idx.view(-1), val.view(-1), begin, count, pull, wl.lr)
        for _ in range(2):
            call(fresh=True)                                       # two rounds of history for the stale windows to reach into
        for _ in range(warmup):
            call()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(reps):
            call()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    for name, idx, stale in (("uniform", idx_u, False), ("clustered", idx_c, False), ("stale", idx_u, True)):
        theta = wlmod.initial_parameters(wl, dev)
        srv = binding.Server(theta, history_pairs=4 * W * K, max_window_updates=4 * W)
        ms = timed(srv, idx, stale)
        assert srv.last_error() == 0
        out[name] = {"apply_ms": round(ms, 4), "apply_pairs_per_s": round(W * K / ms * 1e3, 1),
                     "apply_alg_frac_of_hbm_peak": round(W * K * 28.0 / ms / 1e6 / peak, 4)}
        del srv, theta
    return out


def run_competitors(binding, wl, grads, dev, peak, keep=(1, 100), reps=5, warmup=3):
    """The paper's two competitors on the same inputs, next to AdaComp at the same keep fraction:
    ASGD (dense updates) and Comp-ASGD (whole-model top-k), both with the learning rate divided by the
    update's staleness.  Every worker pulls at the start of a round; a round = W updates.  Ingress
    bytes per update follow the paper's accounting (size of what the server receives)."""
    W, P = grads.shape[0], wl.n_params
    stream = torch.cuda.current_stream()

    def timed(fn):
        for _ in range(warmup):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(reps):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    out = {"keep": "%d/%d" % keep, "workers": W, "round": "W updates, all pulled at the start of the round"}
    begin = lambda K: np.arange(W, dtype=np.uint64) * np.uint64(K)
    # ASGD: W dense updates
    theta = wlmod.initial_parameters(wl, dev)
    srv = binding.Server(theta, history_pairs=1, max_window_updates=2 * W)
    srv.set_rule(1)
    def asgd_round():
        ts = srv.timestamp
        for w in range(W):
            srv.apply_dense(grads[w, :P], ts, wl.lr)
    ms = timed(asgd_round)
    out["asgd"] = {"apply_ms_per_round": round(ms, 4), "updates_per_s": round(W / ms * 1e3, 1),
                   "apply_gbs_12B_per_param": round(W * 12.0 * P / ms / 1e6, 1),
                   "apply_frac_of_hbm_peak": round(W * 12.0 * P / ms / 1e6 / peak, 4),
                   "ingress_bytes_per_update": 4 * P}
    assert srv.last_error() == 0
    # Comp-ASGD: whole-model top-k (one segment), sparse updates under the global rule
    k = binding.adacomp_keep_count(P, keep[0], keep[1])
    sel = binding.Selector(binding.segments_from([0], [P], [k]), W, dev)
    idx, val = sel.select(grads)
    sel_ms = timed(lambda: sel.select(grads, idx, val))
    count = np.full(W, k, np.uint32)
    app_ms = timed(lambda: srv.apply(idx.view(-1), val.view(-1), begin(k), count, np.full(W, srv.timestamp, np.uint64), wl.lr))
    out["comp_asgd"] = {"select": "one segment over all %d parameters" % P,
                        "select_ms_per_round": round(sel_ms, 4), "select_scanned_gbs": round(W * 4.0 * P / sel_ms / 1e6, 1),
                        "apply_ms_per_round": round(app_ms, 4), "apply_pairs_per_s": round(W * k / app_ms * 1e3, 1),
                        "ingress_bytes_per_update": 8 * k}
    assert sel.last_error()[0] == 0 and srv.last_error() == 0
    del sel, srv
    # AdaComp at the same keep fraction: per-tensor top-k, per-parameter staleness
    sel = binding.Selector(binding.make_segments(wl.tensor_sizes, keep), W, dev)
    K = sel.pairs_per_worker
    idx, val = sel.select(grads)
    sel_ms = timed(lambda: sel.select(grads, idx, val))
    srv = binding.Server(theta, history_pairs=2 * W * K, max_window_updates=2 * W)
    count = np.full(W, K, np.uint32)
    app_ms = timed(lambda: srv.apply(idx.view(-1), val.view(-1), begin(K), count, np.full(W, srv.timestamp, np.uint64), wl.lr))
    out["adacomp"] = {"select_ms_per_round": round(sel_ms, 4), "select_scanned_gbs": round(W * 4.0 * P / sel_ms / 1e6, 1),
                      "apply_ms_per_round": round(app_ms, 4), "apply_pairs_per_s": round(W * K / app_ms * 1e3, 1),
                      "ingress_bytes_per_update": 8 * K}
    assert sel.last_error()[0] == 0 and srv.last_error() == 0
    # the two history structures on the same updates: chains (automatic mode) against the paper's sorted
    # lists with one search per update of the window; "fresh" = all pulled at the start of the round
    # (windows of 0 .. W - 1 updates), "stale" = every update pulled 2 W updates before it is applied
    hist = {}
    for name, mode in (("chains", 0), ("sorted_lists", 4)):
        srv = binding.Server(theta, history_pairs=4 * W * K, max_window_updates=4 * W)
        srv.set_mode(mode)
        fresh = lambda: srv.apply(idx.view(-1), val.view(-1), begin(K), count, np.full(W, srv.timestamp, np.uint64), wl.lr)
        stale = lambda: srv.apply(idx.view(-1), val.view(-1), begin(K), count,
                                  srv.timestamp + np.arange(W, dtype=np.uint64) - np.uint64(2 * W), wl.lr)
        f_ms = timed(fresh)
        s_ms = timed(stale)
        hist[name] = {"fresh_apply_ms_per_round": round(f_ms, 4), "stale_apply_ms_per_round": round(s_ms, 4)}
        assert srv.last_error() == 0
        del srv
    out["history_structures"] = hist
    return out


def run_encoding(binding, points, W, peak, reps=5, warmup=3):
    """The index coding on what the last step selected, per keep fraction: bytes per pair on the wire
    (coded index + 4-byte value, against 8 plain) and the time to code and decode W updates."""
    stream = torch.cuda.current_stream()
    out = []
    for p in points:
        words, off = binding.adacomp_encode_indices(p.idx)
        cap = words.shape[1]

        def timed(fn):
            for _ in range(warmup):
                fn()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(reps):
                fn()
            b.record(stream)
            torch.cuda.synchronize()
            return a.elapsed_time(b) / reps
        raw = binding.raw()
        dev_index = p.idx.device.index or 0
        back = torch.empty_like(p.idx)
        enc_ms = timed(lambda: binding._check(raw.adacomp_encode_indices(p.idx.data_ptr(), p.K, W, words.data_ptr(), cap, off.data_ptr(),
                                                                         dev_index, int(stream.cuda_stream)), "encode"))
        dec_ms = timed(lambda: binding._check(raw.adacomp_decode_indices(words.data_ptr(), cap, off.data_ptr(), p.K, W, back.data_ptr(),
                                                                         dev_index, int(stream.cuda_stream)), "decode"))
        if not torch.equal(back, p.idx):
            raise SystemExit("index coding: the round trip changed an index")
        coded_words = float(off[:, -1].sum().item())
        del words, off, back
        # the values, packed losslessly
        vwords, voff = binding.adacomp_encode_values(p.val)
        vcap = vwords.shape[1]
        vback = torch.empty_like(p.val)
        venc_ms = timed(lambda: binding._check(raw.adacomp_encode_values(p.val.data_ptr(), p.K, W, vwords.data_ptr(), vcap, voff.data_ptr(),
                                                                         dev_index, int(stream.cuda_stream)), "encode values"))
        vdec_ms = timed(lambda: binding._check(raw.adacomp_decode_values(vwords.data_ptr(), vcap, voff.data_ptr(), p.K, W, vback.data_ptr(),
                                                                         dev_index, int(stream.cuda_stream)), "decode values"))
        if not torch.equal(vback.view(torch.int32), p.val.view(torch.int32)):
            raise SystemExit("value packing: the round trip changed a value")
        value_words = float(voff[:, -1].sum().item())
        idx_bytes, val_bytes = 4.0 * coded_words / (W * p.K), 4.0 * value_words / (W * p.K)
        out.append({"keep": f"{p.keep[0]}/{p.keep[1]}", "plain_bytes_per_pair": 8.0,
                    "bytes_per_pair": round(4.0 + idx_bytes, 3),                      # coded indices, plain values
                    "bytes_per_pair_values_packed": round(idx_bytes + val_bytes, 3),  # coded indices, packed values
                    "index_bytes": round(idx_bytes, 3), "value_bytes": round(val_bytes, 3),
                    "encode_ms": round(enc_ms, 4), "decode_ms": round(dec_ms, 4),
                    "encode_pairs_per_s": round(W * p.K / enc_ms * 1e3, 1), "decode_pairs_per_s": round(W * p.K / dec_ms * 1e3, 1),
                    "values_encode_ms": round(venc_ms, 4), "values_decode_ms": round(vdec_ms, 4)})
        del vwords, voff, vback
    return out


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", type=int, default=4)
    ap.add_argument("--keep", default=None, help="one keep fraction a/b instead of the workload's list")
    ap.add_argument("--workers", type=int, default=None, help="override the number of workers (smaller captures)")
    ap.add_argument("--divide", type=int, default=None,
                    help="every tensor this many times smaller, the number of workers kept (smaller captures of the "
                         "kernels that take all workers' updates in one launch)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--apply-mode", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-competitors", action="store_true")
    ap.add_argument("--sharded", action="store_true",
                    help="N > 1: one server sharded by parameter range over the ranks (each rank selects for W / N workers, "
                         "the updates' slices are exchanged, every rank applies its range) instead of N independent replicas")
    return ap.parse_args()


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(names, f[5:9]):
                    if v.lower() == "active":
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def parse_keep(text):
    a, b = text.split("/")
    return int(a), int(b)


def setup_dist(args):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    elif args.sharded:
        # one rank: the exchange of the sharded server is a local copy, but its path is the one that runs
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29533")
        dist.init_process_group("gloo", rank=0, world_size=1)
    return world, rank, local


# ------------------------------------------------------------------------------------------ native arm

class Point:
    """One keep fraction of the workload: its selector, output buffers and pair count."""

    def __init__(self, binding, wl, keep, dev):
        self.keep = keep
        self.segs = binding.make_segments(wl.tensor_sizes, keep)
        self.sel = binding.Selector(self.segs, wl.n_workers, dev)
        self.K = self.sel.pairs_per_worker
        self.idx = torch.empty((wl.n_workers, self.K), dtype=torch.int32, device=dev)
        self.val = torch.empty((wl.n_workers, self.K), dtype=torch.float32, device=dev)
        self.count = np.full(wl.n_workers, self.K, dtype=np.uint32)


def step_schedule(wl, rng, srv_ts, last_push_ts):
    """Arrival order and pull timestamps of one round starting at server timestamp srv_ts."""
    W = wl.n_workers
    order = rng.permutation(W)
    if wl.schedule == "rounds":
        pull = np.where(last_push_ts[order] < 0, srv_ts, last_push_ts[order] + 1)
        pull = np.maximum(pull, srv_ts - (2 * W - 1)).astype(np.uint64)
    else:
        pull = np.full(W, srv_ts, dtype=np.uint64)
    last_push_ts[order] = srv_ts + np.arange(W)
    return order, pull


def run_native(args):
    from paper_1702_04683_b200 import binding
    world, rank, local = setup_dist(args)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    import dataclasses
    sharded = bool(args.sharded)
    wl = wlmod.workload(args.workload, seed=0 if sharded else rank)
    if args.workers:
        wl = dataclasses.replace(wl, n_workers=args.workers)
    if args.divide:
        wl = wl.scaled(args.divide)
    keeps = [parse_keep(args.keep)] if args.keep else list(wl.keep_fractions)
    W, P = wl.n_workers, wl.n_params
    stream = torch.cuda.current_stream()

    if sharded:
        # ONE server over all ranks: rank r hosts W / N workers and owns a contiguous range of the parameters
        from paper_1702_04683_b200 import sharding
        if W % world:
            raise SystemExit("--sharded needs a worker count that the number of ranks divides")
        W_local = W // world
        wl_local = dataclasses.replace(wl, n_workers=W_local)
        grads = wlmod.round_gradients(wl, 0, dev, workers=range(rank * W_local, (rank + 1) * W_local))
        points = [Point(binding, wl_local, k, dev) for k in keeps]
        K_max = max(p.K for p in points)
        lo, hi = sharding.parameter_ranges(P, world)[rank]
        theta = wlmod.initial_parameters(wl, dev)[lo:hi].clone()
        ssrv = sharding.ShardedServer(theta, P, W_local, history_pairs=2 * W * K_max, max_window_updates=2 * W)
        srv = ssrv.applier
        rng = np.random.default_rng(1234)                            # the same arrival order on every rank
    else:
        grads = wlmod.round_gradients(wl, 0, dev)                   # resident before the timer starts
        points = [Point(binding, wl, k, dev) for k in keeps]
        K_max = max(p.K for p in points)
        theta = wlmod.initial_parameters(wl, dev)
        srv = binding.Server(theta, history_pairs=2 * W * K_max, max_window_updates=2 * W)
        rng = np.random.default_rng(1234 + rank)
    srv.set_mode(args.apply_mode)
    last_push = np.full(W, -1, dtype=np.int64)

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def one_step(record):
        marks = []
        for p in points:
            order, pull = step_schedule(wl, rng, srv.timestamp, last_push)
            e0 = ev(); e0.record(stream)
            p.sel.select(grads, p.idx, p.val)
            e1 = ev(); e1.record(stream)
            if sharded:
                ssrv.step(p.idx, p.val, order, pull, wl.lr)
            else:
                srv.apply(p.idx.view(-1), p.val.view(-1), order.astype(np.uint64) * np.uint64(p.K), p.count, pull, wl.lr)
            e2 = ev(); e2.record(stream)
            marks.append((e0, e1, e2))
        if record is not None:
            record.append(marks)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        one_step(None)
    for p in points:
        p.sel.set_profiling(2)         # CUDA events around the scan kernel of every timed select call (no syncs)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = binding.adacomp_kernel_launches()
    rec = []
    t0, t1 = ev(), ev()
    barrier()
    t0.record(stream)
    for _ in range(args.steps):
        one_step(rec)
    t1.record(stream)
    barrier()
    launches = binding.adacomp_kernel_launches() - launches0
    clocks = sampler.stop() if rank == 0 else None
    total_ms = t0.elapsed_time(t1)
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([total_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    scan_profiles = [p.sel.profile() for p in points]        # the scan kernel, over the timed steps
    # where the rest of a select call goes: two more steps, not timed, with events around every kernel
    for p in points:
        p.sel.set_profiling(1)
    for _ in range(2):
        one_step(None)
    barrier()
    stage_profiles = [p.sel.profile() for p in points]
    for p in points:
        p.sel.set_profiling(0)
    status = [p.sel.last_error()[0] for p in points] + [srv.last_error()]
    if any(status):
        raise SystemExit(f"device-side error recorded during the benchmark: {status}")

    # per keep fraction: mean select / apply time over the timed steps
    peak, peak_kind = hbm_peak()
    pts = []
    sel_ms_all, sel_bytes_all = 0.0, 0.0
    scan_ms_all, scan_bytes_all, scan_launches = 0.0, 0.0, 0
    W_sel = W // world if sharded else W          # workers one rank selects for
    apply_points = []
    for i, p in enumerate(points):
        calls = scan_profiles[i].pop("calls")
        stages = stage_profiles[i]
        stages.pop("calls")
        scan_ms_timed = scan_profiles[i]["bracket_scan"]
        scan_ms_all += scan_ms_timed
        scan_bytes_all += W_sel * 4.0 * P
        scan_launches += calls
        sel_ms = statistics.mean(m[i][0].elapsed_time(m[i][1]) for m in rec)
        app_ms = statistics.mean(m[i][1].elapsed_time(m[i][2]) for m in rec)
        scanned = W_sel * 4.0 * P
        sel_alg = W_sel * (4.0 * P + 8.0 * p.K)
        pairs = W * p.K / (world if sharded else 1)
        # what the apply launch must move when it sweeps Theta and heads once (16 B per parameter it owns) and reads the
        # pairs and writes their links (12 B per pair), against the 28 B per pair of the per-pair formulation
        sweep_bytes = 16.0 * (P / (world if sharded else 1)) + 12.0 * pairs
        cap_mb = apply_traffic_mb(args.workload, p.keep)
        sweeps = args.apply_mode == 3 or (args.apply_mode == 0 and pairs >= 0.08 * (P / (world if sharded else 1)))
        apply_points.append({"keep": f"{p.keep[0]}/{p.keep[1]}", "apply_ms": round(app_ms, 4),
                             "alg_gbs_28B_per_pair": round(pairs * 28.0 / app_ms / 1e6, 1),
                             "alg_frac": round(pairs * 28.0 / app_ms / 1e6 / peak, 4),
                             # only where the launch does sweep (the library's rule: pairs >= 8 % of the parameters)
                             "sweep_formulation_gbs": round(sweep_bytes / app_ms / 1e6, 1) if sweeps else None,
                             "sweep_formulation_frac": round(sweep_bytes / app_ms / 1e6 / peak, 4) if sweeps else None,
                             "dram_mb_ncu_quarter_size_x4": cap_mb})
        pts.append({
            "keep": f"{p.keep[0]}/{p.keep[1]}", "pairs_per_update": p.K,
            "select_ms": round(sel_ms, 4), "apply_ms": round(app_ms, 4),
            "select_scanned_gbs": round(scanned / sel_ms / 1e6, 1),
            "select_frac_of_hbm_peak": round(sel_alg / sel_ms / 1e6 / peak, 4),
            "selected_elems_per_s": round(pairs / sel_ms * 1e3, 1),
            "apply_pairs_per_s": round(pairs / app_ms * 1e3, 1),
            "apply_updates_per_s": round(W / app_ms * 1e3, 1),
            "apply_alg_gbs_28B_per_pair": round(pairs * 28.0 / app_ms / 1e6, 1),
            "apply_alg_frac_of_hbm_peak": round(pairs * 28.0 / app_ms / 1e6 / peak, 4),
            "scan_kernel_ms": round(scan_ms_timed, 4),                       # in the timed steps
            # every kernel of the call, from two extra steps after the timed ones (events between the kernels lengthen a call)
            "select_stage_ms": {k: round(v, 4) for k, v in stages.items() if v > 0},
        })
        sel_ms_all += sel_ms
        sel_bytes_all += sel_alg
    ms_per_step = total_ms / args.steps
    scanned_per_step = len(points) * W * 4.0 * P
    value = (1 if sharded else world) * scanned_per_step / ms_per_step / 1e6     # a sharded job scans W workers in all

    out = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_per_step, 4), "higher_is_better": True,
        "scaling": "strong" if sharded else "weak", "vs_baseline": None, "dtype": "u32 keys / f32 update arithmetic", "data": "synthetic",
        "config": {"workload": wl.name, "tensors": len(wl.tensor_sizes), "params": P, "workers": W,
                   "keep_fractions": [pt["keep"] for pt in pts], "step": "select + apply for every keep fraction",
                   "l2": "inputs larger than L2 (%.1f GB of gradients per keep fraction)" % (W * 4.0 * P / 1e9),
                   "apply_mode": args.apply_mode,
                   "multi_gpu": ("one server sharded by parameter range over the ranks: each rank selects for W / N workers, the updates' "
                                 "slices are exchanged (send / recv), every rank applies its range") if sharded
                   else "independent replicas, one per rank (no data-path collective)"},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "points": pts,
        # dominant kernel: the single streaming pass over the dense gradients.  Algorithmic bytes per
        # launch = workers x 4 bytes x parameters; duration = mean over its launches in the timed
        # region, from CUDA events recorded on the launching stream around the kernel.
        "roofline": {"bound": "hbm", "kernel": "k_bracket_scan (the one pass over the dense gradients)", "launches_timed": int(scan_launches),
                     "achieved": round(scan_bytes_all / scan_ms_all / 1e6, 1) if scan_ms_all else None,
                     "peak": peak, "peak_kind": "of " + peak_kind, "unit": "GB/s",
                     "frac": round(scan_bytes_all / scan_ms_all / 1e6 / peak, 4) if scan_ms_all else None,
                     "traffic": (lambda t: round(t / 1e9, 3) if t else None)(scan_traffic_bytes(args.workload, keeps, W)),
                     "traffic_unit": "GB per launch (ncu dram read + write of a 4-worker capture x W / 4, mean over the keep fractions; algorithmic: %.1f GB)" % (W_sel * 4.0 * P / 1e9),
                     # the apply kernels, per keep fraction: the dominant kernel of the launch against the same peak
                     "apply": {"what": "one adacomp_apply launch of W updates per keep fraction; alg = 28 B per pair; sweep formulation = "
                                       "16 B per parameter + 12 B per pair (what a launch that sweeps Theta and heads once must move)",
                               "points": apply_points},
                     "select_call": {"what": "all kernels of adacomp_select, read 4P + write 8K per worker",
                                     "achieved": round(sel_bytes_all / sel_ms_all / 1e6, 1),
                                     "frac": round(sel_bytes_all / sel_ms_all / 1e6 / peak, 4)}},
    }
    if world == 1 and not args.no_competitors:
        out["encoding"] = run_encoding(binding, points, W, peak)
    if world == 1 and not args.no_competitors and args.keep is None and not sharded:
        out["competitors"] = run_competitors(binding, wl, grads, dev, peak)
        out["apply_variants"] = run_apply_variants(binding, wl, dev, peak)
    if world == 1 and not args.no_e2e and not sharded:
        out["e2e"] = run_e2e(args, binding, wl, points, srv, grads, rng, last_push, dev, stream)
    if world == 1 and rank == 0 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(wl, keeps, grads)
    if rank == 0:
        print(json.dumps(out))
    if world > 1 or sharded:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_e2e(args, binding, wl, points, srv, grads, rng, last_push, dev, stream):
    """Same step through the host entry point: every step copies the gradients host -> device
    from pinned memory and reads the selected pairs back."""
    W, P = wl.n_workers, wl.n_params
    try:
        h_grads = torch.empty((W, P), dtype=torch.float32, pin_memory=True)
    except RuntimeError as e:
        return {"value": None, "unit": UNIT, "error": "cannot pin %.1f GB of host memory: %s" % (W * P * 4 / 1e9, e)}
    h_grads.copy_(grads)
    staging = torch.empty_like(grads)
    K_max = max(p.K for p in points)
    h_idx = torch.empty((W, K_max), dtype=torch.int32, pin_memory=True)
    h_val = torch.empty((W, K_max), dtype=torch.float32, pin_memory=True)
    h2d = d2h = 0

    def step():
        nonlocal h2d, d2h
        for p in points:
            order, pull = step_schedule(wl, rng, srv.timestamp, last_push)
            hi, hv = h_idx.view(-1)[: W * p.K].view(W, p.K), h_val.view(-1)[: W * p.K].view(W, p.K)
            p.sel.select_host(h_grads, staging, p.idx, p.val, hi, hv)
            srv.apply(p.idx.view(-1), p.val.view(-1), order.astype(np.uint64) * np.uint64(p.K), p.count, pull, wl.lr)
            h2d += W * P * 4
            d2h += W * p.K * 8

    step()
    torch.cuda.synchronize()
    h2d = d2h = 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.e2e_steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.e2e_steps
    return {"value": round(len(points) * W * 4.0 * P / ms / 1e6, 2), "unit": UNIT, "ms_per_step": round(ms, 3),
            "steps": args.e2e_steps, "h2d_bytes_per_step": h2d // args.e2e_steps,
            "d2h_bytes_per_step": d2h // args.e2e_steps,
            "what": "adacomp_select_host (pinned host gradients in, pairs out) + adacomp_apply"}


# ------------------------------------------------------------------------------------------ CPU oracle arms

def oracle_sample_pass(wl, keeps, grads_host, sample_workers):
    """The oracle, as it stands, over `sample_workers` workers' gradients and every keep fraction:
    select each, then apply the sampled updates.  Returns (seconds, bytes scanned)."""
    import oracle
    theta0 = wlmod.initial_parameters(wl, "cpu").numpy()
    srv = oracle.Server(theta0)
    t0 = time.perf_counter()
    scanned = 0
    for keep in keeps:
        ks = [oracle.keep_count(n, *keep) for n in wl.tensor_sizes]
        j = srv.timestamp
        for w in range(sample_workers):
            idx, val = oracle.select_layers(grads_host[w], wl.offsets, wl.tensor_sizes, ks)
            srv.apply(idx, val, j, wl.lr)
            scanned += grads_host[w].size * 4
    return time.perf_counter() - t0, scanned


def cpu_baseline(wl, keeps, grads_dev):
    sample_workers = min(2, wl.n_workers)
    g = grads_dev[:sample_workers].cpu().numpy()
    secs, scanned = oracle_sample_pass(wl, keeps, g, sample_workers)
    return {"value": round(scanned / secs / 1e9, 4), "unit": UNIT, "cores": 1, "kind": "oracle",
            "seconds": round(secs, 2), "host_cores_available": os.cpu_count(),
            "sample": "%d of %d workers, all %d keep fractions: oracle select (partial sort) + oracle apply, one thread"
                      % (sample_workers, wl.n_workers, len(keeps))}


def run_reference(args):
    """The CPU oracle timed on the host, each step a bounded sample of the native arm's step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = wlmod.workload(args.workload)
    keeps = [parse_keep(args.keep)] if args.keep else list(wl.keep_fractions)
    sample_workers = 1
    g = wlmod.round_gradients(wl, 0, "cpu", workers=range(sample_workers)).numpy()
    for _ in range(min(args.warmup, 1)):
        oracle_sample_pass(wl, keeps[:1], g, sample_workers)
    steps = max(1, min(args.steps, 3))
    secs = scanned = 0.0
    for _ in range(steps):
        s, b = oracle_sample_pass(wl, keeps, g, sample_workers)
        secs += s
        scanned += b
    value = scanned / secs / 1e9
    sample = "%d of %d workers per step, all %d keep fractions, %d steps" % (sample_workers, wl.n_workers, len(keeps), steps)
    out = {
        "impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": round(secs / steps * 1e3, 2),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32 keys / f32 update arithmetic",
        "data": "synthetic",
        "config": {"workload": wl.name, "tensors": len(wl.tensor_sizes), "params": wl.n_params, "workers": wl.n_workers,
                   "keep_fractions": ["%d/%d" % k for k in keeps], "step": "select + apply for every keep fraction"},
        "cpu_baseline": {"value": round(value, 4), "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(value, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(out))


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_native(a)
