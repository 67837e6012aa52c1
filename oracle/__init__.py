"""Python face of the CPU oracle (``adacomp_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU
baseline may import this package; the CUDA library and its binding never do.
The oracle is compiled with g++ on first use into ``oracle/liboracle.so``.
Arrays are numpy, fp32 / uint32 / uint64, C-contiguous.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "adacomp_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None

_CXXFLAGS = ["-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.run(["g++", *_CXXFLAGS, "-o", tmp, _SRC], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = ctypes.CDLL(build())
            u32p, f32p, u64p = (ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(ctypes.c_float),
                                ctypes.POINTER(ctypes.c_uint64))
            L.oracle_keep_count.restype = ctypes.c_uint32
            L.oracle_keep_count.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32]
            for name in ("oracle_select_sort", "oracle_select"):
                f = getattr(L, name)
                f.restype = ctypes.c_int
                f.argtypes = [f32p, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint64, u32p, f32p]
            L.oracle_select_layers.restype = ctypes.c_int
            L.oracle_select_layers.argtypes = [f32p, u64p, u32p, u32p, ctypes.c_uint32, ctypes.c_int, u32p, f32p]
            for kind in ("literal", "server", "global"):
                getattr(L, f"oracle_{kind}_create").restype = ctypes.c_void_p
                getattr(L, f"oracle_{kind}_create").argtypes = [ctypes.c_uint64, f32p]
                getattr(L, f"oracle_{kind}_destroy").restype = None
                getattr(L, f"oracle_{kind}_destroy").argtypes = [ctypes.c_void_p]
                getattr(L, f"oracle_{kind}_timestamp").restype = ctypes.c_uint64
                getattr(L, f"oracle_{kind}_timestamp").argtypes = [ctypes.c_void_p]
                getattr(L, f"oracle_{kind}_theta").restype = None
                getattr(L, f"oracle_{kind}_theta").argtypes = [ctypes.c_void_p, f32p]
                getattr(L, f"oracle_{kind}_apply").restype = ctypes.c_int
                getattr(L, f"oracle_{kind}_apply").argtypes = [
                    ctypes.c_void_p, u32p, f32p, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_float, u32p]
            L.oracle_global_apply_dense.restype = ctypes.c_int
            L.oracle_global_apply_dense.argtypes = [ctypes.c_void_p, f32p, ctypes.c_uint64, ctypes.c_float]
            L.oracle_gather.restype = ctypes.c_int
            L.oracle_gather.argtypes = [f32p, ctypes.c_uint64, u32p, ctypes.c_uint64, f32p]
            L.oracle_encode_indices.restype = ctypes.c_uint64
            L.oracle_encode_indices.argtypes = [u32p, ctypes.c_uint64, u32p, u64p]
            L.oracle_decode_indices.restype = ctypes.c_int
            L.oracle_decode_indices.argtypes = [u32p, u64p, ctypes.c_uint64, u32p]
            L.oracle_encode_values.restype = ctypes.c_uint64
            L.oracle_encode_values.argtypes = [f32p, ctypes.c_uint64, u32p, u64p]
            L.oracle_decode_values.restype = ctypes.c_int
            L.oracle_decode_values.argtypes = [u32p, u64p, ctypes.c_uint64, f32p]
            L.oracle_parameter_trace.restype = ctypes.c_int
            L.oracle_parameter_trace.argtypes = [
                ctypes.c_uint32, ctypes.c_float, u32p, f32p, u64p, u64p, ctypes.c_uint64, ctypes.c_uint64,
                ctypes.c_float, u32p, u64p, f32p]
            _lib = L
    return _lib


def keep_count(n: int, c_num: int, c_den: int) -> int:
    return int(lib().oracle_keep_count(n, c_num, c_den))


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def select(g, k: int, offset: int = 0, full_sort: bool = False):
    """SELECT_GRAD on one tensor -> (idx uint32[k], val float32[k]), ascending index."""
    g = _f32(g).ravel()
    idx = np.empty(k, dtype=np.uint32)
    val = np.empty(k, dtype=np.float32)
    fn = lib().oracle_select_sort if full_sort else lib().oracle_select
    rc = fn(_p(g, ctypes.c_float), g.size, k, offset, _p(idx, ctypes.c_uint32), _p(val, ctypes.c_float))
    if rc != 0:
        raise ValueError("oracle select: k > n")
    return idx, val


def select_layers(grad, offsets, ns, ks, full_sort: bool = False):
    """SELECT_GRAD over every tensor of one worker's gradient vector."""
    grad = _f32(grad).ravel()
    offsets = np.ascontiguousarray(offsets, dtype=np.uint64)
    ns = np.ascontiguousarray(ns, dtype=np.uint32)
    ks = np.ascontiguousarray(ks, dtype=np.uint32)
    K = int(ks.astype(np.uint64).sum())
    idx = np.empty(K, dtype=np.uint32)
    val = np.empty(K, dtype=np.float32)
    rc = lib().oracle_select_layers(_p(grad, ctypes.c_float), _p(offsets, ctypes.c_uint64),
                                    _p(ns, ctypes.c_uint32), _p(ks, ctypes.c_uint32), len(ns),
                                    int(full_sort), _p(idx, ctypes.c_uint32), _p(val, ctypes.c_float))
    if rc != 0:
        raise ValueError("oracle select_layers: k > n in some tensor")
    return idx, val


class Server:
    """Algorithm 2 on the CPU. ``literal=True`` evaluates Eq. 3 by membership tests
    over every update of the window; the default keeps per-parameter timestamp lists.
    ``rule="global"`` is the competitors' rule instead (ASGD, Comp-ASGD): one staleness
    i - j for the whole update."""

    def __init__(self, theta0, literal: bool = False, rule: str = "adacomp"):
        if rule not in ("adacomp", "global"):
            raise ValueError("rule must be 'adacomp' or 'global'")
        self._kind = "global" if rule == "global" else ("literal" if literal else "server")
        theta0 = _f32(theta0).ravel()
        self.n_params = theta0.size
        self._h = getattr(lib(), f"oracle_{self._kind}_create")(self.n_params, _p(theta0, ctypes.c_float))

    def apply(self, idx, val, pull_ts: int, alpha: float):
        """One push (update, j). Returns sigma per entry (uint32)."""
        idx = np.ascontiguousarray(idx, dtype=np.uint32)
        val = _f32(val)
        sigma = np.empty(idx.size, dtype=np.uint32)
        rc = getattr(lib(), f"oracle_{self._kind}_apply")(
            self._h, _p(idx, ctypes.c_uint32), _p(val, ctypes.c_float), idx.size, int(pull_ts),
            float(alpha), _p(sigma, ctypes.c_uint32))
        if rc != 0:
            raise ValueError("oracle apply: bad push (j > i, index out of range or not ascending)")
        return sigma

    def apply_dense(self, delta, pull_ts: int, alpha: float):
        """One dense push (the whole gradient, ASGD); only under rule="global"."""
        if self._kind != "global":
            raise ValueError("dense pushes belong to the global-staleness rule")
        delta = _f32(delta).ravel()
        if delta.size != self.n_params:
            raise ValueError("a dense push has one entry per parameter")
        if lib().oracle_global_apply_dense(self._h, _p(delta, ctypes.c_float), int(pull_ts), float(alpha)) != 0:
            raise ValueError("oracle apply_dense: bad push (j > i)")

    @property
    def timestamp(self) -> int:
        return int(getattr(lib(), f"oracle_{self._kind}_timestamp")(self._h))

    def theta(self):
        out = np.empty(self.n_params, dtype=np.float32)
        getattr(lib(), f"oracle_{self._kind}_theta")(self._h, _p(out, ctypes.c_float))
        return out

    def close(self):
        if self._h:
            getattr(lib(), f"oracle_{self._kind}_destroy")(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def gather(g, idx):
    """val[e] = g[idx[e]]."""
    g = _f32(g).ravel()
    idx = np.ascontiguousarray(idx, dtype=np.uint32)
    out = np.empty(idx.size, dtype=np.float32)
    if lib().oracle_gather(_p(g, ctypes.c_float), g.size, _p(idx, ctypes.c_uint32), idx.size, _p(out, ctypes.c_float)) != 0:
        raise ValueError("oracle gather: index out of range")
    return out


def encode_indices(idx):
    """Block-wise gap coding of an ascending index list -> (words uint32, block_off uint64[n_blocks + 1])."""
    idx = np.ascontiguousarray(idx, dtype=np.uint32)
    n_blocks = (idx.size + 255) // 256
    words = np.empty(idx.size + 2 * n_blocks, dtype=np.uint32)          # the most the format can take
    off = np.empty(n_blocks + 1, dtype=np.uint64)
    total = lib().oracle_encode_indices(_p(idx, ctypes.c_uint32), idx.size, _p(words, ctypes.c_uint32), _p(off, ctypes.c_uint64))
    return words[:int(total)].copy(), off


def decode_indices(words, block_off, n_pairs: int):
    words = np.ascontiguousarray(words, dtype=np.uint32)
    block_off = np.ascontiguousarray(block_off, dtype=np.uint64)
    out = np.empty(n_pairs, dtype=np.uint32)
    if lib().oracle_decode_indices(_p(words, ctypes.c_uint32), _p(block_off, ctypes.c_uint64), n_pairs, _p(out, ctypes.c_uint32)) != 0:
        raise ValueError("oracle decode: bad stream")
    return out


def encode_values(val):
    """Lossless block-wise packing of fp32 values (sign, exponent relative to the block's smallest, mantissa)
    -> (words uint32, block_off uint64[n_blocks + 1])."""
    val = _f32(val)
    n_blocks = (val.size + 255) // 256
    words = np.empty(val.size + n_blocks, dtype=np.uint32)              # the most the format can take
    off = np.empty(n_blocks + 1, dtype=np.uint64)
    total = lib().oracle_encode_values(_p(val, ctypes.c_float), val.size, _p(words, ctypes.c_uint32), _p(off, ctypes.c_uint64))
    return words[:int(total)].copy(), off


def decode_values(words, block_off, n_pairs: int):
    words = np.ascontiguousarray(words, dtype=np.uint32)
    block_off = np.ascontiguousarray(block_off, dtype=np.uint64)
    out = np.empty(n_pairs, dtype=np.float32)
    if lib().oracle_decode_values(_p(words, ctypes.c_uint32), _p(block_off, ctypes.c_uint64), n_pairs, _p(out, ctypes.c_float)) != 0:
        raise ValueError("oracle decode: bad stream")
    return out


def parameter_trace(k: int, theta0_k: float, idx, val, pair_begin, pull_ts, alpha: float,
                    first_timestamp: int = 0):
    """History of one parameter through a sequence of pushes -> (sigmas, final theta_k)."""
    idx = np.ascontiguousarray(idx, dtype=np.uint32)
    val = _f32(val)
    pair_begin = np.ascontiguousarray(pair_begin, dtype=np.uint64)
    pull_ts = np.ascontiguousarray(pull_ts, dtype=np.uint64)
    n_updates = pull_ts.size
    sig = np.empty(max(n_updates, 1), dtype=np.uint32)
    hits = ctypes.c_uint64(0)
    out = ctypes.c_float(0.0)
    rc = lib().oracle_parameter_trace(int(k), ctypes.c_float(theta0_k), _p(idx, ctypes.c_uint32),
                                      _p(val, ctypes.c_float), _p(pair_begin, ctypes.c_uint64),
                                      _p(pull_ts, ctypes.c_uint64), n_updates, int(first_timestamp),
                                      ctypes.c_float(alpha), _p(sig, ctypes.c_uint32),
                                      ctypes.byref(hits), ctypes.byref(out))
    if rc != 0:
        raise ValueError("oracle parameter_trace: pull timestamp after its push")
    return sig[: hits.value].copy(), np.float32(out.value)
