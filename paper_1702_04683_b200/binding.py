"""ctypes binding of ``libadacomp.so``: argument marshalling only.

Every step of the hot path runs inside the CUDA library; this module checks tensor
dtype / device / contiguity, passes raw pointers and raises :class:`AdacompError`
on a non-zero status.  The function names mirror ``include/adacomp.h``;
:class:`Selector` and :class:`Server` are small conveniences that own the
workspace tensors (PyTorch allocates all device memory).

Importing this module loads the shared library and fails loudly if it has not
been built (``python -m paper_1702_04683_b200.build``).  There is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libadacomp.so")

OK, ERR_INVALID, ERR_ALLOC, ERR_CUDA, ERR_WINDOW, ERR_CAPACITY, ERR_UNSORTED, ERR_TIMEOUT, ERR_UNIMPLEMENTED = \
    0, -1, -2, -3, -4, -5, -6, -7, -8


class AdacompError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        text = _lib.adacomp_status_string(status).decode()
        extra = f" (cudaError {_lib.adacomp_last_cuda_error()})" if status == ERR_CUDA else ""
        super().__init__(f"{where}: {text}{extra} [{status}]")


class Segment(ctypes.Structure):
    _fields_ = [("offset", ctypes.c_uint64), ("n", ctypes.c_uint32), ("k", ctypes.c_uint32)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_1702_04683_b200.build` "
            "(nvcc, sm_100a). There is no fallback implementation.")
    L = ctypes.CDLL(LIB_PATH)
    vp, u32, u64, i32, f32 = ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int, ctypes.c_float
    P = ctypes.POINTER
    sig = {
        "adacomp_status_string": (ctypes.c_char_p, [i32]),
        "adacomp_version": (i32, []),
        "adacomp_last_cuda_error": (i32, []),
        "adacomp_kernel_launches": (u64, []),
        "adacomp_keep_count": (i32, [u64, u32, u32, P(u32)]),
        "adacomp_select_workspace_bytes": (i32, [P(Segment), u32, u32, P(ctypes.c_size_t)]),
        "adacomp_select_create": (i32, [P(vp), P(Segment), u32, u32, vp, ctypes.c_size_t, i32]),
        "adacomp_select": (i32, [vp, vp, u64, u32, vp, vp, vp]),
        "adacomp_select_host": (i32, [vp, vp, u64, u32, vp, vp, vp, vp, vp, vp]),
        "adacomp_select_set_route": (i32, [vp, i32]),
        "adacomp_select_route_info": (i32, [vp, P(u32)]),
        "adacomp_select_set_profiling": (i32, [vp, i32]),
        "adacomp_select_profile": (i32, [vp, P(f32), u32, P(u64)]),
        "adacomp_select_stage_name": (ctypes.c_char_p, [u32]),
        "adacomp_select_static": (i32, [vp, u32, u32, vp, vp, i32, vp]),
        "adacomp_select_static_last_error": (i32, [i32, vp]),
        "adacomp_select_pairs_per_worker": (i32, [vp, P(u64)]),
        "adacomp_select_last_error": (i32, [vp, vp, P(u64)]),
        "adacomp_select_destroy": (i32, [vp]),
        "adacomp_server_workspace_bytes": (i32, [u64, u64, P(ctypes.c_size_t)]),
        "adacomp_server_create": (i32, [P(vp), u64, u64, u32, vp, ctypes.c_size_t, i32]),
        "adacomp_server_reset": (i32, [vp, vp, vp]),
        "adacomp_server_pull": (i32, [vp, vp, P(u64), vp]),
        "adacomp_apply": (i32, [vp, vp, vp, P(u64), P(u32), P(u64), u32, f32, vp, vp]),
        "adacomp_apply_host": (i32, [vp, vp, vp, P(u64), P(u32), P(u64), u32, f32, vp, vp, vp, vp, vp]),
        "adacomp_server_timestamp": (i32, [vp, P(u64)]),
        "adacomp_server_set_validation": (i32, [vp, i32]),
        "adacomp_server_set_mode": (i32, [vp, i32]),
        "adacomp_encode_capacity_words": (u64, [u64]),
        "adacomp_encode_indices": (i32, [vp, u64, u32, vp, u64, vp, i32, vp]),
        "adacomp_decode_indices": (i32, [vp, u64, vp, u64, u32, vp, i32, vp]),
        "adacomp_encode_values_capacity_words": (u64, [u64]),
        "adacomp_encode_values": (i32, [vp, u64, u32, vp, u64, vp, i32, vp]),
        "adacomp_decode_values": (i32, [vp, u64, vp, u64, u32, vp, i32, vp]),
        "adacomp_server_set_rule": (i32, [vp, i32]),
        "adacomp_apply_dense": (i32, [vp, vp, u64, f32, vp]),
        "adacomp_select_gather": (i32, [vp, vp, u64, u32, vp, vp, vp]),
        "adacomp_server_debug_skip_positions": (i32, [vp, u64]),
        "adacomp_server_last_error": (i32, [vp, vp]),
        "adacomp_server_destroy": (i32, [vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(L, name)
        fn.restype = res
        fn.argtypes = args
    return L, tuple(sig)


_lib, EXPORTS = _load()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise AdacompError(status, where)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: need a contiguous CUDA tensor of {dtype}")
    return t.data_ptr()


def _host(t: torch.Tensor, dtype, name: str) -> int:
    if t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name}: need a contiguous host tensor of {dtype}")
    return t.data_ptr()


def _u64_array(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.uint64)


# ----------------------------------------------------------------------------- plain functions

def adacomp_version() -> int:
    return int(_lib.adacomp_version())


def adacomp_kernel_launches() -> int:
    return int(_lib.adacomp_kernel_launches())


def adacomp_status_string(status: int) -> str:
    return _lib.adacomp_status_string(status).decode()


def adacomp_keep_count(n: int, c_num: int, c_den: int) -> int:
    k = ctypes.c_uint32(0)
    _check(_lib.adacomp_keep_count(n, c_num, c_den, ctypes.byref(k)), "adacomp_keep_count")
    return int(k.value)


def make_segments(sizes: Sequence[int], keep: Tuple[int, int], offsets: Optional[Sequence[int]] = None):
    """Segment table for consecutive tensors of the given sizes and a keep fraction (num, den)."""
    segs = (Segment * len(sizes))()
    off = 0
    for l, n in enumerate(sizes):
        segs[l].offset = offsets[l] if offsets is not None else off
        segs[l].n = n
        segs[l].k = adacomp_keep_count(n, keep[0], keep[1])
        off += n
    return segs


def segments_from(offsets: Sequence[int], ns: Sequence[int], ks: Sequence[int]):
    segs = (Segment * len(ns))()
    for l in range(len(ns)):
        segs[l].offset, segs[l].n, segs[l].k = int(offsets[l]), int(ns[l]), int(ks[l])
    return segs


def adacomp_select_static(grad: torch.Tensor, k: int, idx_out: torch.Tensor, val_out: torch.Tensor,
                          stream: Optional[torch.cuda.Stream] = None) -> None:
    """Top-k-by-magnitude of one tensor through the entry point that allocates nothing: the caller
    brings the input and both outputs, the scratch is a fixed array inside the library."""
    if not (grad.is_cuda and grad.dtype == torch.float32 and grad.dim() == 1 and grad.stride(0) == 1):
        raise TypeError("grad: need a 1-D contiguous CUDA fp32 tensor")
    _check(_lib.adacomp_select_static(grad.data_ptr(), grad.numel(), int(k), _dev(idx_out, torch.int32, "idx_out"),
                                      _dev(val_out, torch.float32, "val_out"), grad.device.index,
                                      _stream_ptr(stream)), "adacomp_select_static")


def adacomp_select_static_last_error(device_index: int = 0, stream: Optional[torch.cuda.Stream] = None) -> int:
    """Waits for the stream; first device-side error of adacomp_select_static calls since the last read."""
    return int(_lib.adacomp_select_static_last_error(int(device_index), _stream_ptr(stream)))


# ----------------------------------------------------------------------------- worker side

def adacomp_encode_capacity_words(pairs_per_worker: int) -> int:
    return int(_lib.adacomp_encode_capacity_words(int(pairs_per_worker)))


def adacomp_encode_indices(idx: torch.Tensor, stream: Optional[torch.cuda.Stream] = None):
    """idx [W, K] (int32 holding uint32 bit patterns) -> (words [W, capacity] int32, block_off [W, n_blocks + 1]
    int64): the block-wise gap coding of every worker's index list."""
    if idx.dim() == 1:
        idx = idx.unsqueeze(0)
    W, K = idx.shape
    cap = adacomp_encode_capacity_words(K)
    words = torch.empty((W, max(cap, 1)), dtype=torch.int32, device=idx.device)
    off = torch.empty((W, (K + 255) // 256 + 1), dtype=torch.int64, device=idx.device)
    _check(_lib.adacomp_encode_indices(_dev(idx, torch.int32, "idx") if K else None, K, W, words.data_ptr(), words.shape[1],
                                       off.data_ptr(), idx.device.index or 0, _stream_ptr(stream)), "adacomp_encode_indices")
    return words, off


def adacomp_decode_indices(words: torch.Tensor, block_off: torch.Tensor, pairs_per_worker: int,
                           stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    W = words.shape[0]
    out = torch.empty((W, pairs_per_worker), dtype=torch.int32, device=words.device)
    _check(_lib.adacomp_decode_indices(_dev(words, torch.int32, "words"), words.shape[1], _dev(block_off, torch.int64, "block_off"),
                                       int(pairs_per_worker), W, out.data_ptr(), words.device.index or 0, _stream_ptr(stream)),
           "adacomp_decode_indices")
    return out


def adacomp_encode_values_capacity_words(pairs_per_worker: int) -> int:
    return int(_lib.adacomp_encode_values_capacity_words(int(pairs_per_worker)))


def adacomp_encode_values(val: torch.Tensor, stream: Optional[torch.cuda.Stream] = None):
    """val [W, K] float32 -> (words [W, capacity] int32, block_off [W, n_blocks + 1] int64): the lossless block-wise
    packing of every worker's values."""
    if val.dim() == 1:
        val = val.unsqueeze(0)
    W, K = val.shape
    cap = adacomp_encode_values_capacity_words(K)
    words = torch.empty((W, max(cap, 1)), dtype=torch.int32, device=val.device)
    off = torch.empty((W, (K + 255) // 256 + 1), dtype=torch.int64, device=val.device)
    _check(_lib.adacomp_encode_values(_dev(val, torch.float32, "val") if K else None, K, W, words.data_ptr(), words.shape[1],
                                      off.data_ptr(), val.device.index or 0, _stream_ptr(stream)), "adacomp_encode_values")
    return words, off


def adacomp_decode_values(words: torch.Tensor, block_off: torch.Tensor, pairs_per_worker: int,
                          stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    W = words.shape[0]
    out = torch.empty((W, pairs_per_worker), dtype=torch.float32, device=words.device)
    _check(_lib.adacomp_decode_values(_dev(words, torch.int32, "words"), words.shape[1], _dev(block_off, torch.int64, "block_off"),
                                      int(pairs_per_worker), W, out.data_ptr(), words.device.index or 0, _stream_ptr(stream)),
           "adacomp_decode_values")
    return out


class Selector:
    """SELECT_GRAD (Algorithm 1) for a fixed tensor layout; owns its device workspace."""

    def __init__(self, segments, max_workers: int, device: Optional[torch.device] = None):
        self.device = torch.device(device if device is not None else "cuda")
        if self.device.index is None:
            self.device = torch.device("cuda", torch.cuda.current_device())
        self.segments = segments
        self.n_segs = len(segments)
        self.max_workers = int(max_workers)
        nbytes = ctypes.c_size_t(0)
        _check(_lib.adacomp_select_workspace_bytes(segments, self.n_segs, self.max_workers, ctypes.byref(nbytes)),
               "adacomp_select_workspace_bytes")
        self.workspace = torch.empty(max(int(nbytes.value), 256), dtype=torch.uint8, device=self.device)
        h = ctypes.c_void_p()
        _check(_lib.adacomp_select_create(ctypes.byref(h), segments, self.n_segs, self.max_workers,
                                          self.workspace.data_ptr(), self.workspace.numel(), self.device.index),
               "adacomp_select_create")
        self._h = h
        k = ctypes.c_uint64(0)
        _check(_lib.adacomp_select_pairs_per_worker(self._h, ctypes.byref(k)), "adacomp_select_pairs_per_worker")
        self.pairs_per_worker = int(k.value)

    def select(self, grads: torch.Tensor, idx_out: Optional[torch.Tensor] = None,
               val_out: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
        """grads: [W, stride] (or [stride]) fp32 on the device -> (idx [W, K] as int32 bit
        pattern of uint32, val [W, K] fp32)."""
        if grads.dim() == 1:
            grads = grads.unsqueeze(0)
        if grads.stride(-1) != 1:
            raise TypeError("grads: innermost dimension must be contiguous")
        W = grads.shape[0]
        stride = grads.stride(0) if W > 1 else grads.shape[1]
        if not (grads.is_cuda and grads.dtype == torch.float32):
            raise TypeError("grads: need a CUDA fp32 tensor")
        K = self.pairs_per_worker
        if idx_out is None:
            idx_out = torch.empty((W, K), dtype=torch.int32, device=grads.device)
        if val_out is None:
            val_out = torch.empty((W, K), dtype=torch.float32, device=grads.device)
        _check(_lib.adacomp_select(self._h, grads.data_ptr(), stride, W, _dev(idx_out, torch.int32, "idx_out"),
                                   _dev(val_out, torch.float32, "val_out"), _stream_ptr(stream)), "adacomp_select")
        return idx_out, val_out

    def select_host(self, h_grads: torch.Tensor, d_grads: torch.Tensor, d_idx: torch.Tensor, d_val: torch.Tensor,
                    h_idx: torch.Tensor, h_val: torch.Tensor, stream: Optional[torch.cuda.Stream] = None):
        W = h_grads.shape[0]
        _check(_lib.adacomp_select_host(self._h, _host(h_grads, torch.float32, "h_grads"), h_grads.shape[1], W,
                                        _dev(d_grads, torch.float32, "d_grads"), _dev(d_idx, torch.int32, "d_idx"),
                                        _dev(d_val, torch.float32, "d_val"), _host(h_idx, torch.int32, "h_idx"),
                                        _host(h_val, torch.float32, "h_val"), _stream_ptr(stream)),
               "adacomp_select_host")

    def gather(self, grads: torch.Tensor, idx: torch.Tensor, val_out: Optional[torch.Tensor] = None,
               stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """val[w][e] = grads[w][idx[w][e]] for idx of shape [W, pairs_per_worker]."""
        g = grads if grads.dim() == 2 else grads.unsqueeze(0)
        W = g.shape[0]
        if idx.numel() != W * self.pairs_per_worker:
            raise ValueError("idx needs pairs_per_worker entries per worker")
        if val_out is None:
            val_out = torch.empty((W, self.pairs_per_worker), dtype=torch.float32, device=g.device)
        if g.stride(1) != 1 or not (g.is_cuda and g.dtype == torch.float32):
            raise TypeError("grads: need a CUDA fp32 tensor whose innermost dimension is contiguous")
        _check(_lib.adacomp_select_gather(self._h, g.data_ptr(), g.stride(0) if W > 1 else g.shape[1],
                                          W, _dev(idx, torch.int32, "idx"), _dev(val_out, torch.float32, "val_out"),
                                          _stream_ptr(stream)), "adacomp_select_gather")
        return val_out

    def set_route(self, route: int):
        """0 = automatic (bracketed single pass where eligible), 1 = general route only."""
        _check(_lib.adacomp_select_set_route(self._h, int(route)), "adacomp_select_set_route")

    def route_info(self) -> dict:
        """Tensors on the cluster route and the cluster shape chosen on this device."""
        info = (ctypes.c_uint32 * 4)()
        _check(_lib.adacomp_select_route_info(self._h, info), "adacomp_select_route_info")
        return {"cluster_tensors": int(info[0]), "blocks_per_cluster": int(info[1]), "ring_slots": int(info[2]) & 255,
                "warps_per_block": int(info[2]) >> 8, "resident_clusters": int(info[3])}

    def set_profiling(self, on):
        """False / 0: off; True / 1: CUDA events around every kernel; 2: around the pass over the gradient only."""
        _check(_lib.adacomp_select_set_profiling(self._h, int(on)), "adacomp_select_set_profiling")

    def profile(self) -> dict:
        """Mean device milliseconds per kernel and call since profiling was switched on."""
        n = 0
        while _lib.adacomp_select_stage_name(n):
            n += 1
        ms = (ctypes.c_float * n)()
        calls = ctypes.c_uint64(0)
        _check(_lib.adacomp_select_profile(self._h, ms, n, ctypes.byref(calls)), "adacomp_select_profile")
        out = {_lib.adacomp_select_stage_name(i).decode(): float(ms[i]) for i in range(n)}
        out["calls"] = int(calls.value)
        return out

    def last_error(self, stream: Optional[torch.cuda.Stream] = None) -> Tuple[int, int]:
        """(status, selections that took the general route in the last call); waits for the stream."""
        stats = (ctypes.c_uint64 * 4)()
        status = _lib.adacomp_select_last_error(self._h, _stream_ptr(stream), stats)
        return int(status), int(stats[0])

    def close(self):
        if getattr(self, "_h", None):
            _lib.adacomp_select_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ----------------------------------------------------------------------------- server side

class Server:
    """Parameter server of Algorithm 2; owns its device workspace, borrows theta."""

    def __init__(self, theta: torch.Tensor, history_pairs: int, max_window_updates: int):
        self.device = theta.device
        self.n_params = theta.numel()
        nbytes = ctypes.c_size_t(0)
        _check(_lib.adacomp_server_workspace_bytes(self.n_params, history_pairs, ctypes.byref(nbytes)),
               "adacomp_server_workspace_bytes")
        self.workspace = torch.empty(max(int(nbytes.value), 256), dtype=torch.uint8, device=self.device)
        h = ctypes.c_void_p()
        _check(_lib.adacomp_server_create(ctypes.byref(h), self.n_params, history_pairs, max_window_updates,
                                          self.workspace.data_ptr(), self.workspace.numel(), self.device.index),
               "adacomp_server_create")
        self._h = h
        self.reset(theta)

    def reset(self, theta: torch.Tensor, stream: Optional[torch.cuda.Stream] = None):
        if theta.numel() != self.n_params:
            raise ValueError("theta has the wrong size")
        self.theta = theta
        _check(_lib.adacomp_server_reset(self._h, _dev(theta, torch.float32, "theta"), _stream_ptr(stream)),
               "adacomp_server_reset")

    def pull(self, theta_copy: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None) -> int:
        ts = ctypes.c_uint64(0)
        ptr = _dev(theta_copy, torch.float32, "theta_copy") if theta_copy is not None else None
        _check(_lib.adacomp_server_pull(self._h, ptr, ctypes.byref(ts), _stream_ptr(stream)), "adacomp_server_pull")
        return int(ts.value)

    def apply(self, idx: torch.Tensor, val: torch.Tensor, pair_begin, pair_count, pull_ts, lr: float,
              sigma_out: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
        """Applies len(pull_ts) updates in array (= arrival) order; update b is pairs
        [pair_begin[b], pair_begin[b] + pair_count[b]) of idx / val."""
        pb, pj = _u64_array(pair_begin), _u64_array(pull_ts)
        pc = np.ascontiguousarray(pair_count, dtype=np.uint32)
        if not (pb.size == pj.size == pc.size):
            raise ValueError("pair_begin, pair_count and pull_ts need one entry per update")
        sig = _dev(sigma_out, torch.int32, "sigma_out") if sigma_out is not None else None
        _check(_lib.adacomp_apply(self._h, _dev(idx, torch.int32, "idx"), _dev(val, torch.float32, "val"),
                                  pb.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64)),
                                  pc.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32)),
                                  pj.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64)), pj.size, float(lr), sig,
                                  _stream_ptr(stream)), "adacomp_apply")

    def apply_host(self, h_idx: torch.Tensor, h_val: torch.Tensor, pair_begin, pair_count, pull_ts, lr: float,
                   d_idx: torch.Tensor, d_val: torch.Tensor, d_sigma: Optional[torch.Tensor] = None,
                   h_sigma: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
        pb, pj = _u64_array(pair_begin), _u64_array(pull_ts)
        pc = np.ascontiguousarray(pair_count, dtype=np.uint32)
        if not (pb.size == pj.size == pc.size):
            raise ValueError("pair_begin, pair_count and pull_ts need one entry per update")
        _check(_lib.adacomp_apply_host(self._h, _host(h_idx, torch.int32, "h_idx"), _host(h_val, torch.float32, "h_val"),
                                       pb.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64)),
                                       pc.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32)),
                                       pj.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64)), pj.size, float(lr),
                                       _dev(d_idx, torch.int32, "d_idx"), _dev(d_val, torch.float32, "d_val"),
                                       _dev(d_sigma, torch.int32, "d_sigma") if d_sigma is not None else None,
                                       _host(h_sigma, torch.int32, "h_sigma") if h_sigma is not None else None,
                                       _stream_ptr(stream)), "adacomp_apply_host")

    @property
    def timestamp(self) -> int:
        ts = ctypes.c_uint64(0)
        _check(_lib.adacomp_server_timestamp(self._h, ctypes.byref(ts)), "adacomp_server_timestamp")
        return int(ts.value)

    def set_validation(self, on: bool):
        _check(_lib.adacomp_server_set_validation(self._h, int(on)), "adacomp_server_set_validation")

    def set_mode(self, mode: int):
        """0 automatic, 1 one launch per update, 2 batches that touch only the named parameters, 3 batches over a dense sweep,
        4 the paper's sorted lists with one search per update of the window (only switchable at timestamp 0)."""
        _check(_lib.adacomp_server_set_mode(self._h, int(mode)), "adacomp_server_set_mode")

    def set_rule(self, rule: int):
        """0 AdaComp (per-parameter staleness), 1 the competitors' rule (the update's staleness i - j)."""
        _check(_lib.adacomp_server_set_rule(self._h, int(rule)), "adacomp_server_set_rule")

    def apply_dense(self, delta: torch.Tensor, pull_ts: int, lr: float, stream: Optional[torch.cuda.Stream] = None):
        """One dense update under rule 1: Theta <- Theta - lr / (i - pull_ts) * delta."""
        if delta.numel() != self.n_params:
            raise ValueError("a dense update has one entry per parameter")
        _check(_lib.adacomp_apply_dense(self._h, _dev(delta, torch.float32, "delta"), int(pull_ts), float(lr),
                                        _stream_ptr(stream)), "adacomp_apply_dense")

    def debug_skip_positions(self, count: int):
        _check(_lib.adacomp_server_debug_skip_positions(self._h, int(count)), "adacomp_server_debug_skip_positions")

    def last_error(self, stream: Optional[torch.cuda.Stream] = None) -> int:
        return int(_lib.adacomp_server_last_error(self._h, _stream_ptr(stream)))

    def close(self):
        if getattr(self, "_h", None):
            _lib.adacomp_server_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def raw():
    """The ctypes library object, for tests that call the C ABI directly."""
    return _lib
