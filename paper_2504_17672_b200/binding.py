"""ctypes binding of libcocodc.so with the same names as the C ABI (include/cocodc.h).

Argument marshalling only.  Tensors are torch CUDA tensors used as plain device
memory: the binding passes their addresses and the current CUDA stream.
"""

from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np
import torch

from . import build as _build

OK, ERR_INVALID_ARG, ERR_ALIGNMENT, ERR_ALIAS, ERR_NONFINITE, ERR_TIMEOUT, ERR_CUDA, ERR_NOMEM = range(8)
COMP_NONE, COMP_TAYLOR = 0, 1
SIGN_FORWARD, SIGN_PRINTED, SIGN_DESCENT = 0, 1, 2
BUDGET_COUNT, BUDGET_PARAMS, BUDGET_PARAMS_EXACT = 0, 1, 2
STAGE_OUTER, STAGE_MERGE, STAGE_SCORE, STAGE_ALL, STAGE_SUMSQ, STAGE_DEFER = 1, 2, 4, 7, 8, 16

EXPORTS = (
    "cocodc_create", "cocodc_destroy", "cocodc_sync_budget", "cocodc_fragment_scores",
    "cocodc_select_fragments", "cocodc_outer_step", "cocodc_outer_step_host", "cocodc_merge", "cocodc_snapshot", "cocodc_snapshot_host",
    "cocodc_poll_status", "cocodc_launch_count", "cocodc_status_string",
    "cocodc_fragment_scores_noalloc", "cocodc_selftest_bounded_wait",
    "cocodc_pseudo_gradient_sum", "cocodc_outer_step_received",
    "cocodc_select_fragments_at", "cocodc_outer_step_at", "cocodc_outer_step_received_peers",
    "cocodc_scores_from_sumsq", "cocodc_bind_in_flight", "cocodc_flush_scores", "cocodc_initiate", "cocodc_initiate_at",
)
NOALLOC_MAX_K, NOALLOC_MAX_SEGMENTS = 64, 64


class CocodcError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = int(code)
        super().__init__(f"{where}: {status_string(code)} (status {int(code)})")


class _Partition(ctypes.Structure):
    _fields_ = [("N", ctypes.c_int64), ("K", ctypes.c_int32), ("n_segments", ctypes.c_int32),
                ("frag_seg_ptr", ctypes.POINTER(ctypes.c_int32)),
                ("seg_offset", ctypes.POINTER(ctypes.c_int64)),
                ("seg_len", ctypes.POINTER(ctypes.c_int64))]


class _Hyper(ctypes.Structure):
    _fields_ = [("M", ctypes.c_int32), ("comp_mode", ctypes.c_int32), ("sign_mode", ctypes.c_int32),
                ("reserved", ctypes.c_int32), ("H", ctypes.c_int64), ("tau", ctypes.c_int64),
                ("outer_lr", ctypes.c_float), ("momentum", ctypes.c_float),
                ("lam", ctypes.c_float), ("alpha", ctypes.c_float)]


@dataclass
class Hyper:
    """Hyper-parameters of one completion, in the paper's symbols."""
    M: int
    H: int = 100
    tau: int = 1
    outer_lr: float = 0.7
    momentum: float = 0.9
    lam: float = 0.5
    alpha: float = 1.0
    comp_mode: int = COMP_TAYLOR
    sign_mode: int = SIGN_FORWARD

    def _c(self) -> _Hyper:
        return _Hyper(self.M, self.comp_mode, self.sign_mode, 0, self.H, self.tau,
                      self.outer_lr, self.momentum, self.lam, self.alpha)


def _load() -> ctypes.CDLL:
    path = _build.LIBRARY
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build the CUDA library first "
            "(python -m paper_2504_17672_b200.build, or __graft_entry__.build()); there is no fallback path")
    lib = ctypes.CDLL(path)
    vp, i32, i64, u32, f64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint32, ctypes.c_double
    lib.cocodc_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(_Partition), i32, i32]
    lib.cocodc_destroy.argtypes = [vp]
    lib.cocodc_sync_budget.argtypes = [i32, i64, f64, f64, f64, ctypes.POINTER(i64), ctypes.POINTER(i64)]
    lib.cocodc_fragment_scores.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.cocodc_scores_from_sumsq.argtypes = [vp, vp, vp, vp, vp, i64, i64, vp, vp, vp, vp]
    lib.cocodc_bind_in_flight.argtypes = [vp, vp]
    lib.cocodc_flush_scores.argtypes = [vp, vp]
    lib.cocodc_initiate.argtypes = [vp, vp, vp, vp, i64, i64, i32, i64, vp, vp, vp, vp, vp, vp, i64, i64, i32, vp]
    lib.cocodc_initiate_at.argtypes = [vp, vp, vp, vp, vp, i64, i32, i64, vp, vp, vp, vp, vp, vp, i64, i64, i32, vp]
    lib.cocodc_select_fragments.argtypes = [vp, vp, vp, vp, i64, i64, i32, i64, vp, vp, vp, vp, vp]
    lib.cocodc_outer_step.argtypes = [vp, ctypes.POINTER(_Hyper), vp, vp, i64, i64, vp, vp, vp, vp, vp, vp,
                                      i64, i64, vp, vp, vp, vp, u32, vp]
    lib.cocodc_outer_step_host.argtypes = [vp, ctypes.POINTER(_Hyper), vp, vp, i64, i64, vp, vp, vp, vp, vp, i32,
                                           i64, i64, vp, vp, vp, i32, vp, ctypes.c_uint64, vp]
    lib.cocodc_snapshot_host.argtypes = [vp, vp, vp, i64, i64, vp, i32, vp, i32, vp]
    lib.cocodc_merge.argtypes = [vp, ctypes.POINTER(_Hyper), vp, vp, i64, i64, vp, vp, vp, vp, vp]
    lib.cocodc_snapshot.argtypes = [vp, vp, vp, i64, i64, vp, i32, vp, vp, vp]
    lib.cocodc_fragment_scores_noalloc.argtypes = [ctypes.POINTER(_Partition), vp, vp, vp, vp, i32, vp]
    lib.cocodc_selftest_bounded_wait.argtypes = [vp, i32, vp]
    lib.cocodc_select_fragments_at.argtypes = [vp, vp, vp, vp, vp, i64, i32, i64, vp, vp, vp, vp, vp]
    lib.cocodc_outer_step_at.argtypes = [vp, ctypes.POINTER(_Hyper), vp, vp, i64, i64, vp, vp, vp, vp, vp, vp,
                                         vp, vp, vp, vp, vp, vp, u32, vp]
    lib.cocodc_pseudo_gradient_sum.argtypes = [vp, vp, i64, vp, vp, i32, vp, vp, vp, vp]
    lib.cocodc_outer_step_received.argtypes = [vp, ctypes.POINTER(_Hyper), i32, vp, vp, i64, i64, vp, vp, vp, vp,
                                               vp, vp, vp, i64, i64, vp, vp, vp, vp]
    lib.cocodc_outer_step_received_peers.argtypes = [vp, ctypes.POINTER(_Hyper), i32, vp, vp, i64, i64, vp, vp, vp,
                                                     ctypes.POINTER(vp), i32, vp, vp, vp, i64, i64, vp, vp, vp, vp]
    lib.cocodc_poll_status.argtypes = [vp, vp]
    lib.cocodc_launch_count.argtypes = [vp]
    lib.cocodc_launch_count.restype = i64
    lib.cocodc_status_string.argtypes = [ctypes.c_int]
    lib.cocodc_status_string.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("cocodc_launch_count", "cocodc_status_string"):
            getattr(lib, name).restype = ctypes.c_int
    return lib


_lib = _load()


def library() -> ctypes.CDLL:
    return _lib


def status_string(code: int) -> str:
    return _lib.cocodc_status_string(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != OK:
        raise CocodcError(code, where)


def _p(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def cocodc_sync_budget(K: int, H: int, gamma: float, Tc: float, Ts: float):
    """Eq. 8-9 on the host: returns (N, h)."""
    N, h = ctypes.c_int64(), ctypes.c_int64()
    _check(_lib.cocodc_sync_budget(K, H, gamma, Tc, Ts, ctypes.byref(N), ctypes.byref(h)), "cocodc_sync_budget")
    return N.value, h.value


def cocodc_fragment_scores_noalloc(N: int, frag_seg_ptr, seg_offset, seg_len, delta_g, interval, norms, scores,
                                   device: int = 0, stream=None) -> None:
    """Fragment norms and scores without a context and without any device allocation.

    For callers that may not allocate on the device (allocator hooks, pre-partitioned memory,
    allocation-free hot paths): the library's own fixed scratch array is used instead of context
    memory.  At most NOALLOC_MAX_K fragments / NOALLOC_MAX_SEGMENTS segments; calls that overlap on
    the GPU race on that array, so keep them on one stream.  The fragment table is host data."""
    ptr = np.ascontiguousarray(frag_seg_ptr, dtype=np.int32)
    off = np.ascontiguousarray(seg_offset, dtype=np.int64)
    ln = np.ascontiguousarray(seg_len, dtype=np.int64)
    part = _Partition(int(N), len(ptr) - 1, len(off),
                      ptr.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                      off.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)),
                      ln.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)))
    _check(_lib.cocodc_fragment_scores_noalloc(ctypes.byref(part), _p(delta_g), _p(interval), _p(norms), _p(scores),
                                               int(device), _stream(stream)), "cocodc_fragment_scores_noalloc")


class Context:
    """Owns a cocodc_ctx for one fragment partition on one device."""

    def __init__(self, N: int, frag_seg_ptr: Sequence[int], seg_offset: Sequence[int],
                 seg_len: Sequence[int], max_M: int, device: int = 0):
        self._h = ctypes.c_void_p()
        ptr = np.ascontiguousarray(frag_seg_ptr, dtype=np.int32)
        off = np.ascontiguousarray(seg_offset, dtype=np.int64)
        ln = np.ascontiguousarray(seg_len, dtype=np.int64)
        part = _Partition(int(N), len(ptr) - 1, len(off),
                          ptr.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                          off.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)),
                          ln.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)))
        self.N, self.K, self.device = int(N), len(ptr) - 1, int(device)
        _check(_lib.cocodc_create(ctypes.byref(self._h), ctypes.byref(part), int(max_M), int(device)), "cocodc_create")

    def close(self) -> None:
        if self._h:
            _lib.cocodc_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def launch_count(self) -> int:
        return int(_lib.cocodc_launch_count(self._h))

    def cocodc_fragment_scores(self, delta_g, interval, norms, scores, sumsq_out=None, stream=None) -> None:
        _check(_lib.cocodc_fragment_scores(self._h, _p(delta_g), _p(interval), _p(norms), _p(scores),
                                           _p(sumsq_out), _stream(stream)), "cocodc_fragment_scores")

    def cocodc_scores_from_sumsq(self, sumsq, ids, n_ids, interval, t_p: int, t_l: int, last_sync, norms, scores,
                                 stream=None) -> None:
        """Eq. 10 from fp64 sums of squares [K]: completion mode with an id list, stand-alone (all K) without."""
        _check(_lib.cocodc_scores_from_sumsq(self._h, _p(sumsq), _p(ids), _p(n_ids), _p(interval), int(t_p),
                                             int(t_l), _p(last_sync), _p(norms), _p(scores), _stream(stream)),
               "cocodc_scores_from_sumsq")

    def cocodc_bind_in_flight(self, in_flight) -> None:
        """Bind (or, with None, unbind) the caller's device uint8[K] mask of fragments in flight."""
        self._in_flight = in_flight          # keeps the tensor alive while the context points at it
        _check(_lib.cocodc_bind_in_flight(self._h, _p(in_flight)), "cocodc_bind_in_flight")

    def cocodc_flush_scores(self, stream=None) -> None:
        """Form the scores a completion launched with STAGE_DEFER left unformed (no-op when there is none)."""
        _check(_lib.cocodc_flush_scores(self._h, _stream(stream)), "cocodc_flush_scores")

    def cocodc_select_fragments(self, scores, last_sync, ineligible, t_now: int, H: int, budget_kind: int,
                                budget: int, mask, ids, n_sel, pool_offset=None, stream=None) -> None:
        _check(_lib.cocodc_select_fragments(self._h, _p(scores), _p(last_sync), _p(ineligible), int(t_now), int(H),
                                            int(budget_kind), int(budget), _p(mask), _p(ids), _p(n_sel),
                                            _p(pool_offset), _stream(stream)), "cocodc_select_fragments")

    def cocodc_initiate(self, scores, last_sync, ineligible, t_now: int, H: int, budget_kind: int, budget: int,
                        mask, ids, n_sel, pool_offset, w_now, w_snap, now_stride: int, snap_stride: int, M: int,
                        stream=None) -> None:
        """Algorithm 2 and the snapshot of what it picks, one launch (cocodc_select_fragments + cocodc_snapshot)."""
        _check(_lib.cocodc_initiate(self._h, _p(scores), _p(last_sync), _p(ineligible), int(t_now), int(H),
                                    int(budget_kind), int(budget), _p(mask), _p(ids), _p(n_sel), _p(pool_offset),
                                    _p(w_now), _p(w_snap), int(now_stride), int(snap_stride), int(M),
                                    _stream(stream)), "cocodc_initiate")

    def cocodc_initiate_at(self, scores, last_sync, ineligible, t_now, H: int, budget_kind: int, budget: int,
                           mask, ids, n_sel, pool_offset, w_now, w_snap, now_stride: int, snap_stride: int, M: int,
                           stream=None) -> None:
        """As cocodc_initiate with t_now a device int64[1] tensor."""
        _check(_lib.cocodc_initiate_at(self._h, _p(scores), _p(last_sync), _p(ineligible), _p(t_now), int(H),
                                       int(budget_kind), int(budget), _p(mask), _p(ids), _p(n_sel), _p(pool_offset),
                                       _p(w_now), _p(w_snap), int(now_stride), int(snap_stride), int(M),
                                       _stream(stream)), "cocodc_initiate_at")

    def cocodc_outer_step(self, hyper: Hyper, w_now, w_snap, now_stride: int, snap_stride: int, snap_offset,
                          theta_g, momentum, delta_g_out, ids, n_ids, t_p: int, t_l: int, last_sync,
                          norms, scores, stages: int = STAGE_ALL, stream=None, sumsq_out=None) -> None:
        h = hyper._c()
        _check(_lib.cocodc_outer_step(self._h, ctypes.byref(h), _p(w_now), _p(w_snap), int(now_stride),
                                      int(snap_stride), _p(snap_offset), _p(theta_g), _p(momentum),
                                      _p(delta_g_out), _p(ids), _p(n_ids), int(t_p), int(t_l), _p(last_sync),
                                      _p(norms), _p(scores), _p(sumsq_out), int(stages), _stream(stream)),
               "cocodc_outer_step")

    def cocodc_outer_step_host(self, hyper: Hyper, w_now, w_snap, now_stride: int, snap_stride: int, snap_offset,
                               theta_g, momentum, delta_g_out, ids, n_ids: int, t_p: int, t_l: int,
                               last_sync, norms, scores, workspace, snap_on_device: bool = False,
                               stream=None) -> None:
        """Host-buffer variant: every tensor is a CPU tensor, except `workspace` (CUDA) and, with
        snap_on_device, `w_snap` (CUDA)."""
        h = hyper._c()
        _check(_lib.cocodc_outer_step_host(self._h, ctypes.byref(h), _p(w_now), _p(w_snap), int(now_stride),
                                           int(snap_stride), _p(snap_offset), _p(theta_g), _p(momentum),
                                           _p(delta_g_out), _p(ids), int(n_ids), int(t_p), int(t_l),
                                           _p(last_sync), _p(norms), _p(scores), 1 if snap_on_device else 0, _p(workspace),
                                           workspace.numel() * workspace.element_size(), _stream(stream)),
               "cocodc_outer_step_host")

    def cocodc_select_fragments_at(self, scores, last_sync, ineligible, t_now, H: int, budget_kind: int,
                                   budget: int, mask, ids, n_sel, pool_offset=None, stream=None) -> None:
        """As cocodc_select_fragments with t_now a device int64[1] tensor."""
        _check(_lib.cocodc_select_fragments_at(self._h, _p(scores), _p(last_sync), _p(ineligible), _p(t_now), int(H),
                                               int(budget_kind), int(budget), _p(mask), _p(ids), _p(n_sel),
                                               _p(pool_offset), _stream(stream)), "cocodc_select_fragments_at")

    def cocodc_outer_step_at(self, hyper: Hyper, w_now, w_snap, now_stride: int, snap_stride: int, snap_offset,
                             theta_g, momentum, delta_g_out, ids, n_ids, t_p, t_l, last_sync,
                             norms, scores, stages: int = STAGE_ALL, stream=None, sumsq_out=None) -> None:
        """As cocodc_outer_step with t_p and t_l device int64[1] tensors."""
        h = hyper._c()
        _check(_lib.cocodc_outer_step_at(self._h, ctypes.byref(h), _p(w_now), _p(w_snap), int(now_stride),
                                         int(snap_stride), _p(snap_offset), _p(theta_g), _p(momentum),
                                         _p(delta_g_out), _p(ids), _p(n_ids), _p(t_p), _p(t_l), _p(last_sync),
                                         _p(norms), _p(scores), _p(sumsq_out), int(stages), _stream(stream)),
               "cocodc_outer_step_at")

    def cocodc_pseudo_gradient_sum(self, w_snap, snap_stride: int, snap_offset, theta_g, M: int, sum_out,
                                   ids, n_ids, stream=None) -> None:
        _check(_lib.cocodc_pseudo_gradient_sum(self._h, _p(w_snap), int(snap_stride), _p(snap_offset), _p(theta_g),
                                               int(M), _p(sum_out), _p(ids), _p(n_ids), _stream(stream)),
               "cocodc_pseudo_gradient_sum")

    def cocodc_outer_step_received(self, hyper: Hyper, M_total: int, w_now, w_snap, now_stride: int,
                                   snap_stride: int, snap_offset, theta_g, momentum, delta_sum, delta_g_out,
                                   ids, n_ids, t_p: int, t_l: int, last_sync, norms, scores, stream=None) -> None:
        h = hyper._c()
        _check(_lib.cocodc_outer_step_received(self._h, ctypes.byref(h), int(M_total), _p(w_now), _p(w_snap),
                                               int(now_stride), int(snap_stride), _p(snap_offset), _p(theta_g),
                                               _p(momentum), _p(delta_sum), _p(delta_g_out), _p(ids), _p(n_ids),
                                               int(t_p), int(t_l), _p(last_sync), _p(norms), _p(scores),
                                               _stream(stream)), "cocodc_outer_step_received")

    def cocodc_outer_step_received_peers(self, hyper: Hyper, M_total: int, w_now, w_snap, now_stride: int,
                                         snap_stride: int, snap_offset, theta_g, momentum, delta_sums, delta_g_out,
                                         ids, n_ids, t_p: int, t_l: int, last_sync, norms, scores,
                                         stream=None) -> None:
        """delta_sums: sequence of device tensors (or integer device addresses, e.g. of peer-mapped buffers)."""
        h = hyper._c()
        addrs = [int(x) if isinstance(x, int) else x.data_ptr() for x in delta_sums]
        arr = (ctypes.c_void_p * len(addrs))(*addrs)
        _check(_lib.cocodc_outer_step_received_peers(self._h, ctypes.byref(h), int(M_total), _p(w_now), _p(w_snap),
                                                     int(now_stride), int(snap_stride), _p(snap_offset), _p(theta_g),
                                                     _p(momentum), arr, len(addrs), _p(delta_g_out), _p(ids),
                                                     _p(n_ids), int(t_p), int(t_l), _p(last_sync), _p(norms),
                                                     _p(scores), _stream(stream)), "cocodc_outer_step_received_peers")

    def cocodc_merge(self, hyper: Hyper, w_now, w_snap, now_stride: int, snap_stride: int, snap_offset,
                     theta_g_new, ids, n_ids, stream=None) -> None:
        h = hyper._c()
        _check(_lib.cocodc_merge(self._h, ctypes.byref(h), _p(w_now), _p(w_snap), int(now_stride), int(snap_stride),
                                 _p(snap_offset), _p(theta_g_new), _p(ids), _p(n_ids), _stream(stream)),
               "cocodc_merge")

    def cocodc_snapshot(self, w_now, w_snap, now_stride: int, snap_stride: int, snap_offset, M: int,
                        ids, n_ids, stream=None) -> None:
        _check(_lib.cocodc_snapshot(self._h, _p(w_now), _p(w_snap), int(now_stride), int(snap_stride),
                                    _p(snap_offset), int(M), _p(ids), _p(n_ids), _stream(stream)),
               "cocodc_snapshot")

    def cocodc_snapshot_host(self, w_now, w_snap, now_stride: int, snap_stride: int, snap_offset, M: int,
                             ids, n_ids: int, stream=None) -> None:
        """S0 from a host w_now into a device w_snap; ids and snap_offset are CPU tensors."""
        _check(_lib.cocodc_snapshot_host(self._h, _p(w_now), _p(w_snap), int(now_stride), int(snap_stride),
                                         _p(snap_offset), int(M), _p(ids), int(n_ids), _stream(stream)),
               "cocodc_snapshot_host")

    def cocodc_selftest_bounded_wait(self, polls: int, stream=None) -> None:
        """Runs a bounded wait that must run out; the status word then reads ERR_TIMEOUT."""
        _check(_lib.cocodc_selftest_bounded_wait(self._h, int(polls), _stream(stream)), "cocodc_selftest_bounded_wait")

    def cocodc_poll_status(self, stream=None) -> int:
        """Waits for the stream; returns and clears the device status word."""
        return int(_lib.cocodc_poll_status(self._h, _stream(stream)))
