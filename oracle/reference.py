"""CPU oracle for CoCoDC's per-fragment outer synchronisation step.

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's
CPU-baseline leg may call this; the product never does, and this module
imports nothing of the CUDA library.

The element-wise arithmetic (Eq. 1-7, Algorithm 1) lives in cocodc_oracle.c,
in double precision on the fp32 input bits.  This module adds what is small
and integer-valued: walking a fragment's segments, Eq. 10's score, Algorithm
2's selection extended to a budget, and Eq. 8-9's schedule sizing.

Parity pins (tests/test_oracle_pins.py): closed forms and worked values for
every function here.  Unpinned by the paper itself: which of the three sign
readings of Eq. 4/Eq. 7 the authors ran, and the outer optimizer's exact
formula and settings (the paper names SGD with Nesterov momentum only as an example of OuterOptim);
the Nesterov reading is pinned to the torch CPU optimizer of that name.
"""

from __future__ import annotations

import ctypes
import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from . import build as _build

COMP_NONE, COMP_TAYLOR = 0, 1
SIGN_FORWARD, SIGN_PRINTED, SIGN_DESCENT = 0, 1, 2
BUDGET_COUNT, BUDGET_PARAMS, BUDGET_PARAMS_EXACT = 0, 1, 2

_lib = None


def load_library(path: str):
    """Load a build of cocodc_oracle.c and declare its signatures (tests also load deliberately broken builds)."""
    lib = ctypes.CDLL(path)
    _declare(lib)
    return lib


def _declare(lib):
    d, l, i, p = ctypes.c_double, ctypes.c_long, ctypes.c_int, ctypes.c_void_p
    lib.cocodc_oracle_outer_elements.restype = d
    lib.cocodc_oracle_outer_elements.argtypes = [
        l, i, p, l, p, l, p, p, d, d, d, d, l, l, i, i, i, p, i, i, p, p, p, p]
    lib.cocodc_oracle_pseudo_gradient_sum.restype = None
    lib.cocodc_oracle_pseudo_gradient_sum.argtypes = [l, i, p, l, p, p]
    lib.cocodc_oracle_merge_elements.restype = None
    lib.cocodc_oracle_merge_elements.argtypes = [l, i, p, l, p, l, p, d, d, l, l, i, i, p]
    lib.cocodc_oracle_sumsq.restype = d
    lib.cocodc_oracle_sumsq.argtypes = [l, p]


def _clib():
    global _lib
    if _lib is None:
        _lib = load_library(_build.build())
    return _lib


@dataclass
class Hyper:
    """Hyper-parameters of one outer step, in the paper's symbols."""
    M: int
    H: int = 100
    tau: int = 1
    outer_lr: float = 0.7      # eta
    momentum: float = 0.9      # mu
    lam: float = 0.5           # lambda
    alpha: float = 1.0
    comp_mode: int = COMP_TAYLOR
    sign_mode: int = SIGN_FORWARD


Fragments = Sequence[Sequence[Tuple[int, int]]]


def _f32(x) -> np.ndarray:
    x = np.asarray(x)
    assert x.dtype == np.float32, x.dtype
    return x


def _ptr(x: np.ndarray, elem_offset: int = 0) -> int:
    return x.ctypes.data + elem_offset * x.itemsize


# --------------------------------------------------------------------------
# Eq. 8-9: schedule sizing
# --------------------------------------------------------------------------

def sync_budget(K: int, H: int, gamma: float, Tc: float, Ts: float) -> Tuple[int, int]:
    """N = max(K, floor(gamma*H*Tc/Ts)) (Eq. 8) and h = floor(H/N), at least 1 (Eq. 9)."""
    if K <= 0 or H <= 0 or not (0.0 < gamma <= 1.0) or Tc <= 0 or Ts <= 0:
        raise ValueError("bad schedule arguments")
    N = max(K, int(math.floor(gamma * H * Tc / Ts)))
    h = max(1, H // N)
    return N, h


# --------------------------------------------------------------------------
# Eq. 10: per-fragment score
# --------------------------------------------------------------------------

def fragment_sumsq(fragments: Fragments, x: np.ndarray) -> np.ndarray:
    x = _f32(x)
    lib = _clib()
    out = np.zeros(len(fragments), dtype=np.float64)
    for p, segs in enumerate(fragments):
        s = 0.0
        for off, ln in segs:
            s += lib.cocodc_oracle_sumsq(ln, _ptr(x, off))
        out[p] = s
    return out


def fragment_scores(fragments: Fragments, delta_g: np.ndarray,
                    interval: Optional[Sequence[int]] = None):
    """norms[p] = ||delta_g restricted to fragment p||_2 and R_p = norm / max(1, I_p) (Eq. 10)."""
    norms = np.sqrt(fragment_sumsq(fragments, delta_g))
    K = len(fragments)
    I = np.ones(K, dtype=np.int64) if interval is None else np.maximum(1, np.asarray(interval, dtype=np.int64))
    return norms, norms / I.astype(np.float64)


# --------------------------------------------------------------------------
# Algorithm 2 / Eq. 11 under a budget
# --------------------------------------------------------------------------

def select_fragments(scores: Sequence[float], last_sync: Sequence[int], sizes: Sequence[int],
                     t_now: int, H: int, budget_kind: int, budget: int,
                     ineligible: Optional[Sequence[int]] = None):
    """Priority order, then a greedy walk under the budget.

    Order: eligible fragments that have gone H or more steps since their last
    completed sync, by ascending index (Algorithm 2 returns the first such
    fragment); then the other eligible fragments by score, largest first, ties
    to the lower index (Eq. 11; +inf marks never-synced fragments).  The head
    of the order is always taken (Algorithm 2 always returns a fragment); each
    later fragment is taken iff its cost (1, or its size) still fits.

    BUDGET_PARAMS_EXACT is an option outside the paper (its Algorithm 2 returns one fragment per decision):
    the walk stops at the first fragment that is neither overdue nor never-synced (score +inf); the fragments
    from there on are a knapsack, solved by trying every subset -- largest sum of scores (added in priority
    order) among those whose sizes fit the rest of the budget, equal sums to the subset tried first when
    subsets are numbered with the first fragment of the order as the lowest bit.  If nothing at all was taken,
    the first fragment of the order is.
    Returns (mask uint8[K], ids int32[n_sel] in admission order, n_sel).
    """
    K = len(scores)
    R = [float(s) for s in scores]
    if any(math.isnan(r) for r in R):
        raise ValueError("NaN score")
    if budget < 0 or budget_kind not in (BUDGET_COUNT, BUDGET_PARAMS, BUDGET_PARAMS_EXACT):
        raise ValueError("bad budget")
    elig = [p for p in range(K) if ineligible is None or not ineligible[p]]
    overdue = [p for p in elig if int(t_now) - int(last_sync[p]) >= H]
    rest = [p for p in elig if p not in overdue]
    rest.sort(key=lambda p: (-R[p], p))
    order = overdue + rest
    mask = np.zeros(K, dtype=np.uint8)
    ids: List[int] = []
    remaining = int(budget)
    free: List[int] = []
    for j, p in enumerate(order):
        if budget_kind == BUDGET_PARAMS_EXACT and p not in overdue and R[p] != math.inf:
            free = order[j:]
            break
        cost = 1 if budget_kind == BUDGET_COUNT else int(sizes[p])
        if j == 0 or cost <= remaining:
            mask[p] = 1
            ids.append(p)
            remaining -= cost
    if free:
        best_value, best_subset = None, 0
        for subset in range(1 << len(free)):
            members = [p for j, p in enumerate(free) if (subset >> j) & 1]
            if sum(int(sizes[p]) for p in members) > remaining:
                continue
            value = 0.0
            for p in members:
                value += R[p]
            if best_value is None or value > best_value:
                best_value, best_subset = value, subset
        if best_subset == 0 and not ids:
            best_subset = 1
        for j, p in enumerate(free):
            if (best_subset >> j) & 1:
                mask[p] = 1
                ids.append(p)
    return mask, np.asarray(ids, dtype=np.int32), len(ids)


# --------------------------------------------------------------------------
# Eq. 1-7: the outer step on the processed fragments
# --------------------------------------------------------------------------

@dataclass
class FragmentResult:
    """Double-precision outputs for one processed fragment, segments concatenated."""
    w_now: Optional[np.ndarray]   # [M, n_p] merged local parameters (None if the merge was not asked for)
    theta_g: np.ndarray           # [n_p] new global state G
    momentum: np.ndarray          # [n_p] new momentum u'
    delta_g: np.ndarray           # [n_p] mean pseudo-gradient
    sumsq: float
    norm: float
    score: float


def _snap_base(snap_offset, p: int, native_off: int, pos_in_frag: int) -> int:
    """Element offset of a segment inside one worker's row of w_snap."""
    if snap_offset is None:
        return native_off
    return int(snap_offset[p]) + pos_in_frag


def outer_step(fragments: Fragments, hp: Hyper, w_now: np.ndarray, w_snap: np.ndarray,
               theta_g: np.ndarray, momentum: np.ndarray, ids: Sequence[int],
               t_p: int, t_l: int, last_sync: Sequence[int],
               snap_offset: Optional[Sequence[int]] = None, do_merge: bool = True,
               threads: int = 1, recv_sum: Optional[np.ndarray] = None, M_total: Optional[int] = None):
    """Run Eq. 1-2, Algorithm 1 / Eq. 3 and Eq. 10 on the fragments in `ids`.

    w_now, w_snap: float32 [M, .]; theta_g, momentum: float32 [N].  w_snap is
    laid out like w_now unless snap_offset[p] gives fragment p's start inside a
    packed row.  Inputs are not modified.
    recv_sum and M_total: the worker-per-device deployment of Section 2.1 - the sum of all M_total workers'
    pseudo-gradients is given, either all-reduced already (float32 [N]) or as the contributing devices' partial
    sums (a sequence of float32 [N] arrays, added up here), and the M local workers are only merged.
    Returns (results {p: FragmentResult}, new last_sync int64[K]).
    """
    recv_list = []
    if recv_sum is not None:
        recv_list = [_f32(recv_sum)] if isinstance(recv_sum, np.ndarray) and recv_sum.ndim == 1 \
            else [_f32(x) for x in recv_sum]
        if not M_total or M_total < 1:
            raise ValueError("M_total must accompany recv_sum")
    lib = _clib()
    w_now, w_snap, theta_g, momentum = _f32(w_now), _f32(w_snap), _f32(theta_g), _f32(momentum)
    M = hp.M
    assert w_now.shape[0] == M and w_snap.shape[0] == M
    assert w_now.strides[1] == 4 and w_snap.strides[1] == 4
    now_stride, snap_stride = w_now.strides[0] // 4, w_snap.strides[0] // 4
    if hp.tau < 0 or hp.H <= 0 or M <= 0:
        raise ValueError("bad hyper-parameters")
    ids = [int(p) for p in ids]
    if len(set(ids)) != len(ids) or any(p < 0 or p >= len(fragments) for p in ids):
        raise ValueError("bad fragment ids")
    new_last = np.asarray(last_sync, dtype=np.int64).copy()
    results: Dict[int, FragmentResult] = {}
    for p in ids:
        segs = fragments[p]
        n_p = sum(l for _, l in segs)
        out_now = np.empty((M, n_p), dtype=np.float64) if do_merge else None
        out_g = np.empty(n_p, dtype=np.float64)
        out_u = np.empty(n_p, dtype=np.float64)
        out_d = np.empty(n_p, dtype=np.float64)
        sumsq = 0.0
        pos = 0
        for off, ln in segs:
            sb = _snap_base(snap_offset, p, off, pos)
            # the C routine writes worker m's outputs at now_out[m*n + i]; hand it a
            # contiguous [M, ln] block per piece and copy it into place
            pieces = [(0, ln)] if threads <= 1 else _split(ln, threads)

            def run(piece):
                lo, cnt = piece
                blk = np.empty((M, cnt), dtype=np.float64) if do_merge else None
                s = lib.cocodc_oracle_outer_elements(
                    cnt, M, _ptr(w_snap, sb + lo), snap_stride, _ptr(w_now, off + lo), now_stride,
                    _ptr(theta_g, off + lo), _ptr(momentum, off + lo),
                    hp.outer_lr, hp.momentum, hp.lam, hp.alpha, hp.tau, hp.H,
                    hp.comp_mode, hp.sign_mode, 1 if do_merge else 0,
                    (ctypes.c_void_p * max(1, len(recv_list)))(*[_ptr(x, off + lo) for x in recv_list]),
                    len(recv_list), int(M_total or 0),
                    blk.ctypes.data if do_merge else None,
                    _ptr(out_g, pos + lo), _ptr(out_u, pos + lo), _ptr(out_d, pos + lo))
                if do_merge:
                    out_now[:, pos + lo:pos + lo + cnt] = blk
                return s

            if threads <= 1:
                partial = [run(pc) for pc in pieces]
            else:
                with ThreadPoolExecutor(max_workers=threads) as ex:
                    partial = list(ex.map(run, pieces))
            for s in partial:
                sumsq += s
            pos += ln
        norm = math.sqrt(sumsq)
        interval = max(1, int(t_p) - int(last_sync[p]))          # I_p of Eq. 10
        results[p] = FragmentResult(out_now, out_g, out_u, out_d, sumsq, norm, norm / interval)
        new_last[p] = int(t_l)
    return results, new_last


def pseudo_gradient_sum(fragments: Fragments, M: int, w_snap: np.ndarray, theta_g: np.ndarray, ids: Sequence[int],
                        snap_offset: Optional[Sequence[int]] = None) -> Dict[int, np.ndarray]:
    """Per listed fragment, the sum over the M local workers of theta^m_{p,t_p} - theta^g (what one device
    hands to the all-reduce of Section 2.1), float64 [n_p], segments concatenated."""
    lib = _clib()
    w_snap, theta_g = _f32(w_snap), _f32(theta_g)
    snap_stride = w_snap.strides[0] // 4
    out: Dict[int, np.ndarray] = {}
    for p in [int(q) for q in ids]:
        n_p = sum(l for _, l in fragments[p])
        res = np.empty(n_p, dtype=np.float64)
        pos = 0
        for off, ln in fragments[p]:
            sb = _snap_base(snap_offset, p, off, pos)
            lib.cocodc_oracle_pseudo_gradient_sum(ln, M, _ptr(w_snap, sb), snap_stride, _ptr(theta_g, off),
                                                  _ptr(res, pos))
            pos += ln
        out[p] = res
    return out


def _split(n: int, parts: int):
    parts = max(1, min(parts, n))
    step = -(-n // parts)
    return [(lo, min(step, n - lo)) for lo in range(0, n, step)]


def merge(fragments: Fragments, hp: Hyper, w_now: np.ndarray, w_snap: np.ndarray,
          theta_g_new: np.ndarray, ids: Sequence[int],
          snap_offset: Optional[Sequence[int]] = None) -> Dict[int, np.ndarray]:
    """Algorithm 1 (or Eq. 3) alone: merged local parameters {p: float64 [M, n_p]}."""
    lib = _clib()
    w_now, w_snap, theta_g_new = _f32(w_now), _f32(w_snap), _f32(theta_g_new)
    M = hp.M
    now_stride, snap_stride = w_now.strides[0] // 4, w_snap.strides[0] // 4
    out: Dict[int, np.ndarray] = {}
    for p in [int(q) for q in ids]:
        segs = fragments[p]
        n_p = sum(l for _, l in segs)
        res = np.empty((M, n_p), dtype=np.float64)
        pos = 0
        for off, ln in segs:
            sb = _snap_base(snap_offset, p, off, pos)
            blk = np.empty((M, ln), dtype=np.float64)
            lib.cocodc_oracle_merge_elements(
                ln, M, _ptr(w_snap, sb), snap_stride, _ptr(w_now, off), now_stride,
                _ptr(theta_g_new, off), hp.lam, hp.alpha, hp.tau, hp.H, hp.comp_mode, hp.sign_mode,
                blk.ctypes.data)
            res[:, pos:pos + ln] = blk
            pos += ln
        out[p] = res
    return out


def snapshot(fragments: Fragments, w_now: np.ndarray, ids: Sequence[int], M: int,
             snap_offset: Optional[Sequence[int]], w_snap: np.ndarray) -> np.ndarray:
    """Record theta^m_{p,t_p} (Algorithm 1's input): copy the fragments in `ids` into w_snap."""
    out = np.array(w_snap, copy=True)
    for p in [int(q) for q in ids]:
        pos = 0
        for off, ln in fragments[p]:
            sb = _snap_base(snap_offset, p, off, pos)
            out[:M, sb:sb + ln] = w_now[:M, off:off + ln]
            pos += ln
    return out


def gather_fragment(fragments: Fragments, x: np.ndarray, p: int) -> np.ndarray:
    """Concatenate fragment p's segments out of a flat (or [M, N]) array."""
    return np.concatenate([x[..., off:off + ln] for off, ln in fragments[p]], axis=-1)
