"""Seeded random buffers for a workload.

Recipe (per fragment p with drift scale s_p, per worker m):

    theta_g[p]    ~ N(0, sigma_global)                       global state of the last sync
    w_snap[m][p]  = theta_g[p] + s_p * z_m,  z_m ~ N(0, 1)   local parameters when the sync started
    w_now[m][p]   = w_snap[m][p] + (s_p / sigma_drift) * (e + 0.1 * eps_m)
                    e ~ N(0, sigma_drift) shared by all workers (common movement over the delay),
                    eps_m ~ N(0, sigma_drift) per worker
    momentum      = 0, or N(0, momentum_sigma) when asked for

Random numbers come from torch generators seeded per (workload seed, buffer,
fragment, worker), so a fragment's values do not depend on which other
fragments are generated or on the layout of the snapshot buffer.  The values
are generated once, on the device asked for; whoever needs them elsewhere
copies the bits.
"""

from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional, Sequence

import numpy as np
import torch

from .configs import Workload

_BUF_GLOBAL, _BUF_SNAP, _BUF_SHARED, _BUF_WORKER, _BUF_MOM, _BUF_GAP = range(6)


def _seed(seed: int, buf: int, p: int, m: int) -> int:
    x = (seed * 0x9E3779B97F4A7C15 + buf * 0xBF58476D1CE4E5B9 + p * 0x94D049BB133111EB
         + m * 0xD6E8FEB86659FD93 + 0x2545F4914F6CDD1D) & 0xFFFFFFFFFFFFFFFF
    x ^= x >> 31
    x = (x * 0x7FB5D329728EA185) & 0xFFFFFFFFFFFFFFFF
    x ^= x >> 27
    return x & 0x7FFFFFFFFFFFFFFF


def _randn(n: int, device, seed: int) -> torch.Tensor:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return torch.randn(n, generator=g, device=device, dtype=torch.float32)


def fragment_scales(w: Workload) -> np.ndarray:
    """Per-fragment drift scale s_p (float64[K]), drawn on the host from the workload seed."""
    rng = np.random.default_rng(w.seed)
    K = w.K
    if w.scale_kind == "const":
        return np.full(K, w.sigma_drift, dtype=np.float64)
    if w.scale_kind == "loguniform":
        return np.exp(rng.uniform(np.log(1e-4), np.log(1e-2), size=K))
    if w.scale_kind == "student_t":
        z = rng.standard_normal(K)
        chi2 = rng.chisquare(3, size=K)
        t3 = z / np.sqrt(chi2 / 3.0)
        return np.clip(w.sigma_drift * np.abs(t3), 1e-6, 1.0)
    raise ValueError(w.scale_kind)


@dataclass
class DeviceBuffers:
    theta_g: torch.Tensor            # [N]
    momentum: torch.Tensor           # [N]
    w_now: torch.Tensor              # [M, N]
    w_snap: torch.Tensor             # [M, N] (full layout) or [M, pool_len] (pool layout)
    snap_offset: Optional[torch.Tensor]  # int64[K] element offset of each fragment in a w_snap row; None = same layout as w_now
    scales: np.ndarray               # float64[K]

    @property
    def now_stride(self) -> int:
        return self.w_now.stride(0)

    @property
    def snap_stride(self) -> int:
        return self.w_snap.stride(0)


def _scatter(dst_row: torch.Tensor, segments, vec: torch.Tensor) -> None:
    pos = 0
    for off, ln in segments:
        dst_row[off:off + ln] = vec[pos:pos + ln]
        pos += ln


def generate(w: Workload, device="cpu", *, snap_layout: str = "full",
             pool_ids: Optional[Sequence[int]] = None, pool_len: Optional[int] = None,
             pool_offsets: Optional[Dict[int, int]] = None,
             momentum_sigma: float = 0.0, worker_offset: int = 0, shard: int = 0) -> DeviceBuffers:
    """Fill the buffers of one workload.

    snap_layout="full": w_snap is [M, N] laid out like w_now.
    snap_layout="pool": w_snap is [M, pool_len]; only fragments in `pool_ids`
    get a snapshot, packed back to back (segments of a fragment concatenated)
    in the order given, each start rounded up to a multiple of 4 elements
    unless `pool_offsets` places them explicitly.
    worker_offset: the M workers generated here are workers worker_offset .. worker_offset + M - 1 of a larger
    job (the workers of one device when they are spread over several); the global state does not depend on it.
    shard: which element range of a larger model this is (a model split over several devices by parameter range):
    another shard has the same fragment table and drift scales but its own random values.
    """
    device = torch.device(device)
    part = w.partition
    N, M, K = w.N, w.M, w.K
    scales = fragment_scales(w)
    vseed = w.seed + 1_000_003 * shard          # seed of the value streams; the scales keep the workload's own

    theta_g = torch.empty(N, dtype=torch.float32, device=device)
    momentum = torch.zeros(N, dtype=torch.float32, device=device)
    w_now = torch.empty((M, N), dtype=torch.float32, device=device)
    covered = sum(part.frag_size(p) for p in range(K))
    if covered != N:  # gaps between fragments (test workloads only): fill the background first
        theta_g.copy_(_randn(N, device, _seed(vseed, _BUF_GAP, 0, 0)) * w.sigma_global)
        for m in range(M):
            w_now[m].copy_(theta_g + _randn(N, device, _seed(vseed, _BUF_GAP, 1, m)) * w.sigma_drift)

    snap_offset = None
    if snap_layout == "full":
        w_snap = torch.empty((M, N), dtype=torch.float32, device=device)
        if covered != N:
            w_snap.copy_(w_now)
        in_pool = set(range(K))
    elif snap_layout == "pool":
        ids = list(pool_ids if pool_ids is not None else range(K))
        offs = np.full(K, -1, dtype=np.int64)
        pos = 0
        for p in ids:
            if pool_offsets is not None and p in pool_offsets:
                pos = int(pool_offsets[p])
            else:
                pos = (pos + 3) // 4 * 4
            offs[p] = pos
            pos += part.frag_size(p)
        plen = int(pool_len) if pool_len is not None else (pos + 3) // 4 * 4
        assert plen >= pos
        w_snap = torch.zeros((M, max(plen, 4)), dtype=torch.float32, device=device)
        snap_offset = torch.from_numpy(offs).to(device)
        in_pool = set(ids)
    else:
        raise ValueError(snap_layout)

    for p in range(K):
        segs = part.fragments[p]
        n = part.frag_size(p)
        s = float(scales[p])
        tg = _randn(n, device, _seed(vseed, _BUF_GLOBAL, p, 0)).mul_(w.sigma_global)
        _scatter(theta_g, segs, tg)
        if momentum_sigma > 0.0:
            _scatter(momentum, segs, _randn(n, device, _seed(vseed, _BUF_MOM, p, 0)).mul_(momentum_sigma))
        e = _randn(n, device, _seed(vseed, _BUF_SHARED, p, 0)).mul_(w.sigma_drift)
        for m in range(M):
            snap = _randn(n, device, _seed(vseed, _BUF_SNAP, p, m + worker_offset)).mul_(s).add_(tg)
            if p in in_pool:
                if snap_offset is None:
                    _scatter(w_snap[m], segs, snap)
                else:
                    o = int(snap_offset[p])
                    w_snap[m, o:o + n] = snap
            eps = _randn(n, device, _seed(vseed, _BUF_WORKER, p, m + worker_offset)).mul_(0.1 * w.sigma_drift)
            eps.add_(e).mul_(s / w.sigma_drift).add_(snap)
            _scatter(w_now[m], segs, eps)
            del snap, eps
        del tg, e
    return DeviceBuffers(theta_g=theta_g, momentum=momentum, w_now=w_now, w_snap=w_snap,
                         snap_offset=snap_offset, scales=scales)
