"""Fragment schedule of CoCoDC around the C-ABI calls (Section 2.1 time line, Section 3.2 schedule).

`RoundDriver.after_local_step(t)` is called once per local training step t = 1, 2, ...:

  * every synchronisation initiated at t - tau completes now: `cocodc_outer_step` on its fragment list
    (Eq. 1-2, Algorithm 1, Eq. 10);
  * every h steps (Eq. 8-9) a new synchronisation is initiated: `cocodc_initiate` = Algorithm 2 (fragments
    still in flight are ineligible) and the snapshot of the chosen fragments, one launch.

All schedule state (scores, last_sync, id lists, masks, pool offsets, the in-flight mask) lives on the device
and is updated by the library's kernels; the driver only marshals arguments and keeps track of which slot was
initiated when.  Several synchronisations can
be in flight at once (tau > h); each has its own slot: id list, mask and snapshot pool.
"""

from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import torch

from . import binding as B


@dataclass
class _Slot:
    ids: torch.Tensor
    n_ids: torch.Tensor
    mask: torch.Tensor
    pool_off: torch.Tensor
    pool: torch.Tensor
    t_p: int = -1          # step of initiation; -1 = free


class RoundDriver:
    def __init__(self, ctx: "B.Context", hyper: "B.Hyper", w_now: torch.Tensor, theta_g: torch.Tensor,
                 momentum: torch.Tensor, frag_sizes, *, gamma: float, Tc: float, Ts: float,
                 budget_kind: int = B.BUDGET_COUNT, budget: int = 1, pool_len: Optional[int] = None):
        self.ctx, self.hyper = ctx, hyper
        self.w_now, self.theta_g, self.momentum = w_now, theta_g, momentum
        dev = w_now.device
        K = ctx.K
        self.K = K
        self.budget_kind, self.budget = budget_kind, budget
        # Eq. 8-9: syncs per H local steps and the interval between initiations
        self.N_sync, self.h = B.cocodc_sync_budget(K, hyper.H, gamma, Tc, Ts)
        sizes = sorted((int(s) for s in frag_sizes), reverse=True)
        if pool_len is None:
            cap = (budget + sizes[0]) if budget_kind == B.BUDGET_PARAMS else sum(sizes[:max(1, budget)])
            pool_len = (cap + 8 * K + 1023) // 1024 * 1024
        n_slots = max(1, -(-hyper.tau // self.h)) + 1
        self.slots: List[_Slot] = [
            _Slot(ids=torch.full((K,), -1, dtype=torch.int32, device=dev),
                  n_ids=torch.zeros(1, dtype=torch.int32, device=dev),
                  mask=torch.zeros(K, dtype=torch.uint8, device=dev),
                  pool_off=torch.full((K,), -1, dtype=torch.int64, device=dev),
                  pool=torch.zeros((hyper.M, pool_len), dtype=torch.float32, device=dev))
            for _ in range(n_slots)]
        self.scores = torch.full((K,), float("inf"), dtype=torch.float32, device=dev)   # never synced: +inf
        self.norms = torch.zeros(K, dtype=torch.float32, device=dev)
        self.last_sync = torch.zeros(K, dtype=torch.int64, device=dev)
        # Algorithm 2's in-flight bookkeeping: the selection kernel marks what it admits, the completion clears it
        self.in_flight = torch.zeros(K, dtype=torch.uint8, device=dev)
        ctx.cocodc_bind_in_flight(self.in_flight)
        self.initiated = 0
        self.completed = 0
        # optional callable(kind, phase, slot, t) with kind in {"complete", "initiate"} and phase in
        # {"before", "after"}; lets a caller inspect the state around each event
        self.observer = None

    def _notify(self, kind: str, phase: str, slot: _Slot, t: int) -> None:
        if self.observer is not None:
            self.observer(kind, phase, slot, t)

    # -- the two events of a fragment's synchronisation ------------------------------------------

    def _complete(self, slot: _Slot, t_l: int) -> None:
        self._notify("complete", "before", slot, t_l)
        self.ctx.cocodc_outer_step(self.hyper, self.w_now, slot.pool, self.w_now.stride(0), slot.pool.stride(0),
                                   slot.pool_off, self.theta_g, self.momentum, None, slot.ids, slot.n_ids,
                                   slot.t_p, t_l, self.last_sync, self.norms, self.scores)
        self._notify("complete", "after", slot, t_l)
        slot.t_p = -1
        self.completed += 1

    def _initiate(self, slot: _Slot, t_p: int) -> None:
        self._notify("initiate", "before", slot, t_p)
        self.ctx.cocodc_initiate(self.scores, self.last_sync, None, t_p, self.hyper.H, self.budget_kind, self.budget,
                                 slot.mask, slot.ids, slot.n_ids, slot.pool_off, self.w_now, slot.pool,
                                 self.w_now.stride(0), slot.pool.stride(0), self.hyper.M)
        slot.t_p = t_p
        self.initiated += 1
        self._notify("initiate", "after", slot, t_p)

    # -- one local step --------------------------------------------------------------------------

    def after_local_step(self, t: int) -> None:
        for slot in self.slots:
            if slot.t_p >= 0 and t - slot.t_p >= self.hyper.tau:
                self._complete(slot, t)
        if t % self.h == 0:
            free = next((s for s in self.slots if s.t_p < 0), None)
            if free is not None:
                self._initiate(free, t)
