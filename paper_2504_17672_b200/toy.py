"""Toy convergence driver: M workers descend their own quadratic objectives with plain SGD and are kept
together by the outer synchronisation step under a delay of tau local steps.

It stands in for the paper's experiment (Section 4), which needs a dataset and a 150 M-parameter model:
here the effect of the compensation strength lambda, of the overlap depth tau and of the method variant can
be looked at in seconds.  Worker m minimises f_m(w) = 1/2 sum_i a_i (w_i - c_{m,i})^2 with non-identical
optima c_m = c* + spread * z_m (non-IID data, Section 2.1); the global objective is their mean, whose
optimum is the mean of the c_m.  The inner steps are ordinary torch operations (they are not part of the
library's path); every synchronisation goes through the C-ABI calls via schedule.RoundDriver.

    python -m paper_2504_17672_b200.toy            # prints the final global loss for a few settings
"""

from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple

import torch

from . import binding as B
from .schedule import RoundDriver


@dataclass
class ToyResult:
    variant: str
    lam: float
    tau: int
    losses: List[Tuple[int, float]]      # (local step, global objective at the mean of the workers)
    syncs: int

    @property
    def final(self) -> float:
        return self.losses[-1][1]


def run_toy(variant: str = "cocodc", *, M: int = 4, K: int = 4, frag: int = 4096, H: int = 20, tau: int = 4,
            lam: float = 0.5, steps: int = 400, inner_lr: float = 0.05, grad_noise: float = 0.02,
            spread: float = 0.5, gamma: float = 0.4, Tc: float = 1.0, Ts: float = 1.0, seed: int = 0,
            device: str = "cuda", log_every: int = 20) -> ToyResult:
    """variant: "cocodc" (delay compensation), "streaming_diloco" (Eq. 3 blend, alpha = 0.5) or "diloco"
    (one fragment, blocking sync every H steps)."""
    dev = torch.device(device)
    g = torch.Generator(device=dev).manual_seed(seed)
    N = K * frag
    a = 0.5 + torch.rand(N, generator=g, device=dev)                       # curvatures in [0.5, 1.5]
    c_star = torch.randn(N, generator=g, device=dev)
    c = c_star[None, :] + spread * torch.randn((M, N), generator=g, device=dev)
    c_bar = c.mean(0)
    w = torch.zeros((M, N), device=dev)                                    # all workers start at the origin
    theta_g = torch.zeros(N, device=dev)
    momentum = torch.zeros(N, device=dev)

    def global_loss() -> float:
        wm = w.mean(0)
        return float((0.5 * a * (wm - c_bar) ** 2).sum().item())

    if variant == "diloco":
        ptr, off, ln = [0, 1], [0], [N]
        sizes = [N]
    else:
        ptr = list(range(K + 1))
        off = [k * frag for k in range(K)]
        ln = [frag] * K
        sizes = ln
    ctx = B.Context(N, ptr, off, ln, M, device=dev.index or 0)
    if variant == "cocodc":
        hyper = B.Hyper(M=M, H=H, tau=tau, lam=lam, alpha=1.0)
    elif variant == "streaming_diloco":
        hyper = B.Hyper(M=M, H=H, tau=tau, lam=0.0, alpha=0.5, comp_mode=B.COMP_NONE)
    elif variant == "diloco":
        hyper = B.Hyper(M=M, H=H, tau=0, lam=0.0, alpha=1.0, comp_mode=B.COMP_NONE)
    else:
        raise ValueError(variant)
    drv = None
    if variant != "diloco":
        drv = RoundDriver(ctx, hyper, w, theta_g, momentum, sizes, gamma=gamma, Tc=Tc, Ts=Ts,
                          budget_kind=B.BUDGET_COUNT, budget=1)
    ids = torch.zeros(1, dtype=torch.int32, device=dev)
    n_ids = torch.ones(1, dtype=torch.int32, device=dev)
    last_sync = torch.zeros(len(sizes), dtype=torch.int64, device=dev)
    norms = torch.zeros(len(sizes), device=dev)
    scores = torch.zeros(len(sizes), device=dev)
    losses = [(0, global_loss())]
    syncs = 0
    for t in range(1, steps + 1):
        grad = a[None, :] * (w - c) + grad_noise * torch.randn(w.shape, generator=g, device=dev)
        w.sub_(inner_lr * grad)                                            # one local step on every worker
        if drv is not None:
            drv.after_local_step(t)
        elif t % H == 0:                                                   # DiLoCo: blocking sync of the whole model
            ctx.cocodc_outer_step(hyper, w, w, w.stride(0), w.stride(0), None, theta_g, momentum, None, ids, n_ids,
                                  t, t, last_sync, norms, scores)
            syncs += 1
        if t % log_every == 0 or t == steps:
            losses.append((t, global_loss()))
    status = ctx.cocodc_poll_status()
    if status != B.OK:
        raise RuntimeError(f"device status {status}: {B.status_string(status)}")
    if drv is not None:
        syncs = drv.completed
    return ToyResult(variant, lam, tau, losses, syncs)


def main() -> None:
    print(f"{'variant':18s} {'lambda':>6s} {'tau':>3s} {'syncs':>5s} {'start':>10s} {'final':>10s}")
    for variant, lam, tau in (("diloco", 0.0, 0), ("streaming_diloco", 0.0, 4), ("cocodc", 0.0, 4),
                              ("cocodc", 0.5, 4), ("cocodc", 1.0, 4), ("streaming_diloco", 0.0, 8),
                              ("cocodc", 0.5, 8)):
        r = run_toy(variant, lam=lam, tau=max(tau, 0) if variant != "diloco" else 4)
        print(f"{variant:18s} {lam:6.2f} {tau:3d} {r.syncs:5d} {r.losses[0][1]:10.3f} {r.final:10.5f}")


if __name__ == "__main__":
    main()
