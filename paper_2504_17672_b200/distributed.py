"""Worker-per-device deployment of the completion step (Section 2.1): each rank holds M_local of the
M_total workers, and Eq. 1's sum over all workers is an all-reduce of the per-rank pseudo-gradient sums.

    cocodc_pseudo_gradient_sum  ->  all-reduce of the listed fragments' ranges  ->  cocodc_outer_step_received

The all-reduce is torch.distributed's (NCCL over NVLink on GPUs, gloo in CPU tests); received data lands
in this rank's own memory before any kernel reads it.  The global state, the momentum and the schedule
arrays are replicated: every rank computes the same outer update from the same reduced sum, which keeps
them identical without further exchange (the determinism argument of Section 3.2).
"""

from __future__ import annotations

from typing import Iterable, Sequence, Tuple

import torch
import torch.distributed as dist


def fragment_ranges(fragments: Sequence[Sequence[Tuple[int, int]]], ids: Iterable[int]):
    """(offset, length) of every segment of the listed fragments, in list order."""
    return [(int(o), int(l)) for p in ids for (o, l) in fragments[int(p)]]


def allreduce_ranges(buf: torch.Tensor, ranges, group=None, bucket_elems: int = 64 << 20) -> int:
    """Sum `buf[o:o+l]` over the ranks for every (o, l) in `ranges`, in place.  Long ranges are cut into
    buckets so that one collective never exceeds `bucket_elems` elements.  Returns the number of collectives."""
    calls = 0
    for o, l in ranges:
        for lo in range(o, o + l, bucket_elems):
            hi = min(o + l, lo + bucket_elems)
            dist.all_reduce(buf[lo:hi], op=dist.ReduceOp.SUM, group=group)
            calls += 1
    return calls


def complete_fragments(ctx, hyper, M_total: int, fragments, ids_host: Sequence[int], ids_dev, n_ids_dev,
                       w_now, w_snap, snap_offset, theta_g, momentum, sum_buf, t_p: int, t_l: int,
                       last_sync, norms, scores, group=None) -> None:
    """One completion with the workers spread over the ranks of `group`.

    ids_host must equal the device list (the selection is deterministic and identical on every rank, so the
    host can know it without a collective); sum_buf is an fp32 [N] scratch buffer."""
    ctx.cocodc_pseudo_gradient_sum(w_snap, w_snap.stride(0), snap_offset, theta_g, hyper.M, sum_buf, ids_dev, n_ids_dev)
    allreduce_ranges(sum_buf, fragment_ranges(fragments, ids_host), group=group)
    ctx.cocodc_outer_step_received(hyper, M_total, w_now, w_snap, w_now.stride(0), w_snap.stride(0), snap_offset,
                                   theta_g, momentum, sum_buf, None, ids_dev, n_ids_dev, t_p, t_l,
                                   last_sync, norms, scores)


def combine_sharded_norms(norms_local: torch.Tensor, interval: torch.Tensor = None, group=None):
    """Parameter-range sharding: every rank holds a slice of each fragment (all workers of that slice), so
    the element-wise steps need no exchange and only Eq. 10's norm spans ranks.  Given the norms each rank
    computed over its own slices, returns (norms, scores) of the whole fragments, identical on every rank:
    one all-reduce of K doubles (the sums of squares), then R_p = norm_p / max(1, I_p)."""
    sq = norms_local.double() ** 2
    dist.all_reduce(sq, op=dist.ReduceOp.SUM, group=group)
    norms = sq.sqrt()
    if interval is None:
        scores = norms.clone()
    else:
        scores = norms / interval.clamp(min=1).double()
    return norms.float(), scores.float()
