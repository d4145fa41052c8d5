"""Worker-per-device deployment of the completion step (Section 2.1): each rank holds M_local of the
M_total workers, and Eq. 1's sum over all workers is an all-reduce of the per-rank pseudo-gradient sums.

    cocodc_pseudo_gradient_sum  ->  all-reduce of the listed fragments' ranges  ->  cocodc_outer_step_received

The all-reduce is torch.distributed's (NCCL over NVLink on GPUs, gloo in CPU tests); received data lands
in this rank's own memory before any kernel reads it.  complete_fragments_peers is the variant without a
collective: the step itself adds the ranks' sums, read from the peers' mapped memory.  The global state, the momentum and the schedule
arrays are replicated: every rank computes the same outer update from the same reduced sum, which keeps
them identical without further exchange (the determinism argument of Section 3.2).
"""

from __future__ import annotations

from typing import Callable, Iterable, Sequence, Tuple

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


def complete_fragments_peers(ctx, hyper, M_total: int, rank: int, sum_bufs: Sequence, ids_dev, n_ids_dev,
                             w_now, w_snap, snap_offset, theta_g, momentum, t_p: int, t_l: int,
                             last_sync, norms, scores, barrier: Callable[[], None]) -> None:
    """The same completion with the exchange folded into the step: no all-reduce, every rank reads the other
    ranks' pseudo-gradient sums straight from their memory while it streams the fragment.

    sum_buf[r] is rank r's fp32 [N] buffer as seen from THIS process, for every rank in the same order:
    sum_bufs[rank] a tensor of this device, the others tensors or integer device addresses of peer memory mapped
    into this process (peer access between devices of one process, CUDA IPC handles, or a symmetric-memory
    allocation).  `barrier()` must return only when the work every rank has issued so far has finished on its
    device (for instance stream synchronisation followed by a process-group barrier): it separates the ranks'
    writes of their sums from the reads by the others, and those reads from the next overwrite.  The sums are
    added left to right in fp32 by every rank alike, so the replicated state stays bit-identical."""
    own = sum_bufs[rank]
    ctx.cocodc_pseudo_gradient_sum(w_snap, w_snap.stride(0), snap_offset, theta_g, hyper.M, own, ids_dev, n_ids_dev)
    barrier()
    ctx.cocodc_outer_step_received_peers(hyper, M_total, w_now, w_snap, w_now.stride(0), w_snap.stride(0),
                                         snap_offset, theta_g, momentum, list(sum_bufs), None, ids_dev, n_ids_dev,
                                         t_p, t_l, last_sync, norms, scores)
    barrier()


def scores_from_sharded_sumsq(ctx, sumsq: torch.Tensor, ids_dev, n_ids_dev, t_p: int, t_l: int, last_sync, norms,
                              scores, group=None) -> None:
    """Parameter-range sharding: every rank holds a slice of each fragment (all workers of that slice), so the
    element-wise steps need no exchange and only Eq. 10's norm spans ranks.

    `sumsq` (device fp64 [K]) holds this rank's sums of squares of the listed fragments, as cocodc_outer_step
    wrote them with STAGE_SUMSQ.  One all-reduce of those K doubles, then the library forms norms and scores from
    the totals and stamps last_sync - the same values on every rank, so the replicated selection that follows
    picks the same fragments everywhere."""
    dist.all_reduce(sumsq, op=dist.ReduceOp.SUM, group=group)
    ctx.cocodc_scores_from_sumsq(sumsq, ids_dev, n_ids_dev, None, t_p, t_l, last_sync, norms, scores)
