#!/usr/bin/env python
"""Benchmark of the CoCoDC outer synchronisation step on B200.

One step = one pass of the whole path over the fragments in flight:
    cocodc_outer_step (S1-S6, fused) on the fragments whose sync completes now,
    cocodc_initiate for the next set: cocodc_select_fragments (S7) and cocodc_snapshot (S0) of that set in one launch.
The metric is fragment parameters completed per second (whole job), with the achieved HBM rate of
the fused kernel beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]
                    [--deployment replicas|param_shard|worker_per_device]

N > 1: one rank per GPU over NCCL.  Started under torch.distributed.run (RANK / WORLD_SIZE in the environment)
the process is one of the ranks; started plainly with --gpus N it launches the N ranks itself.  Deployments:
    replicas           every rank owns an independent parameter shard of the same shape (no data-path collective)
    param_shard        rank r owns one element range (all workers of it) of a model N times larger: S1-S5 are
                       local, the K per-fragment sums of squares are all-reduced as fp64 before the scores are
                       formed, selection runs replicated and must agree on every rank (Section 3.2)
    worker_per_device  the workers are spread over the ranks (Section 2.1, one worker per device in the paper):
                       per-device pseudo-gradient sums, all-reduce of the listed fragments, completion from
                       the received sum
"""

from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import synth

METRIC = "outer_step_params_per_s"
UNIT = "params/s"
DEFAULT_WORKLOAD = "llama_1b"


def bytes_per_param(M: int) -> int:
    """Algorithmic HBM bytes of the fused step per fragment parameter: reads 4M (recorded) + 4M (current)
    + 4 (global) + 4 (momentum), writes 4M + 4 + 4."""
    return 12 * M + 16


# --------------------------------------------------------------------------------------------
# helpers
# --------------------------------------------------------------------------------------------

def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clock/throttle samples taken while the timed region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
        return self

    def __exit__(self, *exc):
        self.result = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return False
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            try:
                pw.append(float(parts[3]))
            except ValueError:
                pass
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if sm:
            self.result = {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                           "samples": len(sm), "power_w": statistics.median(pw) if pw else None}
        return False


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def shard_units(n_units: int, world: int, rank: int):
    """Contiguous block of units owned by `rank` (used when a fixed list of problems is split)."""
    base, rem = divmod(n_units, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def aggregate(total_units_local: float, seconds_local: float, world: int, backend_ready: bool):
    """Whole-job figures: units summed over ranks, time = max over ranks."""
    if world == 1 or not backend_ready:
        return total_units_local, seconds_local
    import torch.distributed as dist
    dev = torch.device("cuda", torch.cuda.current_device()) if dist.get_backend() == "nccl" else torch.device("cpu")
    u = torch.tensor([total_units_local], dtype=torch.float64, device=dev)
    t = torch.tensor([seconds_local], dtype=torch.float64, device=dev)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(u.item()), float(t.item())


def pool_capacity(w: synth.Workload) -> int:
    sizes = np.sort(w.partition.frag_sizes)[::-1]
    if w.budget_kind == "params":
        cap = int(w.budget + sizes[0])
    else:
        cap = int(sizes[:max(1, w.budget)].sum())
    return (cap + 8 * w.K + 1023) // 1024 * 1024


# --------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------

class DeviceJob:
    """Workload resident in HBM plus its schedule state, stepped through the C-ABI binding."""

    def __init__(self, w: synth.Workload, device: torch.device, variant: str = "cocodc",
                 deployment: str = "replicas", world: int = 1, M_total: int = 0, worker_offset: int = 0,
                 shard: int = 0, defer_scores: bool = False):
        from paper_2504_17672_b200 import binding as B
        self.B, self.w, self.dev, self.variant = B, w, device, variant
        # the completion leaves the last steps of Eq. 10 to the initiation that follows it in the same step
        self.defer = defer_scores and deployment == "replicas" and variant != "diloco"
        self.deployment, self.world, self.M_total = deployment, world, (M_total or w.M)
        ptr, off, ln = w.partition.csr()
        self.ctx = B.Context(w.N, ptr, off, ln, w.M, device=device.index or 0)
        K = w.K
        self.sizes = w.partition.frag_sizes
        self.kind = B.BUDGET_PARAMS if w.budget_kind == "params" else B.BUDGET_COUNT
        # scores of an earlier round: the expected change norm of this seed, s_p * sqrt(n_p)
        scores0 = (synth.fragment_scales(w) * np.sqrt(self.sizes)).astype(np.float32)
        self.scores = torch.from_numpy(scores0).to(device)
        self.norms = torch.zeros(K, dtype=torch.float32, device=device)
        self.last_sync = torch.zeros(K, dtype=torch.int64, device=device)
        self.mask = torch.zeros(K, dtype=torch.uint8, device=device)
        # id list and its length live in one row of K + 1 integers; use_row() points the job at another row, so
        # that a benchmark can keep every step's list (selection writes straight into the next row: no copies)
        self.use_row(torch.full((K + 1,), -1, dtype=torch.int32, device=device))
        self.n_ids.zero_()
        self.pool_off = torch.full((K,), -1, dtype=torch.int64, device=device)
        self.t = w.tau
        self.hyper = B.Hyper(M=w.M, H=w.H, tau=w.tau, outer_lr=w.outer_lr, momentum=w.momentum, lam=w.lam,
                             alpha=w.alpha)
        if variant == "streaming_diloco":      # Eq. 1-3 only: no compensation, blend with alpha = 0.5
            self.hyper.comp_mode, self.hyper.alpha = B.COMP_NONE, 0.5
        elif variant == "diloco":              # blocking sync of the whole model: snapshot = current, no delay
            self.hyper.comp_mode, self.hyper.tau = B.COMP_NONE, 0
        # first selection, then generate the buffers with the selected fragments' snapshots in the pool
        self.select()
        torch.cuda.synchronize(device)
        n = int(self.n_ids.item())
        ids0 = self.ids[:n].tolist()
        offs = {p: int(self.pool_off[p].item()) for p in ids0}
        self.bufs = synth.generate(w, device, snap_layout="pool", pool_ids=ids0, pool_offsets=offs,
                                   pool_len=pool_capacity(w), worker_offset=worker_offset, shard=shard)
        if variant == "diloco":
            self.ids.copy_(torch.arange(K, dtype=torch.int32, device=device))
            self.n_ids.fill_(K)
        if deployment == "param_shard":
            self.sumsq = torch.zeros(K, dtype=torch.float64, device=device)
        if deployment == "worker_per_device":
            self.sum_buf = torch.zeros(w.N, dtype=torch.float32, device=device)
        self.collective_bytes = 0       # bytes this rank handed to collectives on the data path

    def use_row(self, row: torch.Tensor):
        self.idbuf = row
        self.ids, self.n_ids = row[:self.w.K], row[self.w.K:]

    def select(self):
        w = self.w
        self.ctx.cocodc_select_fragments(self.scores, self.last_sync, None, self.t, w.H, self.kind, w.budget,
                                         self.mask, self.ids, self.n_ids, self.pool_off)

    def outer_param_shard(self):
        """This rank's element range: S1-S5 and the local sums of squares; Eq. 10 is finished after the all-reduce."""
        B, b, w = self.B, self.bufs, self.w
        self.sumsq.zero_()      # entries of fragments not listed now must not carry old totals into the all-reduce
        self.ctx.cocodc_outer_step(self.hyper, b.w_now, b.w_snap, b.now_stride, b.snap_stride, self.pool_off,
                                   b.theta_g, b.momentum, None, self.ids, self.n_ids, self.t, self.t + w.tau,
                                   None, None, None, stages=B.STAGE_OUTER | B.STAGE_MERGE | B.STAGE_SUMSQ,
                                   sumsq_out=self.sumsq)

    def scores_param_shard(self):
        import torch.distributed as dist
        w = self.w
        if self.world > 1:
            dist.all_reduce(self.sumsq, op=dist.ReduceOp.SUM)
            self.collective_bytes += self.sumsq.numel() * 8
        self.ctx.cocodc_scores_from_sumsq(self.sumsq, self.ids, self.n_ids, None, self.t, self.t + w.tau,
                                          self.last_sync, self.norms, self.scores)

    def pseudo_sum_and_exchange(self):
        """Worker-per-device: this rank's pseudo-gradient sums, then the all-reduce of Section 2.1 over the
        listed fragments' ranges (the id list is read back: the host slices the buffer for the collective)."""
        from paper_2504_17672_b200 import distributed as D
        b, w = self.bufs, self.w
        self.ctx.cocodc_pseudo_gradient_sum(b.w_snap, b.snap_stride, self.pool_off, b.theta_g, w.M, self.sum_buf,
                                            self.ids, self.n_ids)
        if self.world > 1:
            n = int(self.n_ids.item())
            ids_h = self.ids[:n].tolist()
            ranges = D.fragment_ranges(w.partition.fragments, ids_h)
            D.allreduce_ranges(self.sum_buf, ranges)
            self.collective_bytes += 4 * sum(l for _, l in ranges)

    def outer_received(self):
        b, w = self.bufs, self.w
        self.ctx.cocodc_outer_step_received(self.hyper, self.M_total, b.w_now, b.w_snap, b.now_stride, b.snap_stride,
                                            self.pool_off, b.theta_g, b.momentum, self.sum_buf, None, self.ids,
                                            self.n_ids, self.t, self.t + w.tau, self.last_sync, self.norms,
                                            self.scores)

    def outer(self):
        b, w = self.bufs, self.w
        if self.deployment == "param_shard":
            return self.outer_param_shard()
        if self.deployment == "worker_per_device":
            return self.outer_received()
        if self.variant == "diloco":
            self.ctx.cocodc_outer_step(self.hyper, b.w_now, b.w_now, b.now_stride, b.now_stride, None,
                                       b.theta_g, b.momentum, None, self.ids, self.n_ids, self.t, self.t,
                                       self.last_sync, self.norms, self.scores)
            return
        self.ctx.cocodc_outer_step(self.hyper, b.w_now, b.w_snap, b.now_stride, b.snap_stride, self.pool_off,
                                   b.theta_g, b.momentum, None, self.ids, self.n_ids, self.t, self.t + w.tau,
                                   self.last_sync, self.norms, self.scores,
                                   stages=self.B.STAGE_ALL | (self.B.STAGE_DEFER if self.defer else 0))

    def initiate(self):
        """Algorithm 2 for the next set and the snapshot of what it picks (cocodc_initiate: one launch)."""
        b, w = self.bufs, self.w
        self.ctx.cocodc_initiate(self.scores, self.last_sync, None, self.t, w.H, self.kind, w.budget, self.mask,
                                 self.ids, self.n_ids, self.pool_off, b.w_now, b.w_snap, b.now_stride, b.snap_stride,
                                 w.M)

    def snapshot(self):
        b = self.bufs
        self.ctx.cocodc_snapshot(b.w_now, b.w_snap, b.now_stride, b.snap_stride, self.pool_off, self.w.M,
                                 self.ids, self.n_ids)

    def step(self, next_row=None, ev=None):
        """Complete the fragments in flight, choose the next set, record their snapshots."""
        if self.deployment == "worker_per_device":
            self.pseudo_sum_and_exchange()
        if ev is not None:
            ev[0].record()
        self.outer()
        if ev is not None:
            ev[1].record()
        if self.deployment == "param_shard":
            self.scores_param_shard()
        if self.variant == "diloco":
            self.t += self.w.H
            return
        self.t += self.w.tau
        if next_row is not None:      # the next set's list goes to a fresh row; this step's row stays as its record
            self.use_row(next_row)
        self.initiate()


def timed_device_leg(job: DeviceJob, K: int, W: int, device: torch.device, local: int, barrier):
    """W warm-up steps, then exactly K timed steps between two barriers; CUDA events around the whole region and
    around every completion call.  Returns the raw figures of this rank."""
    w = job.w
    # row i: the ids step i completes and their count (row K: the set still in flight at the end)
    log = torch.full((K + 1, w.K + 1), -1, dtype=torch.int32, device=device)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(W):
        job.step()
    status = job.ctx.cocodc_poll_status()
    if status != 0:
        raise RuntimeError(f"device status after warm-up: {job.B.status_string(status)}")
    log[0].copy_(job.idbuf)
    job.use_row(log[0])
    barrier()
    launches0 = job.ctx.launch_count
    bytes0 = job.collective_bytes
    with ClockSampler(local) as clocks:
        t_begin.record()
        for i in range(K):
            job.step(log[i + 1], evs[i])
        t_end.record()
        barrier()
    status = job.ctx.cocodc_poll_status()
    if status != 0:
        raise RuntimeError(f"device status after the timed region: {job.B.status_string(status)}")
    log_h = log.cpu().numpy()
    if job.variant == "diloco":           # one fixed list (all fragments), no selection
        log_h[:] = log_h[0]
    ids_h, n_h = log_h[:K, :w.K], log_h[:K, w.K]
    sizes_of = lambda i: int(job.sizes[log_h[i, :log_h[i, w.K]]].sum())
    per_step = [sizes_of(i) for i in range(K)]
    # the set whose snapshot step i takes is the set step i + 1 completes
    per_step_snapshot = [0] * K if job.variant == "diloco" else [sizes_of(i + 1) for i in range(K)]
    return {
        "seconds": t_begin.elapsed_time(t_end) / 1e3,
        "per_step": per_step,
        "per_step_snapshot": per_step_snapshot,
        "outer_ms": [a.elapsed_time(b) for a, b in evs],
        "launches": job.ctx.launch_count - launches0,
        "collective_bytes": job.collective_bytes - bytes0,
        "clocks": clocks.result,
        "ids": ids_h, "n": n_h,
    }


def completion_bytes_per_param(M: int, variant: str, deployment: str) -> int:
    """Algorithmic HBM bytes per fragment parameter of the call the roofline record times."""
    if variant == "diloco":
        return 8 * M + 16                      # zero delay: w_now is read once and written once
    if deployment == "worker_per_device":
        return 12 * M + 20                     # the received sum is one more stream
    return bytes_per_param(M)


def roofline_record(w, variant, deployment, leg, K, peak, peak_kind, traffic=None, deferred=False):
    bpp = completion_bytes_per_param(w.M, variant, deployment)
    outer_seconds = sum(leg["outer_ms"]) / 1e3
    params = float(sum(leg["per_step"]))
    achieved = params * bpp / outer_seconds / 1e9
    per_launch = sorted(leg["per_step"][i] * bpp / leg["outer_ms"][i] / 1e6 for i in range(K) if leg["outer_ms"][i] > 0)
    if w.M > 8:
        kernel = "k_outer_ring (fused S1-S6)"
    elif variant == "diloco":
        name = "k_outer_inplace" if w.M in (3, 4, 5) else "k_outer_tma"   # the library's choice per worker count
        kernel = f"{name}<{w.M}> (fused S1-S6, zero delay)"
    elif deployment == "worker_per_device":
        kernel = f"k_outer_tma<{w.M}, received sum> (S2-S6)"
    else:
        kernel = f"k_outer_tma<{w.M}> (fused S1-S6)"
    if deferred:      # the launch ends with the CTAs' sums of squares; the next launch's prologue forms the scores
        kernel = kernel.replace("S1-S6", "S1-S5 + sums of squares of S6")
    return {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": achieved / 8000.0,
            "bytes_per_param": bpp, "ms_per_launch": outer_seconds / K * 1e3,
            "params_per_launch": params / K,
            "achieved_median": per_launch[len(per_launch) // 2] if per_launch else None,
            "achieved_best": per_launch[-1] if per_launch else None,
            "launches_timed": len(per_launch), "traffic": traffic}


def run_ours(args):
    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        print(f"rank {rank}: no CUDA device", file=sys.stderr, flush=True)
        if world > 1:
            time.sleep(3.0)    # the launcher stops the other ranks when one fails: let them report first
        raise RuntimeError("bench.py needs a CUDA device (the CUDA library has no CPU fallback)")
    if local >= torch.cuda.device_count():
        raise RuntimeError(f"rank {rank}: local rank {local} has no GPU ({torch.cuda.device_count()} visible)")
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    backend_ready = False
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
        backend_ready = True
    deployment = args.deployment or ("param_shard" if world > 1 else "replicas")
    if args.variant != "cocodc" and deployment != "replicas":
        raise SystemExit("--variant other than cocodc runs with --deployment replicas")
    w = synth.get_workload(args.workload)
    M_total, worker_offset, shard = w.M, 0, 0
    if deployment == "replicas" and world > 1:
        w = w.with_(seed=w.seed + 1000 * rank)   # every rank owns an independent problem of the same shape
    if deployment == "param_shard":
        # every rank owns a different element range of the same fragments: same table, same drift scales and hence
        # the same initial scores everywhere (the selection is replicated, not communicated), other values
        shard = rank
    if deployment == "worker_per_device":
        M_local = max(1, w.M // world)           # the workers are spread over the ranks; at least one each
        M_total, worker_offset = M_local * world, M_local * rank
        w = w.with_(M=M_local)
    job = DeviceJob(w, device, args.variant, deployment, world, M_total, worker_offset, shard,
                    defer_scores=args.defer_scores)
    K, W = args.steps, args.warmup

    def barrier():
        torch.cuda.synchronize(device)
        if backend_ready:
            import torch.distributed as dist
            dist.barrier()
            torch.cuda.synchronize(device)

    leg = timed_device_leg(job, K, W, device, local, barrier)
    seconds = leg["seconds"]
    params_local = float(sum(leg["per_step"]))
    if deployment == "worker_per_device":
        # every rank completes the same fragments of one replicated model: the job's parameters are one rank's
        total_params, max_seconds = params_local, aggregate(0.0, seconds, world, backend_ready)[1]
    else:
        total_params, max_seconds = aggregate(params_local, seconds, world, backend_ready)
    same_selection = None
    if backend_ready and deployment != "replicas":
        # the decision is replicated, not communicated: every rank must have listed the same fragments
        import torch.distributed as dist
        mine = torch.from_numpy(np.concatenate([leg["ids"].ravel(), leg["n"]])).to(device)
        gathered = [torch.empty_like(mine) for _ in range(world)]
        dist.all_gather(gathered, mine)
        same_selection = all(bool(torch.equal(g, gathered[0])) for g in gathered)
        if not same_selection:
            raise RuntimeError("the ranks selected different fragments")

    peak, peak_kind = read_peaks()
    snap_bpp = 8 * w.M if args.variant != "diloco" else 0
    traffic = (read_traffic_note(w, params_local / K)
               if args.variant == "cocodc" and deployment in ("replicas", "param_shard") else None)
    roof = roofline_record(w, args.variant, deployment, leg, K, peak, peak_kind, traffic, deferred=job.defer)
    step_bytes = params_local * roof["bytes_per_param"] + float(sum(leg["per_step_snapshot"])) * snap_bpp
    if deployment == "worker_per_device":
        step_bytes += params_local * (4 * w.M + 8)       # the pseudo-gradient sum's own pass
    steps_desc = {
        "replicas": ("outer_step(S1-S6, the root and division of Eq. 10 left to the next launch) + "
                     "initiate(those, S7 + S0)" if job.defer else "outer_step(S1-S6) + initiate(S7 + S0)"),
        "param_shard": "outer_step(S1-S5 + sums of squares) + all-reduce of K fp64 + scores_from_sumsq(S6) "
                       "+ initiate(S7 + S0)",
        "worker_per_device": "pseudo_gradient_sum(S1) + all-reduce of the listed fragments + outer_step_received(S2-S6) "
                             "+ initiate(S7 + S0)",
    }
    out = {
        "metric": METRIC, "value": total_params / max_seconds, "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": max_seconds / K * 1e3, "higher_is_better": True,
        "scaling": "strong" if deployment == "worker_per_device" else "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "N": w.N, "K": w.K, "M": w.M, "tau": w.tau, "H": w.H,
                   "budget": f"{w.budget} {w.budget_kind}", "params_per_step": params_local / K,
                   "variant": args.variant, "deployment": deployment,
                   "step": (steps_desc[deployment] if args.variant != "diloco"
                            else "outer_step(S1-S6) over all fragments, blocking"), "snapshot_layout": "pool",
                   "l2": "inputs larger than L2 (every step streams GBs)",
                   "parallelism": {"replicas": f"replicas x{world}",
                                   "param_shard": f"parameter ranges x{world} (model of {world} x N parameters)",
                                   "worker_per_device": f"{M_total} workers over {world} devices, "
                                                        f"{w.M} per device"}[deployment]},
        "gpu_launches": int(leg["launches"]),
        "clocks": leg["clocks"],
        "roofline": roof,
        "step_gbs": step_bytes / seconds / 1e9,
    }
    if deployment != "replicas":
        out["collective"] = {"bytes_per_step_per_rank": leg["collective_bytes"] / K,
                             "what": ("K fp64 sums of squares" if deployment == "param_shard"
                                      else "fp32 pseudo-gradient sums of the listed fragments"),
                             "nvlink_bytes_per_step_per_rank": (2.0 * (world - 1) / world * leg["collective_bytes"] / K),
                             "same_selection_on_every_rank": same_selection}
    if rank == 0 and not args.no_e2e and args.variant == "cocodc" and deployment == "replicas":
        out["e2e"] = run_e2e(job, args)
    elif rank == 0:
        out["e2e"] = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(job, leg["per_step"][-1] if leg["per_step"] else 0, args)
    if (rank == 0 and world == 1 and args.workload == DEFAULT_WORKLOAD and args.variant == "cocodc"
            and deployment == "replicas" and not args.no_3b):
        job.ctx.close()
        del job
        out["roofline_llama_3b"] = second_shape_roofline("llama_3b", args, device, local, peak, peak_kind)
    if rank == 0:
        print(json.dumps(out))
    if backend_ready:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


def second_shape_roofline(name: str, args, device, local, peak, peak_kind):
    """The other shape the bandwidth target names, device-resident only (no host leg: its trainer state would need
    about 80 GB of pinned host memory): the same step on llama_3b, timed the same way."""
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 115 * 2 ** 30:
        return {"workload": name, "skipped": f"needs about 105 GB of device memory, {free / 2 ** 30:.0f} GB free"}
    w = synth.get_workload(name)
    job = DeviceJob(w, device, "cocodc", defer_scores=args.defer_scores)
    K = max(4, min(args.steps, 20))
    leg = timed_device_leg(job, K, 3, device, local, lambda: torch.cuda.synchronize(device))
    roof = roofline_record(w, "cocodc", "replicas", leg, K, peak, peak_kind,
                           read_traffic_note(w, float(sum(leg["per_step"])) / K), deferred=job.defer)
    roof.update({"workload": name, "steps": K, "ms_per_step": leg["seconds"] / K * 1e3,
                 "params_per_s": float(sum(leg["per_step"])) / leg["seconds"],
                 "clocks": leg["clocks"], "gpu_launches": int(leg["launches"])})
    job.ctx.close()
    del job
    gc.collect()
    torch.cuda.empty_cache()
    return roof


def run_sweep(args):
    """Compensation sweep at the 1B shape: tau x lambda x fraction of the 32 fragments completing per call.

    Per variant, from one run: agreement with the CPU oracle (sampled elements of every completed fragment on a
    checked launch: worst relative error, which must stay within 1e-6) and the fused kernel's GB/s from CUDA
    events over a few more launches.  The oracle here is the checker of the sweep's "oracle agreement" column,
    as in the tests; it takes no part in what is timed.  Prints one JSON line with all variants."""
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (the CUDA library has no CPU fallback)")
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import helpers                                   # the parity tests' sampled check (oracle on sampled elements)
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    w0 = synth.get_workload("sweep_1b")
    bufs = synth.generate(w0, device)
    prob = helpers.GpuProblem(w0, bufs, device="cuda:0")
    ctx, B = prob.ctx, prob.B
    K = w0.K
    frag = int(w0.partition.frag_sizes[0])
    peak, peak_kind = read_peaks()
    bpp = bytes_per_param(w0.M)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    variants = []
    reps = max(3, args.steps // 4)
    t = 0
    for frac in (0.25, 0.5, 1.0):
        n = int(round(frac * K))
        ids = list(range(n))
        prob.set_ids(ids)
        for tau in (1, 2, 4, 8):
            for lam in (0.0, 0.25, 0.5, 1.0):
                w = w0.with_(tau=tau, lam=lam)
                prob.w = w
                hp = prob.hyper()
                # fresh outer state per variant (repeated completions of the same snapshots cancel Delta away)
                bufs.momentum.normal_(0.0, 1e-3)
                bufs.theta_g.add_(bufs.momentum)
                bufs.momentum.normal_(0.0, 1e-3)

                def launch():
                    nonlocal t
                    t += tau
                    prob.outer_step(t, t + tau, hyper=hp)
                check = helpers.SampledCheck(prob, ids, seed=len(variants), n_random=20_000)
                launch()
                torch.cuda.synchronize(device)
                parity_worst = check.check(t, t + tau, helpers.orc_hyper(w))    # raises beyond 1e-6
                a.record()
                for _ in range(reps):
                    launch()
                b.record()
                torch.cuda.synchronize(device)
                ms = a.elapsed_time(b) / reps
                gbs = n * frag * bpp / ms / 1e6
                variants.append({"tau": tau, "lambda": lam, "fraction": frac, "fragments": n, "ms": ms,
                                 "gbs": gbs, "frac_of_peak": gbs / peak, "parity_worst": parity_worst,
                                 "parity_ok": bool(parity_worst <= helpers.TOL_PARAM)})
    status = ctx.cocodc_poll_status()
    g = [v["gbs"] for v in variants]
    print(json.dumps({"metric": "outer_step_gbs_per_variant", "workload": w0.name, "unit": "GB/s", "peak": peak,
                      "peak_kind": f"of {peak_kind}", "launches_per_variant": reps, "status": int(status),
                      "min": min(g), "median": statistics.median(g), "max": max(g),
                      "parity_tolerance": helpers.TOL_PARAM, "parity_worst": max(v["parity_worst"] for v in variants),
                      "parity_checked": "sampled elements of every completed fragment, first launch of each variant",
                      "variants": variants}))


def run_micro(args):
    """Every streaming entry point on its own, on the llama_1b buffers: algorithmic GB/s from CUDA events.

    Rows: the fused step and its modes, the unfused halves, snapshot, stand-alone scores (with and without a
    context), and the two calls of the worker-per-device deployment."""
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (the CUDA library has no CPU fallback)")
    from paper_2504_17672_b200 import binding as B
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    w = synth.get_workload(args.workload)
    bufs = synth.generate(w, device)                 # full-size snapshot buffer: every fragment has a snapshot
    ptr, off, ln = w.partition.csr()
    ctx = B.Context(w.N, ptr, off, ln, w.M, device=0)
    K, M = w.K, w.M
    sizes = w.partition.frag_sizes
    chosen = [int(p) for p in np.argsort(-sizes, kind="stable")[:max(1, min(4, K))]]
    n = int(sizes[chosen].sum())
    ids = torch.tensor(chosen + [-1] * (K - len(chosen)), dtype=torch.int32, device=device)
    n_ids = torch.tensor([len(chosen)], dtype=torch.int32, device=device)
    scores = torch.zeros(K, device=device)
    norms = torch.zeros(K, device=device)
    last_sync = torch.zeros(K, dtype=torch.int64, device=device)
    scratch = torch.zeros(w.N, device=device)
    hp = B.Hyper(M=M, H=w.H, tau=w.tau, outer_lr=w.outer_lr, momentum=w.momentum, lam=w.lam, alpha=w.alpha)
    b = bufs
    peak, peak_kind = read_peaks()
    t = [0]

    def outer(stages=7, delta=None, snap=None):
        t[0] += w.tau
        s = b.w_snap if snap is None else snap
        ctx.cocodc_outer_step(hp, b.w_now, s, b.now_stride, s.stride(0), None, b.theta_g, b.momentum, delta,
                              ids, n_ids, t[0], t[0] + w.tau, last_sync, norms, scores, stages)

    hp0 = B.Hyper(M=M, H=w.H, tau=0, outer_lr=w.outer_lr, momentum=w.momentum, lam=0.0, alpha=1.0,
                  comp_mode=B.COMP_NONE)

    def zero_delay():
        t[0] += w.tau
        ctx.cocodc_outer_step(hp0, b.w_now, b.w_now, b.now_stride, b.now_stride, None, b.theta_g, b.momentum, None,
                              ids, n_ids, t[0], t[0], last_sync, norms, scores, 7)

    def received():
        t[0] += w.tau
        ctx.cocodc_outer_step_received(hp, M, b.w_now, b.w_snap, b.now_stride, b.snap_stride, None, b.theta_g,
                                       b.momentum, scratch, None, ids, n_ids, t[0], t[0] + w.tau, last_sync,
                                       norms, scores)

    rows = [
        ("cocodc_outer_step, all stages (S1-S6)", 12 * M + 16, n, lambda: outer()),
        ("cocodc_outer_step + delta_g_out", 12 * M + 20, n, lambda: outer(delta=scratch)),
        ("cocodc_outer_step, zero delay (w_snap == w_now)", 8 * M + 16, n, zero_delay),
        ("cocodc_outer_step, OUTER|SCORE only (S1-S3, S6)", 4 * M + 16, n, lambda: outer(stages=5)),
        ("cocodc_merge (S4-S5)", 12 * M + 4, n,
         lambda: ctx.cocodc_merge(hp, b.w_now, b.w_snap, b.now_stride, b.snap_stride, None, b.theta_g, ids, n_ids)),
        ("cocodc_snapshot (S0)", 8 * M, n,
         lambda: ctx.cocodc_snapshot(b.w_now, b.w_snap, b.now_stride, b.snap_stride, None, M, ids, n_ids)),
        ("cocodc_pseudo_gradient_sum", 4 * M + 8, n,
         lambda: ctx.cocodc_pseudo_gradient_sum(b.w_snap, b.snap_stride, None, b.theta_g, M, scratch, ids, n_ids)),
        ("cocodc_outer_step_received", 12 * M + 20, n, received),
        ("cocodc_outer_step_received_peers, 2 buffers of partial sums (all on this GPU)", 12 * M + 16 + 8, n,
         lambda: received_peers(2)),
        ("cocodc_outer_step_received_peers, 4 buffers of partial sums (all on this GPU)", 12 * M + 16 + 16, n,
         lambda: received_peers(4)),
        ("cocodc_fragment_scores (all fragments)", 4, w.N,
         lambda: ctx.cocodc_fragment_scores(b.theta_g, None, norms, scores)),
    ]
    more = [torch.zeros(w.N, device=device) for _ in range(3)]

    def received_peers(R):
        t[0] += w.tau
        ctx.cocodc_outer_step_received_peers(hp, M * R, b.w_now, b.w_snap, b.now_stride, b.snap_stride, None,
                                             b.theta_g, b.momentum, ([scratch] + more)[:R], None, ids, n_ids, t[0],
                                             t[0] + w.tau, last_sync, norms, scores)

    if K <= B.NOALLOC_MAX_K and len(off) <= B.NOALLOC_MAX_SEGMENTS:
        rows.append(("cocodc_fragment_scores_noalloc (all fragments)", 4, w.N,
                     lambda: B.cocodc_fragment_scores_noalloc(w.N, ptr, off, ln, b.theta_g, None, norms, scores)))
    ev_a, ev_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = max(5, args.steps // 5)
    out = []
    for name, bpp, params, fn in rows:
        for _ in range(3):
            fn()
        torch.cuda.synchronize(device)
        ev_a.record()
        for _ in range(reps):
            fn()
        ev_b.record()
        torch.cuda.synchronize(device)
        ms = ev_a.elapsed_time(ev_b) / reps
        gbs = params * bpp / ms / 1e6
        out.append({"entry": name, "bytes_per_param": bpp, "params": params, "ms": ms, "gbs": gbs,
                    "frac_of_peak": gbs / peak})
    status = ctx.cocodc_poll_status()
    print(json.dumps({"metric": "entry_point_gbs", "workload": w.name, "unit": "GB/s", "peak": peak,
                      "peak_kind": f"of {peak_kind}", "launches_per_entry": reps, "fragments": chosen,
                      "status": int(status), "entries": out}))


def run_workers(args):
    """The fused step, the zero-delay step, the snapshot and the two calls of the worker-per-device deployment
    (pseudo-gradient sum, completion from a received sum) for a range of worker counts M on one fixed shape
    (4 fragments of --workers-fragment parameters per worker): algorithmic GB/s from CUDA events.  M = 1..8 run the
    compile-time instances of the staged kernel, larger M the chunk-ring kernel."""
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (the CUDA library has no CPU fallback)")
    from paper_2504_17672_b200 import binding as B
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    peak, peak_kind = read_peaks()
    frag, K = int(args.workers_fragment), 4
    n = frag * K
    ev_a, ev_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = max(5, args.steps // 5)
    out = []
    status = 0
    for M in [int(x) for x in args.workers_list.split(",")]:
        w = synth.small_workload([frag] * K, M=M, seed=7, tau=4, name=f"workers_{M}")
        b = synth.generate(w, device)
        ptr, off, ln = w.partition.csr()
        ctx = B.Context(w.N, ptr, off, ln, M, device=0)
        ids = torch.arange(K, dtype=torch.int32, device=device)
        n_ids = torch.tensor([K], dtype=torch.int32, device=device)
        scores = torch.zeros(K, device=device)
        norms = torch.zeros(K, device=device)
        last_sync = torch.zeros(K, dtype=torch.int64, device=device)
        hp = B.Hyper(M=M, H=w.H, tau=w.tau, outer_lr=w.outer_lr, momentum=w.momentum, lam=w.lam, alpha=w.alpha)
        hp0 = B.Hyper(M=M, H=w.H, tau=0, outer_lr=w.outer_lr, momentum=w.momentum, lam=0.0, alpha=1.0,
                      comp_mode=B.COMP_NONE)
        t = [0]

        def fused():
            t[0] += w.tau
            ctx.cocodc_outer_step(hp, b.w_now, b.w_snap, b.now_stride, b.snap_stride, None, b.theta_g, b.momentum,
                                  None, ids, n_ids, t[0], t[0] + w.tau, last_sync, norms, scores, 7)

        def zero_delay():
            t[0] += w.tau
            ctx.cocodc_outer_step(hp0, b.w_now, b.w_now, b.now_stride, b.now_stride, None, b.theta_g, b.momentum,
                                  None, ids, n_ids, t[0], t[0], last_sync, norms, scores, 7)

        def snapshot():
            ctx.cocodc_snapshot(b.w_now, b.w_snap, b.now_stride, b.snap_stride, None, M, ids, n_ids)

        sums = torch.zeros(w.N, device=device)

        def pseudo_sum():
            ctx.cocodc_pseudo_gradient_sum(b.w_snap, b.snap_stride, None, b.theta_g, M, sums, ids, n_ids)

        def received():      # the M workers of this device among 2M in all
            t[0] += w.tau
            ctx.cocodc_outer_step_received(hp, 2 * M, b.w_now, b.w_snap, b.now_stride, b.snap_stride, None,
                                           b.theta_g, b.momentum, sums, None, ids, n_ids, t[0], t[0] + w.tau,
                                           last_sync, norms, scores)

        row = {"M": M, "params": n}
        for name, bpp, fn in (("fused", 12 * M + 16, fused), ("zero_delay", 8 * M + 16, zero_delay),
                              ("snapshot", 8 * M, snapshot), ("pseudo_gradient_sum", 4 * M + 8, pseudo_sum),
                              ("received", 12 * M + 20, received)):
            for _ in range(3):
                fn()
            torch.cuda.synchronize(device)
            ev_a.record()
            for _ in range(reps):
                fn()
            ev_b.record()
            torch.cuda.synchronize(device)
            ms = ev_a.elapsed_time(ev_b) / reps
            row[name] = {"bytes_per_param": bpp, "ms": ms, "gbs": n * bpp / ms / 1e6,
                         "frac_of_peak": n * bpp / ms / 1e6 / peak}
        status = status or int(ctx.cocodc_poll_status())
        out.append(row)
        ctx.close()
        del b, ctx
        torch.cuda.empty_cache()
    print(json.dumps({"metric": "fused_step_gbs_by_worker_count", "unit": "GB/s", "peak": peak,
                      "peak_kind": f"of {peak_kind}", "launches_per_entry": reps, "params_per_launch": n,
                      "status": status, "rows": out}))


def kernel_source_sha() -> str:
    """Hash of the fused kernel's sources as the compiler sees them: comments and white space do not count."""
    import hashlib
    import re
    h = hashlib.sha256()
    for name in ("outer.cuh", "outer_tma.cuh", "plan.cuh"):
        with open(os.path.join(ROOT, "paper_2504_17672_b200", "csrc", name), "r") as f:
            text = f.read()
        text = re.sub(r"/\*.*?\*/", " ", text, flags=re.S)
        text = re.sub(r"//[^\n]*", " ", text)
        h.update(" ".join(text.split()).encode())
    return h.hexdigest()[:16]


def read_traffic_note(w, params_per_launch: float):
    """DRAM bytes per launch of the fused kernel: bytes per parameter measured by ncu on the small case
    (profiles/dram_traffic.txt) scaled by the parameters of one launch; None if the kernel sources changed
    since the capture or no capture covers this worker count."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    try:
        with open(path) as f:
            lines = [l.split() for l in f if l.startswith("kernel=")]
    except OSError:
        return None
    sha = kernel_source_sha()
    for fields in lines:
        d = dict(x.split("=", 1) for x in fields)
        if d.get("kernel") == "k_outer_tma" and int(d.get("M", -1)) == w.M and d.get("source_sha") == sha:
            return float(d["bytes_per_param"]) * params_per_launch
    return None


# --------------------------------------------------------------------------------------------
# end to end: parameters in pinned host memory, through the host-buffer entry points
# --------------------------------------------------------------------------------------------

def measure_pcie(dev, gib: float = 1.0, reps: int = 3):
    """Rate of plain pinned copies on this machine with both directions busy at once (GB/s each way): 1 GiB host to
    device and 1 GiB device to host on two streams, CUDA events per stream, best of `reps`."""
    n = int(gib * 2 ** 30) // 4
    try:
        h_in = torch.empty(n, dtype=torch.float32, pin_memory=True)
        h_out = torch.empty(n, dtype=torch.float32, pin_memory=True)
    except RuntimeError:
        return None, None
    h_in.fill_(1.0)
    d_in = torch.empty(n, dtype=torch.float32, device=dev)
    d_out = torch.ones(n, dtype=torch.float32, device=dev)
    s1, s2 = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    best_h2d = best_d2h = 0.0
    for _ in range(reps + 1):
        torch.cuda.synchronize(dev)
        a1, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a2, b2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(s1):
            a1.record()
            d_in.copy_(h_in, non_blocking=True)
            b1.record()
        with torch.cuda.stream(s2):
            a2.record()
            h_out.copy_(d_out, non_blocking=True)
            b2.record()
        torch.cuda.synchronize(dev)
        best_h2d = max(best_h2d, n * 4 / a1.elapsed_time(b1) / 1e6)
        best_d2h = max(best_d2h, n * 4 / a2.elapsed_time(b2) / 1e6)
    del h_in, h_out, d_in, d_out
    return best_h2d, best_d2h


def run_e2e(job: DeviceJob, args):
    """Same step with the trainer's state (w_now, theta_g, momentum, schedule arrays) in pinned host memory.

    Per step: cocodc_outer_step_host streams the completing fragments host->device->host (snapshots were
    put on the device at initiation); selection runs on the device from the host's schedule arrays;
    cocodc_snapshot_host copies the next set's parameters into the device pool."""
    w, dev, B = job.w, job.dev, job.B
    b = job.bufs
    torch.cuda.synchronize(dev)
    try:
        host = {k: torch.empty(getattr(b, k).shape, dtype=torch.float32, pin_memory=True)
                for k in ("w_now", "theta_g", "momentum")}
    except RuntimeError as e:
        return {"value": None, "unit": UNIT, "error": f"pinned host allocation failed: {e}"}
    for k, v in host.items():
        v.copy_(getattr(b, k))
    scores_h = job.scores.cpu()
    norms_h = job.norms.cpu()
    last_h = job.last_sync.cpu()
    n = int(job.n_ids.item())
    ids_h = job.ids.cpu()
    pool_off_h = job.pool_off.cpu()
    ws = torch.empty(768 * 2 ** 20 // 4, dtype=torch.float32, device=dev)
    steps = max(1, min(args.e2e_steps, args.steps))
    t = job.t
    h2d = d2h = 0
    params = 0
    small = w.K * (4 + 8 + 4 + 4 + 8)

    def one(timed):
        nonlocal t, n, ids_h, pool_off_h, h2d, d2h, params
        cnt = int(job.sizes[ids_h[:n].numpy()].sum())
        job.ctx.cocodc_outer_step_host(job.hyper, host["w_now"], b.w_snap, w.N, b.snap_stride, pool_off_h,
                                       host["theta_g"], host["momentum"], None, ids_h, n, t, t + w.tau,
                                       last_h, norms_h, scores_h, ws, snap_on_device=True)
        t += w.tau
        job.scores.copy_(scores_h, non_blocking=True)
        job.last_sync.copy_(last_h, non_blocking=True)
        job.ctx.cocodc_select_fragments(job.scores, job.last_sync, None, t, w.H, job.kind, w.budget, job.mask,
                                        job.ids, job.n_ids, job.pool_off)
        ids_h = job.ids.cpu()
        pool_off_h = job.pool_off.cpu()
        n2 = int(job.n_ids.item())
        cnt2 = int(job.sizes[ids_h[:n2].numpy()].sum())
        job.ctx.cocodc_snapshot_host(host["w_now"], b.w_snap, w.N, b.snap_stride, pool_off_h, w.M, ids_h, n2)
        torch.cuda.synchronize(dev)
        if timed:
            params += cnt
            h2d += cnt * (4 * w.M + 8) + cnt2 * 4 * w.M + small
            d2h += cnt * (4 * w.M + 8) + small
        n = n2

    one(False)                      # warm-up
    t0 = time.perf_counter()
    for _ in range(steps):
        one(True)
    torch.cuda.synchronize(dev)
    dt = time.perf_counter() - t0
    status = job.ctx.cocodc_poll_status()
    res = {"value": params / dt, "unit": UNIT, "h2d_bytes_per_step": h2d // steps,
           "d2h_bytes_per_step": d2h // steps, "steps": steps, "ms_per_step": dt / steps * 1e3,
           "api": "cocodc_outer_step_host + cocodc_select_fragments + cocodc_snapshot_host",
           "host_memory": "pinned", "status": int(status)}
    del host, ws
    # what the bus of this box gives plain pinned copies, both directions busy: the ceiling of the figure above
    pcie_h2d, pcie_d2h = measure_pcie(dev)
    if pcie_h2d:
        res["pcie_h2d_gbs"] = pcie_h2d
        res["pcie_d2h_gbs"] = pcie_d2h
        res["h2d_gbs"] = res["h2d_bytes_per_step"] / res["ms_per_step"] / 1e6
        res["d2h_gbs"] = res["d2h_bytes_per_step"] / res["ms_per_step"] / 1e6
        res["frac_of_pcie"] = res["h2d_gbs"] / pcie_h2d
    return res


# --------------------------------------------------------------------------------------------
# CPU baseline: the oracle, as it stands, on the host cores
# --------------------------------------------------------------------------------------------

def oracle_sample_inputs(w: synth.Workload, n_elems: int, seed: int):
    """A bounded sample of the workload for the oracle: the head of fragment 0, generated on the CPU."""
    small = synth.small_workload([n_elems], M=w.M, seed=seed, tau=w.tau, H=w.H, outer_lr=w.outer_lr,
                                 momentum=w.momentum, lam=w.lam, alpha=w.alpha)
    bufs = synth.generate(small, "cpu")
    return small, {k: getattr(bufs, k).numpy() for k in ("w_now", "w_snap", "theta_g", "momentum")}


def oracle_runner(w: synth.Workload, n_elems: int, threads: int, seed: int = 0):
    """Returns a callable that runs the oracle's fused step once on a prepared sample and returns seconds."""
    from oracle import reference as orc
    small, x = oracle_sample_inputs(w, n_elems, seed)
    hp = orc.Hyper(M=w.M, H=w.H, tau=w.tau, outer_lr=w.outer_lr, momentum=w.momentum, lam=w.lam, alpha=w.alpha)

    def run():
        t0 = time.perf_counter()
        orc.outer_step([[(0, n_elems)]], hp, x["w_now"], x["w_snap"], x["theta_g"], x["momentum"], [0],
                       w.tau, 2 * w.tau, [0], threads=threads)
        return time.perf_counter() - t0
    return run


def host_cores() -> int:
    return len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)


def cpu_baseline(job_or_workload, params_per_step, args):
    w = job_or_workload.w if hasattr(job_or_workload, "w") else job_or_workload
    cores = host_cores()
    n = args.cpu_sample
    run = oracle_runner(w, n, cores)
    run()                                   # page in the sample and the library
    total, reps = 0.0, 0
    while total < args.cpu_seconds and reps < 1000:
        total += run()
        reps += 1
    n1 = min(n, 2_000_000)                  # the same oracle on one core, for scale
    run1 = oracle_runner(w, n1, 1)
    run1()
    t1 = run1()
    return {"value": n * reps / total, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{reps} passes over {n} parameters (one fragment-shaped slice, M={w.M}) of {w.name}, "
                      f"fused step S1-S6, element range split over {cores} threads; {total:.1f} s",
            "seconds": total, "single_thread_value": n1 / t1}


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, timed on the host cores on a bounded sample per step."""
    rank, world, _ = dist_env()
    if rank != 0:
        return
    w = synth.get_workload(args.workload)
    cores = host_cores()
    n = args.reference_sample
    run = oracle_runner(w, n, cores)
    for _ in range(args.warmup):
        run()
    total = 0.0
    for i in range(args.steps):
        total += run()
    value = n * args.steps / total
    sample = (f"each step = {n} parameters (one fragment-shaped slice, M={w.M}) of {w.name}, fused step S1-S6 "
              f"by the CPU oracle over {cores} threads")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "N": w.N, "K": w.K, "M": w.M, "tau": w.tau, "H": w.H,
                   "budget": f"{w.budget} {w.budget_kind}", "sample_params_per_step": n},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def launch_ranks(n: int, argv, extra_env=None) -> int:
    """Start n ranks of this script on this node (one per GPU) under torch.distributed.run and wait for them.

    Used when the script is started plainly with --gpus n > 1; a launcher that has already set RANK / WORLD_SIZE
    (the usual `python -m torch.distributed.run ... bench.py --gpus n`) makes every process a rank directly."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    env = dict(os.environ)
    env.update(extra_env or {})
    return subprocess.run(cmd, env=env).returncode


def run_stub(args):
    """The multi-rank skeleton of the benchmark without a GPU: process group (gloo), barrier, a timed loop of a
    stand-in step, units summed and seconds maximised over the ranks, one JSON line from rank 0.  It exists so
    that the launch path and the reduction can be exercised on a machine without CUDA devices."""
    import torch.distributed as dist
    rank, world, _ = dist_env()
    if world > 1:
        dist.init_process_group("gloo", rank=rank, world_size=world)
    x = torch.ones(1000)
    units = 0.0
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        x = x * 1.0001
        units += 1000.0 * (rank + 1)
    seconds = time.perf_counter() - t0
    total, max_seconds = aggregate(units, seconds, world, world > 1)
    if rank == 0:
        print(json.dumps({"metric": "stub_units_per_s", "value": total / max_seconds, "unit": "units/s",
                          "n_gpus": world, "steps": args.steps, "units": total, "impl": "stub"}))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=list(synth.WORKLOAD_NAMES), default=DEFAULT_WORKLOAD)
    ap.add_argument("--deployment", choices=["replicas", "param_shard", "worker_per_device"], default=None,
                    help="how the path is spread over the GPUs (default: replicas on one GPU, param_shard on several)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-3b", action="store_true", help="skip the device-only roofline record on llama_3b")
    ap.add_argument("--defer-scores", action="store_true",
                    help="leave the last steps of Eq. 10 (root, division by I_p, last_sync) to the initiation that "
                         "follows the completion in the same step (COCODC_STAGE_DEFER) instead of forming them inside "
                         "the completion's own launch")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="wall time spent timing the oracle")
    ap.add_argument("--cpu-sample", type=int, default=16_000_000, help="parameters in the oracle's sample")
    ap.add_argument("--reference-sample", type=int, default=8_000_000)
    ap.add_argument("--variant", choices=["cocodc", "streaming_diloco", "diloco"], default="cocodc",
                    help="which method's arithmetic the step runs (the baselines are modes of the same kernels)")
    ap.add_argument("--micro", action="store_true", help="time every streaming entry point on its own")
    ap.add_argument("--workers", action="store_true",
                    help="time the fused step, its zero-delay and received-sum forms, the snapshot and the pseudo-gradient "
                         "sum for M = 1..34 workers")
    ap.add_argument("--workers-list", default="1,2,3,4,5,6,7,8,9,12,16,24,34", help="worker counts of --workers")
    ap.add_argument("--workers-fragment", type=int, default=24 * 1024 * 1024,
                    help="parameters per fragment (of 4) in the --workers shape")
    ap.add_argument("--sweep", action="store_true",
                    help="the 48 variants of the 1B compensation sweep: GB/s and agreement with the oracle per variant")
    ap.add_argument("--stub-step", action="store_true",
                    help="run the multi-rank skeleton with a CPU stand-in step over gloo (launch-path check, no GPU)")
    args = ap.parse_args()
    if args.gpus > 1 and "RANK" not in os.environ:
        # started plainly: become the launcher of --gpus ranks
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.stub_step:
        run_stub(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.sweep:
        run_sweep(args)
    elif args.micro:
        run_micro(args)
    elif args.workers:
        run_workers(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
