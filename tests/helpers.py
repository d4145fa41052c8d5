"""Shared plumbing of the GPU parity tests: run the CUDA library and the CPU oracle on the same bits."""

from __future__ import annotations

import numpy as np
import torch

import synth
from oracle import reference as orc

TOL_PARAM = 1e-6   # relative error bound on fp32 parameters and momentum
TOL_NORM = 1e-5    # relative error bound on fragment norms and scores


def np_(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy()


def rel_errors(x: np.ndarray, y: np.ndarray, floor=None):
    """(norm-wise relative error, worst element error relative to max(|y_i|, rms(y))).

    `floor` (optional, per element): magnitude of the operands the output was formed from; where it is
    given, errors are measured against max(|y_i|, rms(y), floor_i) and max(||y||, ||floor||)."""
    x = x.astype(np.float64).ravel()
    y = y.astype(np.float64).ravel()
    if y.size == 0:
        return 0.0, 0.0
    diff = np.abs(x - y)
    ny = float(np.sqrt((y * y).sum()))
    rms = ny / np.sqrt(y.size)
    denom = np.maximum(np.abs(y), rms)
    if floor is not None:
        f = np.abs(np.asarray(floor, dtype=np.float64).ravel())
        ny = max(ny, float(np.sqrt((f * f).sum())))
        denom = np.maximum(denom, f)
    normwise = float(np.sqrt((diff * diff).sum())) / ny if ny > 0 else float(diff.max())
    elem = float((diff / np.where(denom > 0, denom, 1.0)).max())
    return normwise, elem


def assert_close(x, y, tol=TOL_PARAM, what="", floor=None):
    nw, el = rel_errors(np.asarray(x), np.asarray(y), floor)
    assert nw <= tol and el <= tol, f"{what}: norm-wise {nw:.3e}, element-wise {el:.3e} > {tol:.1e}"
    return nw, el


# A fragment of a handful of elements has no rms to speak of: when the workers' pseudo-gradients (or the
# momentum term and their mean) cancel in its one element, the rounding error of the operands is all that is
# left of the output and no bound relative to the output holds; the same goes for a new global or local value
# that happens to land near zero.  Below this size the errors are therefore measured against the operands as
# well (rel_errors' floor).
SMALL_FRAGMENT = 64


def operand_floors(frs, before: dict, snap: np.ndarray, snap_offset, p: int, mu: float):
    """(mean_m |theta^m_{t_p} - theta^g|, |mu u| + that, |theta^g|, |theta^m_{t_p}| [M, n]) per element of
    fragment p: the magnitudes of what Eq. 1 averages, of what the momentum update adds, and of the states the
    new global and local parameters start from.  Indexing only; no step of the method."""
    thg = orc.gather_fragment(frs, before["theta_g"], p).astype(np.float64)
    u = orc.gather_fragment(frs, before["momentum"], p).astype(np.float64)
    rows, pos = [], 0
    for off, ln in frs[p]:
        sb = off if snap_offset is None else int(snap_offset[p]) + pos
        rows.append(snap[:, sb:sb + ln].astype(np.float64))
        pos += ln
    b = np.concatenate(rows, axis=1)
    mean_abs_delta = np.abs(b - thg[None, :]).mean(axis=0)
    return mean_abs_delta, np.abs(mu * u) + mean_abs_delta, np.abs(thg), np.abs(b)


def fragments_of(w: synth.Workload):
    return [list(f) for f in w.partition.fragments]


def touched_mask(w: synth.Workload, ids) -> np.ndarray:
    m = np.zeros(w.N, dtype=bool)
    for p in ids:
        for off, ln in w.partition.fragments[int(p)]:
            m[off:off + ln] = True
    return m


def orc_hyper(w: synth.Workload, **kw) -> orc.Hyper:
    d = dict(M=w.M, H=w.H, tau=w.tau, outer_lr=w.outer_lr, momentum=w.momentum, lam=w.lam, alpha=w.alpha)
    d.update(kw)
    return orc.Hyper(**d)


class GpuProblem:
    """A workload resident on the GPU plus its schedule state, driven through the C-ABI binding."""

    def __init__(self, w: synth.Workload, bufs: synth.DeviceBuffers, device="cuda", max_M=None):
        from paper_2504_17672_b200 import binding as B
        self.B = B
        self.w = w
        self.bufs = bufs
        self.dev = torch.device(device)
        ptr, off, ln = w.partition.csr()
        self.ctx = B.Context(w.N, ptr, off, ln, max_M or w.M, device=self.dev.index or 0)
        K = w.K
        self.scores = torch.full((K,), float("inf"), dtype=torch.float32, device=self.dev)
        self.norms = torch.zeros(K, dtype=torch.float32, device=self.dev)
        self.last_sync = torch.zeros(K, dtype=torch.int64, device=self.dev)
        self.mask = torch.zeros(K, dtype=torch.uint8, device=self.dev)
        self.ids = torch.full((K,), -1, dtype=torch.int32, device=self.dev)
        self.n_ids = torch.zeros(1, dtype=torch.int32, device=self.dev)

    def hyper(self, **kw):
        w = self.w
        d = dict(M=w.M, H=w.H, tau=w.tau, outer_lr=w.outer_lr, momentum=w.momentum, lam=w.lam, alpha=w.alpha)
        d.update(kw)
        return self.B.Hyper(**d)

    def set_ids(self, ids):
        ids = list(ids)
        self.ids.fill_(-1)
        if ids:
            self.ids[:len(ids)] = torch.tensor(ids, dtype=torch.int32, device=self.dev)
        self.n_ids.fill_(len(ids))

    def select(self, t_now, budget_kind=None, budget=None, ineligible=None):
        w = self.w
        kind = {"count": 0, "params": 1}[w.budget_kind] if budget_kind is None else budget_kind
        self.ctx.cocodc_select_fragments(self.scores, self.last_sync, ineligible, t_now, w.H, kind,
                                         w.budget if budget is None else budget,
                                         self.mask, self.ids, self.n_ids)

    def snapshot(self):
        b = self.bufs
        self.ctx.cocodc_snapshot(b.w_now, b.w_snap, b.now_stride, b.snap_stride, b.snap_offset, self.w.M,
                                 self.ids, self.n_ids)

    def outer_step(self, t_p, t_l, hyper=None, delta_out=None, stages=7, w_snap=None):
        b = self.bufs
        snap = b.w_snap if w_snap is None else w_snap
        same = snap is b.w_now
        self.ctx.cocodc_outer_step(hyper or self.hyper(), b.w_now, snap, b.now_stride,
                                   b.now_stride if same else b.snap_stride,
                                   None if same else b.snap_offset, b.theta_g, b.momentum, delta_out,
                                   self.ids, self.n_ids, t_p, t_l, self.last_sync, self.norms, self.scores,
                                   stages)

    def merge(self, theta_g_new, hyper=None):
        b = self.bufs
        self.ctx.cocodc_merge(hyper or self.hyper(), b.w_now, b.w_snap, b.now_stride, b.snap_stride,
                              b.snap_offset, theta_g_new, self.ids, self.n_ids)

    def poll(self):
        return self.ctx.cocodc_poll_status()

    def host_state(self):
        """Copies of everything the oracle needs, taken before a GPU call mutates it."""
        b = self.bufs
        return dict(w_now=np_(b.w_now).copy(), w_snap=np_(b.w_snap).copy(), theta_g=np_(b.theta_g).copy(),
                    momentum=np_(b.momentum).copy(), last_sync=np_(self.last_sync).copy(),
                    snap_offset=None if b.snap_offset is None else np_(b.snap_offset).copy(),
                    scores=np_(self.scores).copy(), norms=np_(self.norms).copy())


def check_step_against_oracle(prob: GpuProblem, before: dict, ids, t_p, t_l, ohp: orc.Hyper,
                              delta_out=None, do_merge=True, same=False, check_scores=True):
    """Compare the GPU buffers after cocodc_outer_step with the oracle run on `before`."""
    w = prob.w
    frs = fragments_of(w)
    snap = before["w_now"] if same else before["w_snap"]
    res, new_last = orc.outer_step(frs, ohp, before["w_now"], snap, before["theta_g"], before["momentum"],
                                   ids, t_p, t_l, before["last_sync"],
                                   snap_offset=None if same else before["snap_offset"], do_merge=do_merge)
    after = prob.host_state()
    touched = touched_mask(w, ids)
    # what was not listed must be bit-identical
    for name in ("theta_g", "momentum"):
        assert np.array_equal(after[name][~touched], before[name][~touched]), f"{name} changed outside ids"
    assert np.array_equal(after["w_now"][:, ~touched], before["w_now"][:, ~touched]), "w_now changed outside ids"
    assert np.array_equal(after["w_snap"], before["w_snap"]) or same, "w_snap was written"
    if not do_merge:
        assert np.array_equal(after["w_now"], before["w_now"])
    worst = 0.0
    for p in ids:
        r = res[int(p)]
        g = orc.gather_fragment(frs, after["theta_g"], p)
        u = orc.gather_fragment(frs, after["momentum"], p)
        fl_d = fl_u = fl_g = fl_b = None
        # the operand floors are a contract for test partitions only: none of the named workloads may reach them
        assert g.size >= SMALL_FRAGMENT or w.name not in synth.WORKLOAD_NAMES, (w.name, p, g.size)
        if g.size < SMALL_FRAGMENT:
            fl_d, fl_u, fl_g, fl_b = operand_floors(frs, before, snap, None if same else before["snap_offset"],
                                                    int(p), ohp.momentum)
        worst = max(worst, *assert_close(g, r.theta_g, TOL_PARAM, f"theta_g[{p}]", floor=fl_g))
        worst = max(worst, *assert_close(u, r.momentum, TOL_PARAM, f"momentum[{p}]", floor=fl_u))
        if do_merge:
            wn = orc.gather_fragment(frs, after["w_now"], p)
            for m in range(w.M):
                worst = max(worst, *assert_close(wn[m], r.w_now[m], TOL_PARAM, f"w_now[{m}][{p}]",
                                                 floor=None if fl_b is None else fl_b[m]))
        if delta_out is not None:
            d = orc.gather_fragment(frs, np_(delta_out), p)
            assert_close(d, r.delta_g, TOL_PARAM, f"delta_g[{p}]", floor=fl_d)
        if check_scores:
            assert abs(after["norms"][p] - r.norm) <= TOL_NORM * r.norm, (p, after["norms"][p], r.norm)
            assert abs(after["scores"][p] - r.score) <= TOL_NORM * r.score, (p, after["scores"][p], r.score)
    if check_scores:
        assert np.array_equal(after["last_sync"], new_last)
        rest = np.ones(w.K, dtype=bool)
        rest[list(ids)] = False
        assert np.array_equal(after["scores"][rest], before["scores"][rest])
    return worst


class Guarded:
    """A tensor carved out of a larger allocation with canary words on both sides."""

    PAD = 64

    def __init__(self, shape, dtype, device, fill=None):
        n = int(np.prod(shape))
        self.raw = torch.empty(n + 2 * self.PAD, dtype=dtype, device=device)
        self.canary = 12345.0 if dtype.is_floating_point else 77
        self.raw.fill_(self.canary)
        self.t = self.raw[self.PAD:self.PAD + n].view(*shape)
        if fill is not None:
            self.t.copy_(fill)

    def intact(self) -> bool:
        lo = self.raw[:self.PAD]
        hi = self.raw[-self.PAD:]
        return bool((lo == self.canary).all() and (hi == self.canary).all())


# --------------------------------------------------------------------------
# full-size workloads: sampled element parity + whole-fragment norms
# --------------------------------------------------------------------------

def _fragment_index_maps(w: synth.Workload, p: int, rel: np.ndarray, snap_offset):
    """Map positions inside fragment p (segments concatenated) to native and snapshot element indices."""
    segs = w.partition.fragments[p]
    starts = np.cumsum([0] + [l for _, l in segs])
    which = np.searchsorted(starts, rel, side="right") - 1
    native = np.array([segs[k][0] for k in which], dtype=np.int64) + (rel - starts[which])
    snap = native if snap_offset is None else int(snap_offset[p]) + rel
    return native, snap


def sample_positions(n: int, rng, n_random=100_000, edge=5000, tile=2048) -> np.ndarray:
    parts = [np.arange(0, min(edge, n)), np.arange(max(0, n - edge), n),
             rng.integers(0, n, size=min(n_random, n))]
    for t in rng.integers(0, max(1, n // tile), size=8):
        lo = int(t) * tile
        parts.append(np.arange(max(0, lo - 8), min(n, lo + 8)))
    return np.unique(np.concatenate(parts)).astype(np.int64)


class SampledCheck:
    """Gathers the inputs of sampled elements before a step, and checks the outputs afterwards."""

    def __init__(self, prob: GpuProblem, ids, seed=0, same=False, n_random=100_000, edge=5000):
        self.prob, self.ids, self.same = prob, [int(p) for p in ids], same
        w, b = prob.w, prob.bufs
        rng = np.random.default_rng(seed)
        so = None if (b.snap_offset is None or same) else np_(b.snap_offset)
        self.maps = {}
        self.inputs = {}
        dev = prob.dev
        for p in self.ids:
            rel = sample_positions(w.partition.frag_size(p), rng, n_random=n_random, edge=edge)
            native, snap = _fragment_index_maps(w, p, rel, so)
            ni = torch.from_numpy(native).to(dev)
            si = torch.from_numpy(snap).to(dev)
            src_snap = b.w_now if same else b.w_snap
            self.maps[p] = (ni, si)
            self.inputs[p] = dict(
                w_now=np_(b.w_now.index_select(1, ni)), w_snap=np_(src_snap.index_select(1, si)),
                theta_g=np_(b.theta_g.index_select(0, ni)), momentum=np_(b.momentum.index_select(0, ni)))
        self.last_sync = np_(prob.last_sync).copy()

    def check(self, t_p, t_l, ohp: orc.Hyper, delta_out=None):
        b = self.prob.bufs
        worst = 0.0
        for p in self.ids:
            x = self.inputs[p]
            n = x["theta_g"].shape[0]
            res, _ = orc.outer_step([[(0, n)]], ohp, x["w_now"], x["w_snap"], x["theta_g"], x["momentum"], [0],
                                    t_p, t_l, [int(self.last_sync[p])])
            r = res[0]
            ni, _ = self.maps[p]
            worst = max(worst, *assert_close(np_(b.theta_g.index_select(0, ni)), r.theta_g, TOL_PARAM, f"theta_g[{p}]"))
            worst = max(worst, *assert_close(np_(b.momentum.index_select(0, ni)), r.momentum, TOL_PARAM, f"momentum[{p}]"))
            got = np_(b.w_now.index_select(1, ni))
            for m in range(self.prob.w.M):
                worst = max(worst, *assert_close(got[m], r.w_now[m], TOL_PARAM, f"w_now[{m}][{p}]"))
            if delta_out is not None:
                assert_close(np_(delta_out.index_select(0, ni)), r.delta_g, TOL_PARAM, f"delta_g[{p}]")
        return worst


def fragment_checksums(w: synth.Workload, t: torch.Tensor) -> np.ndarray:
    """Wrap-around integer checksum of every fragment of an [N] or [M, N] fp32 tensor (bit-exactness probe)."""
    out = np.zeros(w.K, dtype=np.int64)
    ti = t.view(torch.int32)
    for p in range(w.K):
        s = 0
        for off, ln in w.partition.fragments[p]:
            s += int(ti[..., off:off + ln].sum(dtype=torch.int64).item())
        out[p] = s
    return out


def oracle_fragment_norm(prob: GpuProblem, p: int, theta_g_before: torch.Tensor = None) -> float:
    """||Delta theta^g_p|| from the oracle on a whole fragment (inputs copied to the host).

    Must be called BEFORE the step (it reads theta_g and w_snap as they are)."""
    w, b = prob.w, prob.bufs
    segs = w.partition.fragments[p]
    n = w.partition.frag_size(p)
    thg = np.concatenate([np_(b.theta_g[o:o + l]) for o, l in segs])
    if b.snap_offset is None:
        snap = np.concatenate([np_(b.w_snap[:, o:o + l]) for o, l in segs], axis=1)
    else:
        so = int(b.snap_offset[p].item())
        snap = np_(b.w_snap[:, so:so + n])
    snap = np.ascontiguousarray(snap)
    zeros = np.zeros(n, dtype=np.float32)
    hp = orc_hyper(w)
    res, _ = orc.outer_step([[(0, n)]], hp, snap, snap, thg, zeros, [0], 1, 1, [0], do_merge=False,
                            threads=host_cores())
    return res[0].norm


# --------------------------------------------------------------------------
# full-size workloads: whole fragments, element by element, streamed through the oracle one at a time
# --------------------------------------------------------------------------

def host_cores() -> int:
    import os
    return len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)


def _gather_fragment_to_host(w: synth.Workload, t: torch.Tensor, p: int, base=None) -> np.ndarray:
    """Fragment p of an [N] or [M, N] device tensor as one contiguous host array (segments concatenated);
    `base`: the fragment sits packed at this element offset instead of at its native offsets."""
    if base is not None:
        n = w.partition.frag_size(p)
        return np.ascontiguousarray(np_(t[..., base:base + n]))
    return np.ascontiguousarray(np.concatenate([np_(t[..., o:o + l]) for o, l in w.partition.fragments[p]], axis=-1))


class FullFragmentCheck:
    """Element-by-element parity on whole fragments of a workload too large to copy to the host at once.

    Before the step: the inputs of every listed fragment are copied to the host.  After it: fragment by fragment
    the oracle runs on those inputs (element range split over the host cores) and every output element of the
    GPU is compared with it; the oracle's norm and score of the whole fragment are compared too."""

    def __init__(self, prob: GpuProblem, ids):
        self.prob, self.ids = prob, [int(p) for p in ids]
        w, b = prob.w, prob.bufs
        so = None if b.snap_offset is None else np_(b.snap_offset)
        self.inputs = {}
        for p in self.ids:
            self.inputs[p] = dict(
                w_now=_gather_fragment_to_host(w, b.w_now, p),
                w_snap=_gather_fragment_to_host(w, b.w_snap, p, None if so is None else int(so[p])),
                theta_g=_gather_fragment_to_host(w, b.theta_g, p),
                momentum=_gather_fragment_to_host(w, b.momentum, p))
        self.last_sync = np_(prob.last_sync).copy()

    def check(self, t_p, t_l, ohp: orc.Hyper):
        prob = self.prob
        w, b = prob.w, prob.bufs
        norms, scores = np_(prob.norms), np_(prob.scores)
        worst = 0.0
        threads = host_cores()
        for p in self.ids:
            assert w.partition.frag_size(p) >= SMALL_FRAGMENT
            x = self.inputs.pop(p)
            n = x["theta_g"].shape[0]
            res, _ = orc.outer_step([[(0, n)]], ohp, x["w_now"], x["w_snap"], x["theta_g"], x["momentum"], [0],
                                    t_p, t_l, [int(self.last_sync[p])], threads=threads)
            r = res[0]
            del x
            worst = max(worst, *assert_close(_gather_fragment_to_host(w, b.theta_g, p), r.theta_g, TOL_PARAM,
                                             f"theta_g[{p}]"))
            worst = max(worst, *assert_close(_gather_fragment_to_host(w, b.momentum, p), r.momentum, TOL_PARAM,
                                             f"momentum[{p}]"))
            got = _gather_fragment_to_host(w, b.w_now, p)
            for m in range(w.M):
                worst = max(worst, *assert_close(got[m], r.w_now[m], TOL_PARAM, f"w_now[{m}][{p}]"))
            assert abs(norms[p] - r.norm) <= TOL_NORM * r.norm, (p, norms[p], r.norm)
            assert abs(scores[p] - r.score) <= TOL_NORM * r.score, (p, scores[p], r.score)
            del res, r, got
        return worst
