"""Worker-per-device deployment (Section 2.1): pseudo-gradient sums per device, all-reduced, then the
completion from the received sum.  One GPU stands in for the devices one after the other (no kernel waits
on another); the cross-rank part is torch.distributed's all-reduce."""

import os
import socket

import numpy as np
import pytest
import torch

import synth
from oracle import reference as orc
from helpers import (GpuProblem, TOL_NORM, TOL_PARAM, assert_close, fragments_of, np_, orc_hyper)
from test_gpu_parity_small import RAGGED

pytestmark = pytest.mark.gpu


def make(M, seed, **kw):
    w = synth.small_workload(RAGGED, M=M, seed=seed, scale_kind="loguniform")
    return GpuProblem(w, synth.generate(w, "cuda", momentum_sigma=1e-3, **kw))


@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 8])
def test_two_phase_on_one_device_is_bit_identical_to_the_fused_step(M):
    a = make(M, seed=200 + M)
    b = make(M, seed=200 + M)
    ids = [4, 0, 2, 1]
    for prob in (a, b):
        prob.set_ids(ids)
    da = torch.zeros(a.w.N, device="cuda")
    a.outer_step(6, 9, delta_out=da)
    before = b.host_state()
    sum_buf = torch.full((b.w.N,), 7.0, device="cuda")
    bb = b.bufs
    b.ctx.cocodc_pseudo_gradient_sum(bb.w_snap, bb.snap_stride, None, bb.theta_g, M, sum_buf, b.ids, b.n_ids)
    # phase one against the oracle, and nothing outside the listed fragments written
    exp = orc.pseudo_gradient_sum(fragments_of(b.w), M, before["w_snap"], before["theta_g"], ids)
    got = np_(sum_buf)
    touched = np.zeros(b.w.N, dtype=bool)
    for p in ids:
        assert_close(orc.gather_fragment(fragments_of(b.w), got, p), exp[p], TOL_PARAM, f"sum[{p}]")
        for o, l in b.w.partition.fragments[p]:
            touched[o:o + l] = True
    assert np.all(got[~touched] == 7.0)
    b.ctx.cocodc_outer_step_received(b.hyper(), M, bb.w_now, bb.w_snap, bb.now_stride, bb.snap_stride, None,
                                     bb.theta_g, bb.momentum, sum_buf, sum_buf, b.ids, b.n_ids, 6, 9,
                                     b.last_sync, b.norms, b.scores)
    assert b.poll() == 0
    for x, y in ((a.bufs.w_now, bb.w_now), (a.bufs.theta_g, bb.theta_g), (a.bufs.momentum, bb.momentum),
                 (a.scores, b.scores), (a.norms, b.norms), (a.last_sync, b.last_sync)):
        assert torch.equal(x, y)
    t = torch.from_numpy(touched).cuda()
    assert torch.equal(da[t], sum_buf[t])                      # delta written in place of the received sum


def test_two_devices_with_two_workers_each():
    """Workers 0-1 on one device, 2-3 on another, replicated outer state; the sums are added as an all-reduce would."""
    full = make(4, seed=210, snap_layout="pool", pool_ids=[3, 1, 0])
    w = full.w
    frs = fragments_of(w)
    ids = [1, 3, 0]
    before = full.host_state()
    devs = []
    for d in range(2):
        w2 = w.with_(M=2)
        bufs = synth.DeviceBuffers(theta_g=full.bufs.theta_g.clone(), momentum=full.bufs.momentum.clone(),
                                   w_now=full.bufs.w_now[2 * d:2 * d + 2].clone(),
                                   w_snap=full.bufs.w_snap[2 * d:2 * d + 2].clone(),
                                   snap_offset=full.bufs.snap_offset.clone(), scales=full.bufs.scales)
        prob = GpuProblem(w2, bufs)
        prob.set_ids(ids)
        prob.sum = torch.zeros(w.N, device="cuda")
        b = prob.bufs
        prob.ctx.cocodc_pseudo_gradient_sum(b.w_snap, b.snap_stride, b.snap_offset, b.theta_g, 2, prob.sum,
                                            prob.ids, prob.n_ids)
        devs.append(prob)
    total = devs[0].sum + devs[1].sum                         # what the all-reduce delivers to both
    ohp = orc_hyper(w)
    for d, prob in enumerate(devs):
        b = prob.bufs
        prob.ctx.cocodc_outer_step_received(prob.hyper(), 4, b.w_now, b.w_snap, b.now_stride, b.snap_stride,
                                            b.snap_offset, b.theta_g, b.momentum, total, None, prob.ids, prob.n_ids,
                                            8, 10, prob.last_sync, prob.norms, prob.scores)
        assert prob.poll() == 0
        res, new_last = orc.outer_step(frs, orc_hyper(w, M=2), before["w_now"][2 * d:2 * d + 2],
                                       before["w_snap"][2 * d:2 * d + 2], before["theta_g"], before["momentum"], ids,
                                       8, 10, before["last_sync"], snap_offset=before["snap_offset"],
                                       recv_sum=np_(total), M_total=4)
        after = prob.host_state()
        for p in ids:
            r = res[p]
            assert_close(orc.gather_fragment(frs, after["theta_g"], p), r.theta_g, TOL_PARAM, "theta_g")
            assert_close(orc.gather_fragment(frs, after["momentum"], p), r.momentum, TOL_PARAM, "momentum")
            wn = orc.gather_fragment(frs, after["w_now"], p)
            for m in range(2):
                assert_close(wn[m], r.w_now[m], TOL_PARAM, f"w_now[{m}]")
            assert abs(after["norms"][p] - r.norm) <= TOL_NORM * r.norm
        assert np.array_equal(after["last_sync"], new_last)
    # the replicated state stays identical on both devices, bit for bit
    for k in ("theta_g", "momentum"):
        assert torch.equal(getattr(devs[0].bufs, k), getattr(devs[1].bufs, k))
    assert torch.equal(devs[0].scores, devs[1].scores)
    # and agrees with all four workers stacked on one device
    full.set_ids(ids)
    full.outer_step(8, 10)
    assert_close(np_(devs[0].bufs.theta_g), np_(full.bufs.theta_g).astype(np.float64), TOL_PARAM, "vs stacked")


@pytest.mark.parametrize("R,M_local", [(1, 2), (2, 1), (2, 2), (3, 1), (4, 1), (4, 4), (8, 1), (8, 3), (2, 5)])
def test_partial_sums_added_inside_the_step(R, M_local):
    """R devices' partial sums handed to the step as R buffers (on a deployment: the peers' mapped memory; here R
    buffers of one GPU).  Against the oracle's total of the partial sums, and bit for bit against the single-buffer
    entry point fed the same left-to-right fp32 sum."""
    M_total = R * M_local
    full = make(M_total, seed=300 + 10 * R + M_local, snap_layout="pool", pool_ids=[2, 4, 0])
    w, frs, ids = full.w, fragments_of(full.w), [4, 0, 2]
    before = full.host_state()
    w_loc = w.with_(M=M_local)
    sums = []
    for d in range(R):                      # phase one on every "device": its local workers' pseudo-gradient sum
        rows = slice(d * M_local, (d + 1) * M_local)
        prob = GpuProblem(w_loc, synth.DeviceBuffers(theta_g=full.bufs.theta_g, momentum=full.bufs.momentum,
                                                     w_now=full.bufs.w_now[rows], w_snap=full.bufs.w_snap[rows],
                                                     snap_offset=full.bufs.snap_offset, scales=full.bufs.scales))
        prob.set_ids(ids)
        buf = torch.zeros(w.N, device="cuda")
        b = prob.bufs
        prob.ctx.cocodc_pseudo_gradient_sum(b.w_snap, full.bufs.snap_stride, b.snap_offset, b.theta_g, M_local, buf,
                                            prob.ids, prob.n_ids)
        sums.append(buf)
    total = sums[0].clone()
    for x in sums[1:]:
        total += x                           # fp32, left to right: what the kernel does
    out = {}
    for which in ("peers", "single"):        # device 0 completes, once per entry point, from identical state
        rows = slice(0, M_local)
        bufs = synth.DeviceBuffers(theta_g=full.bufs.theta_g.clone(), momentum=full.bufs.momentum.clone(),
                                   w_now=full.bufs.w_now[rows].clone(), w_snap=full.bufs.w_snap[rows].clone(),
                                   snap_offset=full.bufs.snap_offset.clone(), scales=full.bufs.scales)
        prob = GpuProblem(w_loc, bufs)
        prob.set_ids(ids)
        b = prob.bufs
        delta = torch.zeros(w.N, device="cuda")
        args = (b.w_now, b.w_snap, b.now_stride, b.snap_stride, b.snap_offset, b.theta_g, b.momentum)
        tail = (delta, prob.ids, prob.n_ids, 8, 10, prob.last_sync, prob.norms, prob.scores)
        if which == "peers":
            prob.ctx.cocodc_outer_step_received_peers(prob.hyper(), M_total, *args, sums, *tail)
        else:
            prob.ctx.cocodc_outer_step_received(prob.hyper(), M_total, *args, total, *tail)
        assert prob.poll() == 0
        out[which] = (prob, delta)
    pp, dp = out["peers"]
    ps, ds = out["single"]
    for x, y in ((pp.bufs.w_now, ps.bufs.w_now), (pp.bufs.theta_g, ps.bufs.theta_g), (pp.bufs.momentum, ps.bufs.momentum),
                 (pp.scores, ps.scores), (pp.norms, ps.norms), (pp.last_sync, ps.last_sync), (dp, ds)):
        assert torch.equal(x, y)
    res, new_last = orc.outer_step(frs, orc_hyper(w, M=M_local), before["w_now"][:M_local], before["w_snap"][:M_local],
                                   before["theta_g"], before["momentum"], ids, 8, 10, before["last_sync"],
                                   snap_offset=before["snap_offset"], recv_sum=[np_(x) for x in sums], M_total=M_total)
    after = pp.host_state()
    for p in ids:
        r = res[p]
        assert_close(orc.gather_fragment(frs, after["theta_g"], p), r.theta_g, TOL_PARAM, "theta_g")
        assert_close(orc.gather_fragment(frs, after["momentum"], p), r.momentum, TOL_PARAM, "momentum")
        assert_close(orc.gather_fragment(frs, np_(dp), p), r.delta_g, TOL_PARAM, "delta_g")
        wn = orc.gather_fragment(frs, after["w_now"], p)
        for m in range(M_local):
            assert_close(wn[m], r.w_now[m], TOL_PARAM, f"w_now[{m}]")
        assert abs(after["norms"][p] - r.norm) <= TOL_NORM * r.norm
    assert np.array_equal(after["last_sync"], new_last)


def test_peer_glue_two_ranks_taken_in_turn():
    """distributed.complete_fragments_peers for two ranks of two workers, run one after the other on one GPU: the
    barrier of the rank that goes first stands in for the other rank's arrival (it runs that rank's phase one)."""
    from paper_2504_17672_b200 import distributed as D
    full = make(4, seed=240)
    w, ids = full.w, [0, 3, 1]
    ranks = []
    for d in range(2):
        bufs = synth.DeviceBuffers(theta_g=full.bufs.theta_g.clone(), momentum=full.bufs.momentum.clone(),
                                   w_now=full.bufs.w_now[2 * d:2 * d + 2].clone(),
                                   w_snap=full.bufs.w_snap[2 * d:2 * d + 2].clone(), snap_offset=None,
                                   scales=full.bufs.scales)
        prob = GpuProblem(w.with_(M=2), bufs)
        prob.set_ids(ids)
        ranks.append(prob)
    sums = [torch.zeros(w.N, device="cuda") for _ in range(2)]
    calls = []

    def barrier_of_rank0():
        calls.append("barrier")
        if len(calls) == 1:                    # the other rank reaches the barrier: its sum is in place
            p1 = ranks[1]
            p1.ctx.cocodc_pseudo_gradient_sum(p1.bufs.w_snap, p1.bufs.snap_stride, None, p1.bufs.theta_g, 2, sums[1],
                                              p1.ids, p1.n_ids)

    for r, prob in enumerate(ranks):
        b = prob.bufs
        D.complete_fragments_peers(prob.ctx, prob.hyper(), 4, r, sums, prob.ids, prob.n_ids, b.w_now, b.w_snap, None,
                                   b.theta_g, b.momentum, 5, 9, prob.last_sync, prob.norms, prob.scores,
                                   barrier_of_rank0 if r == 0 else (lambda: None))
        assert prob.poll() == 0
    assert calls == ["barrier", "barrier"]
    for k in ("theta_g", "momentum"):
        assert torch.equal(getattr(ranks[0].bufs, k), getattr(ranks[1].bufs, k))     # replicated state: same bits
    assert torch.equal(ranks[0].scores, ranks[1].scores)
    full.set_ids(ids)
    full.outer_step(5, 9)
    assert_close(np_(ranks[0].bufs.theta_g), np_(full.bufs.theta_g).astype(np.float64), TOL_PARAM, "vs stacked")
    for d in range(2):
        assert_close(np_(ranks[d].bufs.w_now), np_(full.bufs.w_now[2 * d:2 * d + 2]).astype(np.float64), TOL_PARAM,
                     "w_now vs stacked")


def test_partial_sums_validation():
    prob = make(2, seed=221)
    b, B = prob.bufs, prob.B
    prob.set_ids([0])
    bufs = [torch.zeros(prob.w.N, device="cuda") for _ in range(9)]

    def code(sums, out=None):
        with pytest.raises(B.CocodcError) as e:
            prob.ctx.cocodc_outer_step_received_peers(prob.hyper(), 4, b.w_now, b.w_snap, b.now_stride, b.snap_stride,
                                                      None, b.theta_g, b.momentum, sums, out, prob.ids, prob.n_ids,
                                                      1, 2, prob.last_sync, prob.norms, prob.scores)
        return e.value.code

    assert code([]) == B.ERR_INVALID_ARG
    assert code(bufs) == B.ERR_INVALID_ARG                      # more than the eight buffers a step adds up
    assert code([bufs[0], b.momentum]) == B.ERR_ALIAS
    assert code([bufs[0], bufs[1][1:]]) == B.ERR_ALIGNMENT
    assert code([bufs[0], 0]) == B.ERR_INVALID_ARG              # a null entry
    # in place on one of the listed buffers is allowed
    prob.ctx.cocodc_outer_step_received_peers(prob.hyper(), 4, b.w_now, b.w_snap, b.now_stride, b.snap_stride, None,
                                              b.theta_g, b.momentum, bufs[:2], bufs[1], prob.ids, prob.n_ids, 1, 2,
                                              prob.last_sync, prob.norms, prob.scores)
    assert prob.poll() == 0


def test_received_mode_validation():
    prob = make(2, seed=220)
    b, B = prob.bufs, prob.B
    prob.set_ids([0])
    s = torch.zeros(prob.w.N, device="cuda")

    def code(**kw):
        a = dict(hyper=prob.hyper(), M_total=2, w_now=b.w_now, w_snap=b.w_snap, now_stride=b.now_stride,
                 snap_stride=b.snap_stride, snap_offset=None, theta_g=b.theta_g, momentum=b.momentum, delta_sum=s,
                 delta_g_out=None, ids=prob.ids, n_ids=prob.n_ids, t_p=1, t_l=2, last_sync=prob.last_sync,
                 norms=prob.norms, scores=prob.scores)
        a.update(kw)
        with pytest.raises(B.CocodcError) as e:
            prob.ctx.cocodc_outer_step_received(**a)
        return e.value.code

    assert code(M_total=1) == B.ERR_INVALID_ARG                 # fewer workers in total than held locally
    assert code(delta_sum=None) == B.ERR_INVALID_ARG
    assert code(delta_sum=b.theta_g) == B.ERR_ALIAS
    assert code(w_snap=b.w_now, snap_stride=b.now_stride) == B.ERR_INVALID_ARG   # zero delay is not a two-phase case
    assert code(delta_sum=s[1:]) == B.ERR_ALIGNMENT
    with pytest.raises(B.CocodcError) as e:
        prob.ctx.cocodc_pseudo_gradient_sum(b.w_snap, b.snap_stride, None, b.theta_g, 2, b.theta_g, prob.ids, prob.n_ids)
    assert e.value.code == B.ERR_ALIAS


def test_complete_fragments_through_nccl_world_of_one():
    """The glue (kernel, all-reduce, kernel) on a one-rank NCCL group equals the fused step."""
    import torch.distributed as dist
    from paper_2504_17672_b200 import distributed as D
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        a, b = make(4, seed=230), make(4, seed=230)
        ids = [2, 4, 0]
        for prob in (a, b):
            prob.set_ids(ids)
        a.outer_step(3, 7)
        bb = b.bufs
        sum_buf = torch.zeros(b.w.N, device="cuda")
        D.complete_fragments(b.ctx, b.hyper(), 4, fragments_of(b.w), ids, b.ids, b.n_ids, bb.w_now, bb.w_snap, None,
                             bb.theta_g, bb.momentum, sum_buf, 3, 7, b.last_sync, b.norms, b.scores)
        assert b.poll() == 0
        for x, y in ((a.bufs.w_now, bb.w_now), (a.bufs.theta_g, bb.theta_g), (a.bufs.momentum, bb.momentum),
                     (a.scores, b.scores)):
            assert torch.equal(x, y)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("M_total", [3, 5, 6, 7, 9, 11, 12, 24, 49, 64])
def test_mean_over_workers_is_the_correctly_rounded_quotient(M_total):
    """Eq. 1's division by the worker count never runs a division instruction (its slow path on zero
    numerators costs bandwidth); what it computes must still be the IEEE quotient.  The received-sum step
    exposes the operation directly: Delta = delta_sum / M_total, read back through delta_g_out and compared
    bit for bit with numpy's float32 division on zeros of both signs, huge, tiny and ordinary sums."""
    n = 1 << 16
    w = synth.small_workload([n], M=1, seed=300)
    prob = GpuProblem(w, synth.generate(w, "cuda"))
    prob.set_ids([0])
    rng = np.random.default_rng(M_total)
    s = (rng.standard_normal(n) * np.exp(rng.uniform(-60.0, 60.0, n))).astype(np.float32)
    s[:64] = 0.0
    s[64:128] = -0.0
    s[128:192] = np.float32(M_total) * rng.integers(-1000, 1000, 64).astype(np.float32)   # exact quotients
    s[192:200] = np.float32(3.0e38)
    sums = torch.from_numpy(s).cuda()
    delta = torch.full((n,), 5.0, device="cuda")
    b = prob.bufs
    prob.ctx.cocodc_outer_step_received(prob.hyper(), M_total, b.w_now, b.w_snap, b.now_stride, b.snap_stride, None,
                                        b.theta_g, b.momentum, sums, delta, prob.ids, prob.n_ids, 3, 5,
                                        prob.last_sync, prob.norms, prob.scores)
    prob.poll()                              # sums of 1e38 make the fragment norm overflow: not what is tested here
    want = s / np.float32(M_total)
    got = np_(delta)
    assert got.dtype == np.float32 and want.dtype == np.float32
    bad = np.flatnonzero(got.view(np.uint32) != want.view(np.uint32))
    assert bad.size == 0, (bad[:8], s[bad[:8]], got[bad[:8]], want[bad[:8]])
