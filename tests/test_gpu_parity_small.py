"""GPU-vs-oracle parity of the outer step on small problems that still span several tiles,
ragged edges, odd offsets, every worker count path, every mode, and both snapshot layouts."""

import numpy as np
import pytest
import torch

import synth
from oracle import reference as orc
from helpers import (GpuProblem, Guarded, assert_close, check_step_against_oracle, fragments_of, np_,
                     orc_hyper, touched_mask, TOL_PARAM)

pytestmark = pytest.mark.gpu

# several tiles per fragment (a tile is 2048 elements at M <= 4), odd sizes, odd offsets, gaps, a strided fragment
RAGGED = (60_000, [[(3, 9_001), (40_010, 4_097)], [(9_004, 12_345)], [(21_349, 5)], [(21_360, 18_640)],
                   [(44_111, 15_000)]])


def make(M, seed=0, frs=RAGGED, snap_layout="full", pool_ids=None, pool_offsets=None, **kw):
    w = synth.small_workload(frs, M=M, seed=seed, scale_kind="loguniform", **kw)
    bufs = synth.generate(w, "cuda", snap_layout=snap_layout, pool_ids=pool_ids, pool_offsets=pool_offsets,
                          momentum_sigma=1e-3)
    return GpuProblem(w, bufs)


@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 8])
def test_fused_step_all_worker_counts(M):
    prob = make(M, seed=M)
    ids = [3, 0, 2, 4]
    prob.set_ids(ids)
    before = prob.host_state()
    delta = torch.full((prob.w.N,), 7.0, dtype=torch.float32, device="cuda")
    prob.outer_step(t_p=10, t_l=12, delta_out=delta)
    assert prob.poll() == 0
    check_step_against_oracle(prob, before, ids, 10, 12, orc_hyper(prob.w), delta_out=delta)
    assert bool((delta[torch.from_numpy(~touched_mask(prob.w, ids)).cuda()] == 7.0).all())


@pytest.mark.parametrize("sign", [0, 1, 2])
@pytest.mark.parametrize("alpha", [1.0, 0.5, 0.0])
def test_sign_modes_and_mixing(sign, alpha):
    prob = make(4, seed=20 + sign, tau=4, lam=1.0)
    ids = [1, 4]
    prob.set_ids(ids)
    before = prob.host_state()
    prob.outer_step(5, 9, hyper=prob.hyper(sign_mode=sign, alpha=alpha))
    check_step_against_oracle(prob, before, ids, 5, 9, orc_hyper(prob.w, sign_mode=sign, alpha=alpha))


def test_no_compensation_is_streaming_diloco():
    prob = make(4, seed=30)
    ids = [0, 1, 2, 3, 4]
    prob.set_ids(ids)
    before = prob.host_state()
    prob.outer_step(5, 7, hyper=prob.hyper(comp_mode=0, alpha=0.25))
    check_step_against_oracle(prob, before, ids, 5, 7, orc_hyper(prob.w, comp_mode=orc.COMP_NONE, alpha=0.25))


@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 6, 7, 8, 9])
def test_zero_delay_blocking_sync(M):
    """w_snap == w_now: the DiLoCo case; every worker leaves with the new global state."""
    prob = make(M, seed=40)
    ids = [4, 0]
    prob.set_ids(ids)
    before = prob.host_state()
    prob.outer_step(100, 100, hyper=prob.hyper(tau=0), w_snap=prob.bufs.w_now)
    check_step_against_oracle(prob, before, ids, 100, 100, orc_hyper(prob.w, tau=0), same=True)
    g = np_(prob.bufs.theta_g)
    wn = np_(prob.bufs.w_now)
    t = touched_mask(prob.w, ids)
    for m in range(M):
        assert np.array_equal(wn[m][t], g[t])


def test_three_consecutive_steps_carry_momentum():
    prob = make(4, seed=50)
    rng = np.random.default_rng(0)
    ids = [0, 1, 3]
    for step in range(3):
        prob.set_ids(ids)
        before = prob.host_state()
        prob.outer_step(10 * step + 5, 10 * step + 7)
        check_step_against_oracle(prob, before, ids, 10 * step + 5, 10 * step + 7, orc_hyper(prob.w))
        # local training moves on: new snapshot = current, then drift
        prob.snapshot()
        prob.bufs.w_now.add_(torch.randn_like(prob.bufs.w_now) * 1e-3)
    assert prob.poll() == 0


@pytest.mark.parametrize("M", [1, 2, 3, 4, 6])
def test_unfused_path_equals_fused_bit_for_bit(M):
    """S1-S3 + S6 and S4-S5 as two calls.  The halves read few streams at small M and then run with wider
    tiles than the fused step (4 or 2 tiles per stage), so this also covers those instances."""
    a = make(M, seed=60)
    b = make(M, seed=60)
    ids = [2, 1, 4]
    for prob in (a, b):
        prob.set_ids(ids)
    a.outer_step(3, 5)
    before = b.host_state()
    b.outer_step(3, 5, stages=1 | 4)          # S1-S3 + S6
    check_step_against_oracle(b, before, ids, 3, 5, orc_hyper(b.w), do_merge=False)
    b.merge(b.bufs.theta_g)                    # S4-S5
    for x, y in ((a.bufs.w_now, b.bufs.w_now), (a.bufs.theta_g, b.bufs.theta_g), (a.bufs.momentum, b.bufs.momentum),
                 (a.scores, b.scores), (a.norms, b.norms)):
        assert torch.equal(x, y)
    # merge alone against the oracle
    res = orc.merge(fragments_of(b.w), orc_hyper(b.w), before["w_now"], before["w_snap"],
                    np_(a.bufs.theta_g), ids)
    for p in ids:
        got = orc.gather_fragment(fragments_of(b.w), np_(b.bufs.w_now), p)
        assert_close(got, res[p], TOL_PARAM, f"merge[{p}]")
    # the merge with zero delay (the recorded values are the current ones): Eq. 3 towards the new global state
    before = b.host_state()
    hp = b.hyper(alpha=0.5, comp_mode=0, tau=0)
    bb = b.bufs
    b.ctx.cocodc_merge(hp, bb.w_now, bb.w_now, bb.now_stride, bb.now_stride, None, bb.theta_g, b.ids, b.n_ids)
    assert b.poll() == 0
    res = orc.merge(fragments_of(b.w), orc_hyper(b.w, alpha=0.5, comp_mode=0, tau=0), before["w_now"],
                    before["w_now"], before["theta_g"], ids)
    after = np_(bb.w_now)
    for p in ids:
        assert_close(orc.gather_fragment(fragments_of(b.w), after, p), res[p], TOL_PARAM, f"zero-delay merge[{p}]")
    untouched = ~touched_mask(b.w, ids)
    assert np.array_equal(after[:, untouched], before["w_now"][:, untouched])


@pytest.mark.parametrize("aligned", [True, False])
def test_snapshot_pool_layouts(aligned):
    """Snapshots packed in a pool: 16-byte-compatible offsets take the vector path, others the scalar one."""
    pool_offsets = None if aligned else {4: 1, 0: 15_002, 1: 28_103}
    prob = make(4, seed=70, snap_layout="pool", pool_ids=[4, 0, 1], pool_offsets=pool_offsets)
    ids = [0, 4, 1]
    prob.set_ids(ids)
    before = prob.host_state()
    prob.outer_step(8, 11)
    assert prob.poll() == 0
    check_step_against_oracle(prob, before, ids, 8, 11, orc_hyper(prob.w))
    # a fragment without a pool slot is refused on the device and nothing is touched
    prob.set_ids([0, 2])
    before = prob.host_state()
    prob.outer_step(12, 13)
    assert prob.poll() == prob.B.ERR_INVALID_ARG
    after = prob.host_state()
    for k in ("w_now", "theta_g", "momentum", "last_sync"):
        assert np.array_equal(before[k], after[k])
    # a placement that would run past the end of a pool row is refused too (no out-of-bounds read or write)
    prob.set_ids([1])
    prob.bufs.snap_offset[1] = prob.bufs.w_snap.shape[1] - 100
    prob.outer_step(12, 13)
    assert prob.poll() == prob.B.ERR_INVALID_ARG
    prob.snapshot()
    assert prob.poll() == prob.B.ERR_INVALID_ARG
    after = prob.host_state()
    for k in ("w_now", "w_snap", "theta_g", "momentum", "last_sync"):
        assert np.array_equal(before[k], after[k])


def test_snapshot_kernel_copies_exactly_the_listed_fragments():
    for layout, pool_ids in (("full", None), ("pool", [1, 3, 0])):
        prob = make(3, seed=80, snap_layout=layout, pool_ids=pool_ids)
        ids = [3, 0]
        prob.set_ids(ids)
        before = prob.host_state()
        prob.snapshot()
        assert prob.poll() == 0
        exp = orc.snapshot(fragments_of(prob.w), before["w_now"], ids, 3, before["snap_offset"], before["w_snap"])
        assert np.array_equal(np_(prob.bufs.w_snap), exp)
        assert np.array_equal(np_(prob.bufs.w_now), before["w_now"])


def test_guard_bands_and_untouched_memory():
    """Canary words around every buffer survive; sizes are chosen so the last tile is ragged."""
    w = synth.small_workload([4099, 2048, 1, 6000], M=4, seed=90)
    bufs = synth.generate(w, "cuda", momentum_sigma=1e-3)
    g = {k: Guarded(getattr(bufs, k).shape, torch.float32, "cuda", fill=getattr(bufs, k))
         for k in ("theta_g", "momentum", "w_now", "w_snap")}
    for k, v in g.items():
        setattr(bufs, k, v.t)
    prob = GpuProblem(w, bufs)
    gd = Guarded((w.N,), torch.float32, "cuda")
    ids = [0, 2, 3]
    prob.set_ids(ids)
    before = prob.host_state()
    prob.outer_step(1, 2, delta_out=gd.t)
    prob.snapshot()
    assert prob.poll() == 0
    assert all(v.intact() for v in g.values()) and gd.intact()
    prob.bufs.w_snap.copy_(torch.from_numpy(before["w_snap"]).cuda())
    check_step_against_oracle(prob, before, ids, 1, 2, orc_hyper(w), delta_out=gd.t)


def test_device_side_id_validation():
    prob = make(2, seed=100)
    before = prob.host_state()
    for bad in ([0, 0], [5], [-1], [0, 1, 2, 3, 4, 4]):
        prob.ids.fill_(-1)
        prob.ids[:len(bad)] = torch.tensor(bad[:prob.w.K], dtype=torch.int32, device="cuda")
        prob.n_ids.fill_(len(bad))
        prob.outer_step(1, 2)
        assert prob.poll() == prob.B.ERR_INVALID_ARG, bad
    after = prob.host_state()
    for k in ("w_now", "theta_g", "momentum", "last_sync", "scores"):
        assert np.array_equal(before[k], after[k], equal_nan=True)
    # an empty list is legal and does nothing
    prob.set_ids([])
    prob.outer_step(1, 2)
    assert prob.poll() == 0
    assert np.array_equal(prob.host_state()["w_now"], before["w_now"])


def test_host_validation_errors():
    prob = make(2, seed=110)
    B, b = prob.B, prob.bufs
    prob.set_ids([0])

    def call(**kw):
        a = dict(hyper=prob.hyper(), w_now=b.w_now, w_snap=b.w_snap, now_stride=b.now_stride,
                 snap_stride=b.snap_stride, snap_offset=None, theta_g=b.theta_g, momentum=b.momentum,
                 delta_g_out=None, ids=prob.ids, n_ids=prob.n_ids, t_p=1, t_l=2, last_sync=prob.last_sync,
                 norms=prob.norms, scores=prob.scores, stages=7)
        a.update(kw)
        prob.ctx.cocodc_outer_step(**a)

    def code(**kw):
        with pytest.raises(B.CocodcError) as e:
            call(**kw)
        return e.value.code

    assert code(theta_g=b.momentum) == B.ERR_ALIAS
    assert code(delta_g_out=b.w_now[1]) == B.ERR_ALIAS
    assert code(w_snap=b.w_now[:, 4:], snap_stride=b.now_stride) in (B.ERR_ALIAS, B.ERR_INVALID_ARG)
    assert code(theta_g=b.theta_g[1:]) == B.ERR_ALIGNMENT
    assert code(now_stride=b.now_stride + 2) == B.ERR_ALIGNMENT
    assert code(hyper=prob.hyper(M=3)) == B.ERR_INVALID_ARG          # beyond max_M of the context
    assert code(hyper=prob.hyper(H=0)) == B.ERR_INVALID_ARG
    assert code(hyper=prob.hyper(tau=0)) == B.ERR_INVALID_ARG        # Eq. 4 divides by tau
    assert code(hyper=prob.hyper(sign_mode=3)) == B.ERR_INVALID_ARG
    assert code(stages=2) == B.ERR_INVALID_ARG
    assert code(ids=None) == B.ERR_INVALID_ARG
    assert code(t_p=5, t_l=4) == B.ERR_INVALID_ARG
    assert code(stages=1 | 2 | 8) == B.ERR_INVALID_ARG               # sums asked for without a place for them
    assert code(stages=16 | 1) == B.ERR_INVALID_ARG
    call(hyper=prob.hyper(tau=0, comp_mode=0))                        # legal: no compensation
    assert prob.poll() == 0

    # the other new calls
    K = prob.w.K
    sq = torch.zeros(K, dtype=torch.float64, device="cuda")
    ctx = prob.ctx

    def raises(fn, *a, **kw):
        with pytest.raises(B.CocodcError) as e:
            fn(*a, **kw)
        return e.value.code

    assert raises(ctx.cocodc_scores_from_sumsq, None, prob.ids, prob.n_ids, None, 1, 2, prob.last_sync, prob.norms,
                  prob.scores) == B.ERR_INVALID_ARG
    assert raises(ctx.cocodc_scores_from_sumsq, sq, prob.ids, None, None, 1, 2, prob.last_sync, prob.norms,
                  prob.scores) == B.ERR_INVALID_ARG              # a list without its length
    assert raises(ctx.cocodc_scores_from_sumsq, sq, prob.ids, prob.n_ids, None, 3, 2, prob.last_sync, prob.norms,
                  prob.scores) == B.ERR_INVALID_ARG              # completes before it was initiated
    assert raises(ctx.cocodc_scores_from_sumsq, sq, prob.ids, prob.n_ids, prob.last_sync, 1, 2, prob.last_sync,
                  prob.norms, prob.scores) == B.ERR_INVALID_ARG  # intervals belong to the stand-alone form
    assert raises(ctx.cocodc_fragment_scores, b.theta_g, None, prob.norms, None) == B.ERR_INVALID_ARG
    assert raises(ctx.cocodc_fragment_scores, b.theta_g, None, None, None) == B.ERR_INVALID_ARG

    def initiate(**kw):
        a = dict(scores=prob.scores, last_sync=prob.last_sync, ineligible=None, t_now=5, H=100, budget_kind=0,
                 budget=1, mask=prob.mask, ids=prob.ids, n_sel=prob.n_ids, pool_offset=None, w_now=b.w_now,
                 w_snap=b.w_snap, now_stride=b.now_stride, snap_stride=b.snap_stride, M=2)
        a.update(kw)
        return raises(ctx.cocodc_initiate, **a)

    assert initiate(w_snap=b.w_now) == B.ERR_ALIAS
    assert initiate(now_stride=b.now_stride + 2) == B.ERR_ALIGNMENT
    assert initiate(w_now=b.w_now.view(-1)[1:]) == B.ERR_ALIGNMENT
    assert initiate(M=3) == B.ERR_INVALID_ARG
    assert initiate(budget_kind=7) == B.ERR_INVALID_ARG
    assert initiate(H=0) == B.ERR_INVALID_ARG
    assert initiate(mask=None) == B.ERR_INVALID_ARG
    assert prob.poll() == 0


def test_nonfinite_norm_is_reported():
    prob = make(2, seed=120)
    prob.bufs.w_snap[0, 100] = float("inf")
    prob.set_ids([0])
    prob.outer_step(1, 2)
    assert prob.poll() == prob.B.ERR_NONFINITE
    assert prob.poll() == 0


@pytest.mark.parametrize("M", [4, 1])
@pytest.mark.parametrize("same", [False, True])
def test_host_buffer_entry_point_matches_device_path_and_oracle(same, M):
    """Parameters in host memory, streamed through a small workspace (several chunks per fragment).  M = 1 runs
    the staged kernel with two tiles per stage, so the chunk plans are built for that tile as well."""
    frs = (300_000, [[(3, 90_001), (200_010, 40_097)], [(90_004, 100_000)], [(250_000, 50_000)]])
    w = synth.small_workload(frs, M=M, seed=130, scale_kind="loguniform")
    bufs = synth.generate(w, "cuda", momentum_sigma=1e-3)
    prob = GpuProblem(w, bufs)
    ids = [2, 0]
    prob.set_ids(ids)
    before = prob.host_state()
    host = {k: torch.from_numpy(before[k].copy()).pin_memory() for k in ("w_now", "w_snap", "theta_g", "momentum")}
    delta_h = torch.zeros(w.N).pin_memory()
    last_h = torch.from_numpy(before["last_sync"].copy())
    norms_h = torch.zeros(w.K)
    scores_h = torch.full((w.K,), float("inf"))
    ids_h = torch.tensor(ids, dtype=torch.int32)
    ws = torch.empty(3 * 11 * 8192, dtype=torch.float32, device="cuda")       # 8192-element chunks
    snap_h = host["w_now"] if same else host["w_snap"]
    hp = prob.hyper(tau=0) if same else prob.hyper()
    prob.ctx.cocodc_outer_step_host(hp, host["w_now"], snap_h, w.N, w.N, None, host["theta_g"], host["momentum"],
                                    delta_h, ids_h, len(ids), 8, 8 if same else 10, last_h, norms_h, scores_h, ws)
    assert prob.poll() == 0
    # device path on the same inputs
    delta_d = torch.zeros(w.N, device="cuda")
    prob.outer_step(8, 8 if same else 10, hyper=hp, delta_out=delta_d, w_snap=prob.bufs.w_now if same else None)
    assert prob.poll() == 0
    for k in ("w_now", "theta_g", "momentum"):
        assert torch.equal(host[k], getattr(prob.bufs, k).cpu()), k
    assert torch.equal(delta_h, delta_d.cpu())
    assert torch.equal(last_h, prob.last_sync.cpu())
    assert np.allclose(norms_h.numpy(), np_(prob.norms), rtol=1e-6)
    ohp = orc_hyper(w, tau=0) if same else orc_hyper(w)
    check_step_against_oracle(prob, before, ids, 8, 8 if same else 10, ohp, delta_out=delta_d, same=same)
    if not same:
        # snapshots kept on the device: S0 from the host buffer into a device pool, then the completion
        host2 = {k: torch.from_numpy(before[k].copy()).pin_memory() for k in ("w_now", "theta_g", "momentum")}
        snap_src = torch.from_numpy(before["w_snap"].copy()).pin_memory()      # parameters as they were at t_p
        pool = torch.zeros((w.M, 190_104), device="cuda")
        pool_off = torch.tensor([50_001, -1, 0], dtype=torch.int64)             # fragment 0 lands on an odd offset
        prob.ctx.cocodc_snapshot_host(snap_src, pool, w.N, pool.stride(0), pool_off, w.M, ids_h, len(ids))
        last2 = torch.from_numpy(before["last_sync"].copy())
        n2, s2 = torch.zeros(w.K), torch.full((w.K,), float("inf"))
        prob.ctx.cocodc_outer_step_host(hp, host2["w_now"], pool, w.N, pool.stride(0), pool_off, host2["theta_g"],
                                        host2["momentum"], None, ids_h, len(ids), 8, 10, last2, n2, s2, ws,
                                        snap_on_device=True)
        assert prob.poll() == 0
        for k in ("w_now", "theta_g", "momentum"):
            assert torch.equal(host2[k], host[k]), k
        assert torch.equal(n2, norms_h) and torch.equal(s2, scores_h)
    # too small a workspace is refused
    with pytest.raises(prob.B.CocodcError):
        prob.ctx.cocodc_outer_step_host(hp, host["w_now"], snap_h, w.N, w.N, None, host["theta_g"],
                                        host["momentum"], None, ids_h, len(ids), 8, 10, last_h, norms_h,
                                        scores_h, ws[:1000])


def test_bounded_wait_runs_out_and_leaves_the_context_usable():
    """Failure detection without a fault: a wait that nothing completes ends by itself with a status."""
    prob = make(4, seed=140)
    prob.ctx.cocodc_selftest_bounded_wait(2000)
    assert prob.poll() == prob.B.ERR_TIMEOUT
    assert prob.poll() == 0
    with pytest.raises(prob.B.CocodcError):
        prob.ctx.cocodc_selftest_bounded_wait(0)
    ids = [0, 3]
    prob.set_ids(ids)
    before = prob.host_state()
    prob.outer_step(2, 4)
    assert prob.poll() == 0
    check_step_against_oracle(prob, before, ids, 2, 4, orc_hyper(prob.w))


# several tiles per CTA (148 CTAs x 1024-element tiles), ragged edges, an odd start
MANY_TILES = (1_300_000, [[(4, 600_001)], [(600_008, 650_000)], [(1_250_009, 40_000)]])


@pytest.mark.parametrize("M", [9, 13, 16, 34, 49])
def test_worker_counts_beyond_the_instantiated_ones(M):
    """Run-time worker counts (slot-ring kernel; 49 recorded tiles no longer fit its ring, so the fused mode takes the
    element loop there): fused step, unfused halves bit-identical to it, zero delay, and the two-phase calls."""
    a = make(M, seed=500 + M, frs=MANY_TILES, snap_layout="pool", pool_ids=[1, 0, 2])
    ids = [1, 0, 2]
    a.set_ids(ids)
    before = a.host_state()
    delta = torch.full((a.w.N,), 7.0, dtype=torch.float32, device="cuda")
    a.outer_step(t_p=10, t_l=12, delta_out=delta)
    assert a.poll() == 0
    check_step_against_oracle(a, before, ids, 10, 12, orc_hyper(a.w), delta_out=delta)
    # S1-S3 + S6, then S4-S5: same bits as the fused step
    b = make(M, seed=500 + M, frs=MANY_TILES, snap_layout="pool", pool_ids=[1, 0, 2])
    b.set_ids(ids)
    b.outer_step(10, 12, stages=1 | 4)
    b.merge(b.bufs.theta_g)
    # pseudo-gradient sum + received sum: same bits again
    c = make(M, seed=500 + M, frs=MANY_TILES, snap_layout="pool", pool_ids=[1, 0, 2])
    c.set_ids(ids)
    cb = c.bufs
    s = torch.zeros(c.w.N, device="cuda")
    c.ctx.cocodc_pseudo_gradient_sum(cb.w_snap, cb.snap_stride, cb.snap_offset, cb.theta_g, M, s, c.ids, c.n_ids)
    c.ctx.cocodc_outer_step_received(c.hyper(), M, cb.w_now, cb.w_snap, cb.now_stride, cb.snap_stride, cb.snap_offset,
                                     cb.theta_g, cb.momentum, s, None, c.ids, c.n_ids, 10, 12, c.last_sync, c.norms,
                                     c.scores)
    assert b.poll() == 0 and c.poll() == 0
    for other in (b, c):
        for x, y in ((a.bufs.w_now, other.bufs.w_now), (a.bufs.theta_g, other.bufs.theta_g),
                     (a.bufs.momentum, other.bufs.momentum), (a.scores, other.scores), (a.norms, other.norms)):
            assert torch.equal(x, y)
    # zero delay on the state the first step left
    before = a.host_state()
    a.outer_step(100, 100, hyper=a.hyper(tau=0), w_snap=a.bufs.w_now)
    assert a.poll() == 0
    check_step_against_oracle(a, before, ids, 100, 100, orc_hyper(a.w, tau=0), same=True)


def random_problem_spec(seed):
    """A random fragment table (gaps, odd offsets, several segments), worker count, id list and snapshot layout
    (plain / packed pool / packed pool at arbitrary offsets); returns (rng, workload, ids, generate-kwargs)."""
    rng = np.random.default_rng(1000 + seed)
    M = int(rng.choice([1, 2, 3, 4, 4, 4, 6, 8, 11]))
    K = int(rng.integers(1, 7))
    pos, frs = int(rng.integers(0, 9)), []
    for p in range(K):
        segs = []
        for _ in range(int(rng.integers(1, 4))):
            ln = int(rng.choice([1, 3, 4, 5, 1023, 1024, 1025, 2048, 4099, 9000, 20_000]))
            segs.append((pos, ln))
            pos += ln + int(rng.choice([0, 0, 1, 3, 4, 17]))
        frs.append(segs)
    N = pos + (-pos) % 4 + 4
    w = synth.small_workload((N, frs), M=M, seed=seed, scale_kind="loguniform", tau=int(rng.integers(1, 9)),
                             lam=float(rng.choice([0.0, 0.5, 1.0])))
    ids = [int(p) for p in rng.permutation(K)[:int(rng.integers(1, K + 1))]]
    layout = rng.choice(["full", "pool", "pool_odd"])
    kw = {}
    if layout != "full":
        kw = dict(snap_layout="pool", pool_ids=ids)
        if layout == "pool_odd":
            offs, cur = {}, int(rng.integers(0, 4))
            for p in ids:
                offs[p] = cur
                cur += w.partition.frag_size(p) + int(rng.integers(0, 6))
            kw.update(pool_offsets=offs, pool_len=cur + 8 - cur % 4)
    return rng, w, ids, kw


@pytest.mark.parametrize("seed", range(12))
def test_random_partitions_layouts_and_modes(seed):
    """Randomised sweep: fragment tables with gaps, odd offsets and several segments, random worker counts,
    id lists, snapshot layouts (plain / packed pool with arbitrary offsets), sign modes, mixing factors."""
    rng, w, ids, kw = random_problem_spec(seed)
    M = w.M
    prob = GpuProblem(w, synth.generate(w, "cuda", momentum_sigma=1e-3, **kw))
    prob.set_ids(ids)
    sign = int(rng.integers(0, 3))
    alpha = float(rng.choice([1.0, 1.0, 0.5]))
    comp = int(rng.choice([1, 1, 0]))
    delta = torch.full((w.N,), 3.0, device="cuda") if rng.random() < 0.5 else None
    before = prob.host_state()
    t_p = int(rng.integers(1, 50))
    prob.outer_step(t_p, t_p + w.tau, hyper=prob.hyper(sign_mode=sign, alpha=alpha, comp_mode=comp), delta_out=delta)
    assert prob.poll() == 0
    check_step_against_oracle(prob, before, ids, t_p, t_p + w.tau,
                              orc_hyper(w, sign_mode=sign, alpha=alpha, comp_mode=comp), delta_out=delta)
    # S0 on the same table and layout
    snap_before = prob.host_state()
    prob.snapshot()
    assert prob.poll() == 0
    exp = orc.snapshot(fragments_of(w), snap_before["w_now"], ids, M, snap_before["snap_offset"], snap_before["w_snap"])
    assert np.array_equal(np_(prob.bufs.w_snap), exp)


@pytest.mark.parametrize("seed", range(100, 112))
def test_random_problems_unfused_and_two_phase_equal_the_fused_step(seed):
    """On the same random tables and layouts: S1-S3+S6 then S4-S5 as two calls, and the worker-per-device chain
    (pseudo-gradient sum, then the completion from that sum with every worker local), must reproduce the fused
    step bit for bit.  The halves and the sum read few streams and run with other tile widths and ring depths
    than the fused step, in packed and odd-offset pools too."""
    rng, w, ids, kw = random_problem_spec(seed)
    probs = [GpuProblem(w, synth.generate(w, "cuda", momentum_sigma=1e-3, **kw)) for _ in range(3)]
    for prob in probs:
        prob.set_ids(ids)
    a, b, c = probs
    sign = int(rng.integers(0, 3))
    hp = dict(sign_mode=sign, alpha=float(rng.choice([1.0, 0.5])), comp_mode=int(rng.choice([1, 1, 0])))
    t_p = 7
    t_l = t_p + w.tau
    a.outer_step(t_p, t_l, hyper=a.hyper(**hp))
    b.outer_step(t_p, t_l, hyper=b.hyper(**hp), stages=1 | 4)
    b.merge(b.bufs.theta_g, hyper=b.hyper(**hp))
    cb = c.bufs
    sums = torch.full((w.N,), 3.0, device="cuda")
    c.ctx.cocodc_pseudo_gradient_sum(cb.w_snap, cb.snap_stride, cb.snap_offset, cb.theta_g, w.M, sums, c.ids, c.n_ids)
    c.ctx.cocodc_outer_step_received(c.hyper(**hp), w.M, cb.w_now, cb.w_snap, cb.now_stride, cb.snap_stride,
                                     cb.snap_offset, cb.theta_g, cb.momentum, sums, None, c.ids, c.n_ids, t_p, t_l,
                                     c.last_sync, c.norms, c.scores)
    for other, what in ((b, "unfused"), (c, "two-phase")):
        assert other.poll() == 0
        for name in ("w_now", "theta_g", "momentum", "w_snap"):
            assert torch.equal(getattr(a.bufs, name), getattr(other.bufs, name)), (what, name)
        assert torch.equal(a.norms, other.norms) and torch.equal(a.scores, other.scores), what
        assert torch.equal(a.last_sync, other.last_sync), what
    assert a.poll() == 0
    untouched = torch.from_numpy(~touched_mask(w, ids)).cuda()
    assert bool((sums[untouched] == 3.0).all())


@pytest.mark.parametrize("M", [2, 3, 4])
@pytest.mark.parametrize("depth", [1e-3, 1e-6])
def test_cancellation_regime_error_is_bounded_by_the_operands(M, depth):
    """Where the workers' pseudo-gradients cancel (|Delta| << |delta_m|) and the momentum term cancels against their
    mean, no bound relative to the OUTPUT can hold in fp32: what is left of Delta and u' is rounding error of their
    operands.  The kernel's contract there is a bound relative to the operands,

        |x - y| <= (M + 2) * 2^-24 * (mean_m |delta_m| + |mu * u|)      for x in {Delta, u'},

    per element: M roundings of the sum's terms and partial sums, one of the quotient, one of the momentum update
    (each at most 2^-24 of a value no larger than the operands' magnitudes).  Inputs are built so that the mean
    cancels to `depth` of the pseudo-gradients and u' to `depth` of mu*u; eta and mu are fp32 numbers, so both
    sides compute with the same hyper-parameters."""
    n = 150_000
    w = synth.small_workload((2 * n + 8, [[(1, n)], [(n + 4, n)]]), M=M, seed=500 + M, tau=3)
    mu, eta = float(np.float32(0.9)), float(np.float32(0.7))
    w = w.with_(momentum=mu, outer_lr=eta)
    bufs = synth.generate(w, "cpu")
    rng = np.random.default_rng(M)
    thg = bufs.theta_g.numpy().astype(np.float64)
    snap = bufs.w_snap.numpy()
    # the last worker's pseudo-gradient = -(sum of the others) + depth * noise
    others = (snap[:M - 1].astype(np.float64) - thg[None, :]).sum(axis=0)
    last = -others + depth * 1e-3 * rng.standard_normal(thg.shape)
    snap[M - 1] = (thg + last).astype(np.float32)
    delta_m = snap.astype(np.float64) - thg[None, :]                     # what the workers' values really encode
    mean = delta_m.mean(axis=0)
    # momentum that cancels the mean to `depth`:  mu*u + Delta = depth * |mu*u| * noise
    u_mag = 1e-3 * (1.0 + rng.random(thg.shape))
    u = (-mean + depth * u_mag * rng.standard_normal(thg.shape)) / mu
    big = rng.random(thg.shape) < 0.5                                     # half the elements: a large momentum, cancelled by nothing
    u = np.where(big, u_mag * np.sign(rng.standard_normal(thg.shape)), u)
    bufs.momentum.copy_(torch.from_numpy(u.astype(np.float32)))
    for name in ("theta_g", "momentum", "w_now", "w_snap"):
        setattr(bufs, name, getattr(bufs, name).cuda())
    prob = GpuProblem(w, bufs)
    ids = [1, 0]
    prob.set_ids(ids)
    before = prob.host_state()
    delta = torch.zeros(w.N, device="cuda")
    prob.outer_step(6, 9, delta_out=delta)
    assert prob.poll() == 0
    frs = fragments_of(w)
    res, _ = orc.outer_step(frs, orc_hyper(w), before["w_now"], before["w_snap"], before["theta_g"],
                            before["momentum"], ids, 6, 9, before["last_sync"])
    after = prob.host_state()
    worst = 0.0
    cancelled = 1.0
    for p in ids:
        b = orc.gather_fragment(frs, before["w_snap"], p).astype(np.float64)
        g0 = orc.gather_fragment(frs, before["theta_g"], p).astype(np.float64)
        u0 = orc.gather_fragment(frs, before["momentum"], p).astype(np.float64)
        operands = np.abs(b - g0[None, :]).mean(axis=0) + np.abs(mu * u0)
        bound = (M + 2) * 2.0 ** -24 * operands
        got_d = orc.gather_fragment(frs, np_(delta), p).astype(np.float64)
        got_u = orc.gather_fragment(frs, after["momentum"], p).astype(np.float64)
        for got, exp, what in ((got_d, res[p].delta_g, "Delta"), (got_u, res[p].momentum, "u'")):
            err = np.abs(got - exp)
            assert np.all(err <= bound), (what, p, float((err / bound).max()))
            worst = max(worst, float((err / bound).max()))
        cancelled = min(cancelled, float(np.median(np.abs(res[p].delta_g) / np.abs(b - g0[None, :]).mean(axis=0))))
        # the new global state and the merged parameters keep the ordinary bound: |theta_g| dominates them
        assert_close(orc.gather_fragment(frs, after["theta_g"], p), res[p].theta_g, TOL_PARAM, f"theta_g[{p}]")
        wn = orc.gather_fragment(frs, after["w_now"], p)
        for m in range(M):
            assert_close(wn[m], res[p].w_now[m], TOL_PARAM, f"w_now[{m}][{p}]")
    assert cancelled < 10 * depth + 1e-5, cancelled         # the inputs really are in the cancellation regime
    assert worst > 0.0
    print(f"cancellation regime M={M} depth={depth:g}: worst error / bound = {worst:.3f}, |Delta| / mean|delta_m| = {cancelled:.2e}")


def _check_pooled(prob, before, ids, t_p, t_l):
    """Parity over all listed fragments taken together (fragments of one or a few elements leave the
    per-fragment measure nothing to normalise by when an output is small against its operands)."""
    w = prob.w
    frs = fragments_of(w)
    res, new_last = orc.outer_step(frs, orc_hyper(w), before["w_now"], before["w_snap"], before["theta_g"],
                                   before["momentum"], ids, t_p, t_l, before["last_sync"])
    after = prob.host_state()
    cat = lambda f: np.concatenate([f(p) for p in ids], axis=-1)
    assert_close(cat(lambda p: orc.gather_fragment(frs, after["theta_g"], p)), cat(lambda p: res[p].theta_g), TOL_PARAM, "theta_g")
    assert_close(cat(lambda p: orc.gather_fragment(frs, after["momentum"], p)), cat(lambda p: res[p].momentum), TOL_PARAM, "momentum")
    for m in range(w.M):
        assert_close(cat(lambda p: orc.gather_fragment(frs, after["w_now"], p)[m]), cat(lambda p: res[p].w_now[m]), TOL_PARAM, f"w_now[{m}]")
    norms = np.array([res[p].norm for p in ids])
    got = after["norms"][ids]
    big = norms > 1e-3 * norms.max()
    assert np.all(np.abs(got[big] - norms[big]) <= 1e-5 * norms[big])
    assert np.all(np.abs(got[~big] - norms[~big]) <= 1e-5 * norms.max())
    assert np.array_equal(after["last_sync"], new_last)
    untouched = ~touched_mask(w, ids)
    for k in ("theta_g", "momentum"):
        assert np.array_equal(after[k][untouched], before[k][untouched])
    assert np.array_equal(after["w_now"][:, untouched], before["w_now"][:, untouched])


def test_maximum_fragment_count():
    """K = 1024 fragments (the limit of a context), many of them shorter than a tile, all completed in one call."""
    rng = np.random.default_rng(5)
    sizes = rng.choice([1, 7, 255, 257, 1023, 1024, 1500], size=1024).tolist()
    offs = np.concatenate([[0], np.cumsum(sizes)])
    total = int(offs[-1])
    w = synth.small_workload((total + 8 - total % 4, [[(int(o), int(l))] for o, l in zip(offs[:-1], sizes)]),
                             M=2, seed=150)
    prob = GpuProblem(w, synth.generate(w, "cuda", momentum_sigma=1e-3))
    ids = rng.permutation(1024).tolist()
    prob.set_ids(ids)
    before = prob.host_state()
    prob.outer_step(3, 4)
    assert prob.poll() == 0
    _check_pooled(prob, before, ids, 3, 4)
    # selection over all 1024 under a parameter budget, feeding the next completion
    prob.select(t_now=50, budget_kind=1, budget=int(sum(sizes) // 3))
    n = int(prob.n_ids.item())
    got = np_(prob.ids)[:n].tolist()
    _, eids, en = orc.select_fragments(np_(prob.scores), np_(prob.last_sync), w.partition.frag_sizes, 50, w.H,
                                       orc.BUDGET_PARAMS, int(sum(sizes) // 3))
    assert n == en and got == eids.tolist()
    before = prob.host_state()
    prob.outer_step(50, 52)
    assert prob.poll() == 0
    _check_pooled(prob, before, got, 50, 52)
    with pytest.raises(prob.B.CocodcError):
        ptr = np.arange(1026, dtype=np.int32)
        prob.B.Context(1025, ptr, np.arange(1025), np.ones(1025, dtype=np.int64), 1)


@pytest.mark.parametrize("n_seg", [127, 128, 129])
def test_fragment_tables_on_both_sides_of_the_kernel_argument_limit(n_seg):
    """Fragment tables of up to 128 segments travel as a kernel argument and the streaming kernel expands the id list
    itself; larger ones go through the plan kernel.  Same results on both sides of the limit: completion (all
    fragments, then a permuted subset), snapshot, stand-alone scores, and the rejection of a bad id list."""
    rng = np.random.default_rng(n_seg)
    K = n_seg - 20                       # twenty fragments have two segments
    frs, pos = [], 3
    for p in range(K):
        segs = []
        for _ in range(2 if p < 20 else 1):
            ln = int(rng.choice([5, 700, 1024, 2049, 4100]))
            segs.append((pos, ln))
            pos += ln + int(rng.choice([0, 1, 4]))
        frs.append(segs)
    w = synth.small_workload((pos + 8 - pos % 4, frs), M=3, seed=n_seg, scale_kind="loguniform", tau=2)
    assert w.partition.n_segments == n_seg
    prob = GpuProblem(w, synth.generate(w, "cuda", momentum_sigma=1e-3))
    for ids in (list(range(K)), [int(p) for p in rng.permutation(K)[:K // 3]]):
        prob.set_ids(ids)
        before = prob.host_state()
        n0 = prob.ctx.launch_count
        prob.outer_step(4, 6)
        assert prob.ctx.launch_count - n0 == (1 if n_seg <= 128 else 2)
        assert prob.poll() == 0
        _check_pooled(prob, before, ids, 4, 6)
        snap_before = prob.host_state()
        prob.snapshot()
        assert prob.poll() == 0
        exp = orc.snapshot(fragments_of(w), snap_before["w_now"], ids, w.M, None, snap_before["w_snap"])
        assert np.array_equal(np_(prob.bufs.w_snap), exp)
    x = prob.bufs.theta_g
    norms = torch.zeros(K, device="cuda")
    scores = torch.zeros(K, device="cuda")
    prob.ctx.cocodc_fragment_scores(x, None, norms, scores)
    en, _ = orc.fragment_scores(fragments_of(w), np_(x))
    assert np.all(np.abs(np_(norms) - en) <= 1e-5 * en) and prob.poll() == 0
    prob.ids[:2] = 7                     # listed twice
    prob.n_ids.fill_(2)
    before = prob.host_state()
    prob.outer_step(8, 9)
    assert prob.poll() == prob.B.ERR_INVALID_ARG
    assert np.array_equal(prob.host_state()["theta_g"], before["theta_g"])
    prob.set_ids([1, 0])                 # and the context works on afterwards
    before = prob.host_state()
    prob.outer_step(8, 9)
    assert prob.poll() == 0
    _check_pooled(prob, before, [1, 0], 8, 9)
