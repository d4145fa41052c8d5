"""The schedule driver around the path (Section 2.1 time line, Section 3.2) in the paper's own setting:
M = 4 workers, H = 100, tau = 5, K = 4 strided shards of three layers, lambda = 0.5, gamma = 0.4, which gives
8 synchronisations per H steps (Section 4.1), one fragment per decision (Algorithm 2).

Every event is checked against the oracle from the GPU's own state just before it (selection bit-exact,
completion within the parity tolerance), and the schedule's guarantees are checked at the end."""

import numpy as np
import pytest
import torch

import synth
from oracle import reference as orc
from helpers import TOL_NORM, TOL_PARAM, assert_close, fragments_of, np_

pytestmark = pytest.mark.gpu


def strided_workload(layer=3001, layers=12, shards=4, M=4):
    frs = [[(l * layer, layer) for l in range(k, layers, shards)] for k in range(shards)]
    total = layer * layers
    return synth.small_workload((total + 4 - total % 4, frs), M=M, seed=31, tau=5, H=100,
                                lam=0.5, budget_kind="count", budget=1)


def test_round_driver_in_the_papers_setting():
    from paper_2504_17672_b200 import binding as B
    from paper_2504_17672_b200.schedule import RoundDriver
    w = strided_workload()
    frs = fragments_of(w)
    bufs = synth.generate(w, "cuda")
    ptr, off, ln = w.partition.csr()
    ctx = B.Context(w.N, ptr, off, ln, w.M)
    hyper = B.Hyper(M=w.M, H=w.H, tau=w.tau, outer_lr=w.outer_lr, momentum=w.momentum, lam=w.lam, alpha=1.0)
    drv = RoundDriver(ctx, hyper, bufs.w_now, bufs.theta_g, bufs.momentum, w.partition.frag_sizes,
                      gamma=0.4, Tc=0.2, Ts=1.0, budget_kind=B.BUDGET_COUNT, budget=1)
    assert (drv.N_sync, drv.h) == (8, 12)                       # Section 4.1: eight synchronisations per H steps with these settings
    ohp = orc.Hyper(M=w.M, H=w.H, tau=w.tau, outer_lr=w.outer_lr, momentum=w.momentum, lam=w.lam, alpha=1.0)
    log = {"initiated": [], "completed": [], "pre": None, "worst": 0.0}

    def state():
        return dict(w_now=np_(bufs.w_now).copy(), theta_g=np_(bufs.theta_g).copy(), momentum=np_(bufs.momentum).copy(),
                    scores=np_(drv.scores).copy(), last_sync=np_(drv.last_sync).copy(),
                    in_flight=np_(drv.in_flight).copy(), norms=np_(drv.norms).copy())

    def observer(kind, phase, slot, t):
        if phase == "before":
            log["pre"] = state()
            if kind == "complete":
                log["pre"]["pool"] = np_(slot.pool).copy()
                log["pre"]["pool_off"] = np_(slot.pool_off).copy()
                log["pre"]["ids"] = np_(slot.ids)[:int(slot.n_ids.item())].tolist()
                log["pre"]["t_p"] = slot.t_p
            return
        pre, post = log["pre"], state()
        assert ctx.cocodc_poll_status() == 0
        if kind == "initiate":
            mask, ids, n = orc.select_fragments(pre["scores"], pre["last_sync"], w.partition.frag_sizes, t, w.H,
                                                orc.BUDGET_COUNT, 1, pre["in_flight"])
            got = np_(slot.ids)[:int(slot.n_ids.item())].tolist()
            assert got == ids.tolist() and np.array_equal(np_(slot.mask), mask)
            assert not any(pre["in_flight"][p] for p in got)           # never a fragment that is in flight
            assert np.array_equal(post["in_flight"], pre["in_flight"] + mask)   # marked by the selection kernel itself
            po = np_(slot.pool_off)
            exp_pool = orc.snapshot(frs, pre["w_now"], got, w.M, po, np_(slot.pool))
            assert np.array_equal(np_(slot.pool), exp_pool)             # S0 recorded exactly the chosen fragments
            log["initiated"].append((t, got))
        else:
            ids = pre["ids"]
            res, new_last = orc.outer_step(frs, ohp, pre["w_now"], pre["pool"], pre["theta_g"], pre["momentum"], ids,
                                           pre["t_p"], t, pre["last_sync"], snap_offset=pre["pool_off"])
            assert t - pre["t_p"] == w.tau
            for p in ids:
                r = res[p]
                log["worst"] = max(log["worst"], *assert_close(orc.gather_fragment(frs, post["theta_g"], p), r.theta_g,
                                                               TOL_PARAM, "theta_g"))
                assert_close(orc.gather_fragment(frs, post["momentum"], p), r.momentum, TOL_PARAM, "momentum")
                wn = orc.gather_fragment(frs, post["w_now"], p)
                for m in range(w.M):
                    assert_close(wn[m], r.w_now[m], TOL_PARAM, f"w_now[{m}]")
                assert abs(post["scores"][p] - r.score) <= TOL_NORM * r.score
            assert np.array_equal(post["last_sync"], new_last)
            done = np.zeros(w.K, dtype=np.uint8)
            done[ids] = 1
            assert all(pre["in_flight"][p] == 1 for p in ids)
            assert np.array_equal(post["in_flight"], pre["in_flight"] - done)   # cleared by the completion's last warp
            log["completed"].append((t, ids))

    drv.observer = observer
    gen = torch.Generator(device="cuda").manual_seed(77)
    T = 230
    for t in range(1, T + 1):
        # local training: every worker moves a little
        bufs.w_now.add_(torch.randn(bufs.w_now.shape, generator=gen, device="cuda") * 2e-4)
        drv.after_local_step(t)

    starts = [t for t, _ in log["initiated"]]
    assert starts == list(range(12, T + 1, 12))                                   # every h = 12 steps
    assert [ids for _, ids in log["initiated"][:4]] == [[0], [1], [2], [3]]        # never-synced first, in order
    assert [t for t, _ in log["completed"]] == [s + w.tau for s in starts if s + w.tau <= T]
    # at least K synchronisations per H steps, 8 with this gamma
    for lo in range(12, T - w.H, 12):
        in_window = [ids[0] for t, ids in log["initiated"] if lo <= t < lo + w.H]
        assert len(in_window) >= 8
        # the staleness rule of Algorithm 2 brings every fragment back within H steps of its last
        # completion, up to the delay and the wait for the next initiation slot(s)
        wide = [ids[0] for t, ids in log["initiated"] if lo <= t < lo + w.H + 2 * drv.h]
        assert set(wide) == {0, 1, 2, 3}
    # no fragment goes stale: time since its last completed sync stays below H plus one interval and the delay
    last = np_(drv.last_sync)
    assert np.all(T - last < w.H + 2 * drv.h + w.tau)
    counts = np.bincount([ids[0] for _, ids in log["initiated"]], minlength=4)
    assert counts.min() >= 2 and counts.sum() == len(starts)
    assert log["worst"] <= TOL_PARAM


@pytest.mark.parametrize("variant,lam,tau", [("diloco", 0.0, 0), ("streaming_diloco", 0.0, 4), ("cocodc", 0.0, 4),
                                             ("cocodc", 0.5, 4), ("cocodc", 0.5, 8)])
def test_toy_training_converges_under_every_variant(variant, lam, tau):
    """Workers with different quadratic objectives, synchronised through the library under a delay, reach the
    optimum of the mean objective; the run is reproducible from its seed."""
    from paper_2504_17672_b200.toy import run_toy
    r = run_toy(variant, lam=lam, tau=tau if variant != "diloco" else 4, steps=300, seed=3)
    again = run_toy(variant, lam=lam, tau=tau if variant != "diloco" else 4, steps=300, seed=3)
    assert r.losses == again.losses
    assert r.syncs >= 300 // 20
    start, final = r.losses[0][1], r.final
    assert np.isfinite(final) and final < 0.02 * start, (start, final)


def test_two_parameter_range_shards_keep_the_same_selection():
    """The benchmark's param_shard deployment, two ranks taken in turn on one GPU: each shard completes its element
    range and contributes its sums of squares, the totals (added here where the all-reduce would add them) give
    every shard the same scores and last_sync, and the replicated selection must pick the same fragments on both,
    step after step - without any exchange of the decision itself (Section 3.2)."""
    import bench
    w = synth.get_workload("gpt2_small")
    dev = torch.device("cuda", 0)
    jobs = [bench.DeviceJob(w, dev, "cocodc", "param_shard", world=1, M_total=w.M, worker_offset=0, shard=r)
            for r in range(2)]
    assert not torch.equal(jobs[0].bufs.theta_g, jobs[1].bufs.theta_g)          # different element ranges
    assert torch.equal(jobs[0].ids, jobs[1].ids) and torch.equal(jobs[0].n_ids, jobs[1].n_ids)
    seen = []
    for step in range(6):
        for j in jobs:
            j.outer_param_shard()
        total = jobs[0].sumsq + jobs[1].sumsq
        for j in jobs:
            j.sumsq.copy_(total)
            j.ctx.cocodc_scores_from_sumsq(j.sumsq, j.ids, j.n_ids, None, j.t, j.t + w.tau, j.last_sync, j.norms,
                                           j.scores)
            j.t += w.tau
            j.initiate()
            assert j.ctx.cocodc_poll_status() == 0
        a, b = jobs
        assert torch.equal(a.ids, b.ids) and torch.equal(a.n_ids, b.n_ids), step
        assert torch.equal(a.scores, b.scores) and torch.equal(a.last_sync, b.last_sync), step
        seen.append(np_(a.ids)[:int(a.n_ids.item())].tolist())
    assert len({tuple(s) for s in seen}) > 1          # the schedule moves on


def test_two_worker_groups_keep_the_replicated_state_identical():
    """The benchmark's worker_per_device deployment, two ranks taken in turn on one GPU: each holds two of the four
    workers and the whole (replicated) global state; the pseudo-gradient sums are added where the all-reduce would
    add them, and every rank completes from the same received sum - global state, momentum, scores and the
    selection must stay bit-identical on both ranks, and agree with the four-worker step on one device."""
    import bench
    w4 = synth.get_workload("gpt2_small")
    w2 = w4.with_(M=2)
    dev = torch.device("cuda", 0)
    ranks = [bench.DeviceJob(w2, dev, "cocodc", "worker_per_device", world=1, M_total=4, worker_offset=2 * r)
             for r in range(2)]
    whole = bench.DeviceJob(w4, dev, "cocodc", "replicas")
    assert torch.equal(ranks[0].bufs.theta_g, ranks[1].bufs.theta_g) and torch.equal(ranks[0].bufs.theta_g, whole.bufs.theta_g)
    assert torch.equal(ranks[1].bufs.w_now[0], whole.bufs.w_now[2])               # rank 1 holds workers 2 and 3
    for step in range(4):
        assert torch.equal(ranks[0].ids, whole.ids)
        for j in ranks:
            j.pseudo_sum_and_exchange()
        total = ranks[0].sum_buf + ranks[1].sum_buf
        for j in ranks:
            j.sum_buf.copy_(total)
            j.outer_received()
            j.t += w2.tau
            j.initiate()
            assert j.ctx.cocodc_poll_status() == 0
        whole.step()
        a, b = ranks
        for x, y in ((a.bufs.theta_g, b.bufs.theta_g), (a.bufs.momentum, b.bufs.momentum), (a.scores, b.scores),
                     (a.last_sync, b.last_sync), (a.ids, b.ids), (a.n_ids, b.n_ids)):
            assert torch.equal(x, y), step
        # against all four workers on one device: the same up to the order in which the four differences are added
        ref = whole.bufs.theta_g
        err = float((a.bufs.theta_g - ref).abs().max() / ref.abs().max())
        assert err <= 1e-6, (step, err)
        assert torch.allclose(a.scores, whole.scores, rtol=1e-5)
        # each rank merged its own two workers: they match the four-worker job's rows
        assert float((b.bufs.w_now - whole.bufs.w_now[2:4]).abs().max()) <= 1e-6 * float(whole.bufs.w_now.abs().max())
