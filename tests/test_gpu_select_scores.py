"""Bit-exact parity of the device-side fragment selection (Algorithm 2 under a budget) and
parity of the stand-alone fragment scores (Eq. 10)."""

import numpy as np
import pytest
import torch

import synth
from oracle import reference as orc
from helpers import GpuProblem, fragments_of, np_, TOL_NORM

pytestmark = pytest.mark.gpu


def selection_problem(K, rng, sizes=None):
    sizes = rng.integers(1, 5000, size=K) if sizes is None else sizes
    w = synth.small_workload([int(s) for s in sizes], M=1, seed=0)
    from paper_2504_17672_b200 import binding as B
    ptr, off, ln = w.partition.csr()
    return w, B.Context(w.N, ptr, off, ln, 1), B


@pytest.mark.parametrize("K", [1, 2, 7, 13, 32, 64, 333, 1024])
def test_selection_matches_oracle_bit_for_bit(K):
    rng = np.random.default_rng(K)
    w, ctx, B = selection_problem(K, rng)
    sizes = w.partition.frag_sizes
    dev = "cuda"
    mask = torch.zeros(K, dtype=torch.uint8, device=dev)
    ids = torch.zeros(K, dtype=torch.int32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    for trial in range(12):
        pool = np.array([0.0, 0.5, 1.0, 1.0, 2.5, 3.0, np.inf, np.inf], dtype=np.float32)
        if trial % 2:
            scores = rng.choice(pool, size=K)
        else:
            scores = rng.random(K).astype(np.float32)
        H = 100
        last = rng.integers(0, 200, size=K).astype(np.int64)
        t_now = int(rng.integers(100, 280))
        inel = (rng.random(K) < 0.3).astype(np.uint8) if trial % 3 else None
        if trial == 5 and inel is not None:
            inel[:] = 1
        for kind, budget in ((B.BUDGET_COUNT, int(rng.integers(0, K + 2))),
                             (B.BUDGET_PARAMS, int(rng.integers(0, sizes.sum() + 1))),
                             (B.BUDGET_COUNT, 1)):
            ctx.cocodc_select_fragments(torch.from_numpy(scores).to(dev), torch.from_numpy(last).to(dev),
                                        None if inel is None else torch.from_numpy(inel).to(dev),
                                        t_now, H, kind, budget, mask, ids, n_sel)
            assert ctx.cocodc_poll_status() == 0
            emask, eids, en = orc.select_fragments(scores, last, sizes, t_now, H, kind, budget, inel)
            assert int(n_sel.item()) == en
            assert np.array_equal(np_(mask), emask)
            got = np_(ids)
            assert np.array_equal(got[:en], eids) and (got[en:] == -1).all()


@pytest.mark.parametrize("K", [1, 3, 8, 12, 15])
def test_exact_budget_selection_matches_oracle_bit_for_bit(K):
    """The knapsack option (outside the paper): same subsets, same order, same pool places as the oracle's
    search over all subsets, with forced (overdue / never-synced) and ineligible fragments mixed in."""
    rng = np.random.default_rng(100 + K)
    w, ctx, B = selection_problem(K, rng)
    sizes = w.partition.frag_sizes
    dev = "cuda"
    mask = torch.zeros(K, dtype=torch.uint8, device=dev)
    ids = torch.zeros(K, dtype=torch.int32, device=dev)
    n_sel = torch.zeros(1, dtype=torch.int32, device=dev)
    pool_off = torch.zeros(K, dtype=torch.int64, device=dev)
    for trial in range(10):
        if trial % 2:
            scores = rng.choice(np.array([0.0, 0.5, 1.0, 1.0, 2.5, 3.0, np.inf], dtype=np.float32), size=K)
        else:
            scores = rng.random(K).astype(np.float32)
        last = np.where(rng.random(K) < 0.15, 0, 150).astype(np.int64)
        inel = (rng.random(K) < 0.25).astype(np.uint8) if trial % 3 else None
        budget = int(rng.integers(0, sizes.sum() + 1))
        ctx.cocodc_select_fragments(torch.from_numpy(scores).to(dev), torch.from_numpy(last).to(dev),
                                    None if inel is None else torch.from_numpy(inel).to(dev),
                                    200, 100, B.BUDGET_PARAMS_EXACT, budget, mask, ids, n_sel, pool_off)
        assert ctx.cocodc_poll_status() == 0
        emask, eids, en = orc.select_fragments(scores, last, sizes, 200, 100, orc.BUDGET_PARAMS_EXACT, budget, inel)
        assert int(n_sel.item()) == en
        assert np.array_equal(np_(mask), emask)
        got = np_(ids)
        assert np.array_equal(got[:en], eids) and (got[en:] == -1).all()
        po, pos = np_(pool_off), 0
        for p in eids:          # next multiple of 4, plus the fragment's native offset mod 4
            start = pos + w.partition.fragments[p][0][0] % 4
            assert po[p] == start
            pos = (start + int(sizes[p]) + 3) // 4 * 4
        assert all(po[p] == -1 for p in range(K) if not emask[p])


def test_exact_budget_at_the_candidate_limit():
    """24 candidates (2^24 subsets): integer scores and sizes, so the optimum value is the textbook table's; one more
    candidate is reported through the status word and selects nothing."""
    from paper_2504_17672_b200 import binding as B
    rng = np.random.default_rng(77)
    for K, expect_error in ((24, False), (25, True)):
        sizes = rng.integers(4, 60, size=K)
        w, ctx, _ = selection_problem(K, rng, sizes=sizes)
        R = rng.integers(1, 100, size=K).astype(np.float32)
        budget = int(sizes.sum() // 3)
        mask = torch.zeros(K, dtype=torch.uint8, device="cuda")
        ids = torch.zeros(K, dtype=torch.int32, device="cuda")
        n_sel = torch.full((1,), -5, dtype=torch.int32, device="cuda")
        ctx.cocodc_select_fragments(torch.from_numpy(R).cuda(), torch.full((K,), 150, dtype=torch.int64, device="cuda"),
                                    None, 200, 100, B.BUDGET_PARAMS_EXACT, budget, mask, ids, n_sel)
        status = ctx.cocodc_poll_status()
        if expect_error:
            assert status == B.ERR_INVALID_ARG and int(n_sel.item()) == 0 and int(mask.sum().item()) == 0
            continue
        assert status == 0
        n = int(n_sel.item())
        chosen = np_(ids)[:n]
        assert len(set(chosen.tolist())) == n and np_(mask).sum() == n
        assert sizes[chosen].sum() <= budget
        table = np.zeros(budget + 1)
        for p in range(K):
            for c in range(budget, int(sizes[p]) - 1, -1):
                table[c] = max(table[c], table[c - int(sizes[p])] + float(R[p]))
        assert float(R[chosen].sum()) == table[budget]


def test_selection_rejects_nan_scores():
    rng = np.random.default_rng(1)
    w, ctx, B = selection_problem(6, rng)
    scores = torch.tensor([1.0, float("nan"), 2.0, 0.0, 0.0, 0.0], device="cuda")
    last = torch.zeros(6, dtype=torch.int64, device="cuda")
    mask = torch.ones(6, dtype=torch.uint8, device="cuda")
    ids = torch.zeros(6, dtype=torch.int32, device="cuda")
    n_sel = torch.full((1,), 9, dtype=torch.int32, device="cuda")
    ctx.cocodc_select_fragments(scores, last, None, 5, 100, B.BUDGET_COUNT, 2, mask, ids, n_sel)
    assert ctx.cocodc_poll_status() == B.ERR_NONFINITE
    assert int(n_sel.item()) == 0 and int(mask.sum().item()) == 0
    with pytest.raises(B.CocodcError):
        ctx.cocodc_select_fragments(scores, last, None, 5, 0, B.BUDGET_COUNT, 2, mask, ids, n_sel)
    with pytest.raises(B.CocodcError):
        ctx.cocodc_select_fragments(scores, last, None, 5, 100, 7, 2, mask, ids, n_sel)


def test_selection_feeds_the_outer_step_without_a_host_round_trip():
    """select -> snapshot -> outer_step chained on the stream; the host reads ids only afterwards to check."""
    w = synth.get_workload("tiny")
    prob = GpuProblem(w, synth.generate(w, "cuda", momentum_sigma=1e-3))
    from helpers import check_step_against_oracle, orc_hyper
    # first round: all scores infinite -> fragments 0 and 1 (budget 2), then 2 and 3, ...
    expected_rounds = [[0, 1], [2, 3], [4, 5], [6, 7]]
    t = 0
    for rnd in range(6):
        t += 12
        before = prob.host_state()
        prob.select(t_now=t)
        prob.outer_step(t_p=t, t_l=t + w.tau)
        assert prob.poll() == 0
        n = int(prob.n_ids.item())
        ids = np_(prob.ids)[:n].tolist()
        emask, eids, en = orc.select_fragments(before["scores"], before["last_sync"], w.partition.frag_sizes,
                                               t, w.H, orc.BUDGET_COUNT, w.budget)
        assert ids == eids.tolist()
        if rnd < 4:
            assert ids == expected_rounds[rnd]
        check_step_against_oracle(prob, before, ids, t, t + w.tau, orc_hyper(w))
        prob.snapshot()
        prob.bufs.w_now.add_(torch.randn_like(prob.bufs.w_now) * 1e-3)
    # after every fragment has a finite score the two largest win, unless one is overdue
    assert np.isfinite(np_(prob.scores)).all()


@pytest.mark.parametrize("frs", [
    [5000, 1, 4097, 123_457],
    (300_000, [[(1, 70_001), (200_003, 999)], [(70_002, 129_998)], [(201_002, 98_000)]]),
])
def test_standalone_scores(frs):
    w = synth.small_workload(frs, M=1, seed=3)
    from paper_2504_17672_b200 import binding as B
    ptr, off, ln = w.partition.csr()
    ctx = B.Context(w.N, ptr, off, ln, 1)
    g = torch.Generator(device="cuda").manual_seed(5)
    x = torch.randn(w.N, generator=g, device="cuda") * 1e-3
    K = w.K
    norms = torch.zeros(K, device="cuda")
    scores = torch.zeros(K, device="cuda")
    interval = torch.tensor([0, 3, 100, 7][:K], dtype=torch.int64, device="cuda")
    for iv in (None, interval):
        ctx.cocodc_fragment_scores(x, iv, norms, scores)
        assert ctx.cocodc_poll_status() == 0
        en, es = orc.fragment_scores(fragments_of(w), np_(x), None if iv is None else np_(iv))
        assert np.all(np.abs(np_(norms) - en) <= TOL_NORM * en)
        assert np.all(np.abs(np_(scores) - es) <= TOL_NORM * es)
    # reproducible to the bit from run to run
    first = norms.clone()
    ctx.cocodc_fragment_scores(x, None, norms, scores)
    assert torch.equal(first, norms)
    # closed form: a constant vector
    x.fill_(-0.25)
    ctx.cocodc_fragment_scores(x, None, norms, scores)
    exp = 0.25 * np.sqrt(w.partition.frag_sizes.astype(np.float64))
    assert np.all(np.abs(np_(norms) - exp) <= 1e-6 * exp)
    x[7] = float("nan")
    ctx.cocodc_fragment_scores(x, None, norms, scores)
    assert ctx.cocodc_poll_status() == B.ERR_NONFINITE


def test_schedule_step_replayed_from_a_cuda_graph_equals_eager_steps():
    """Completion + selection + snapshot with device-resident step numbers, recorded once and replayed: bit-identical
    to the same steps issued call by call."""
    w = synth.get_workload("tiny")
    from paper_2504_17672_b200 import binding as B

    def fresh():
        prob = GpuProblem(w, synth.generate(w, "cuda", snap_layout="pool", pool_ids=[0, 1], momentum_sigma=1e-3))
        prob.pool_off = prob.bufs.snap_offset
        prob.scores.copy_(torch.arange(w.K, 0, -1, dtype=torch.float32, device="cuda"))
        prob.set_ids([0, 1])
        return prob

    tau = w.tau
    # eager reference: five steps with host-side step numbers
    a = fresh()
    t = 10
    for _ in range(5):
        b = a.bufs
        a.ctx.cocodc_outer_step(a.hyper(), b.w_now, b.w_snap, b.now_stride, b.snap_stride, a.pool_off, b.theta_g,
                                b.momentum, None, a.ids, a.n_ids, t, t + tau, a.last_sync, a.norms, a.scores)
        t += tau
        a.ctx.cocodc_select_fragments(a.scores, a.last_sync, None, t, w.H, B.BUDGET_COUNT, w.budget, a.mask, a.ids,
                                      a.n_ids, a.pool_off)
        a.ctx.cocodc_snapshot(b.w_now, b.w_snap, b.now_stride, b.snap_stride, a.pool_off, w.M, a.ids, a.n_ids)
    assert a.poll() == 0

    # the same through a graph: clock[0] = t_p, clock[1] = t_l = the next selection's t_now
    g = fresh()
    clock = torch.tensor([10, 10 + tau], dtype=torch.int64, device="cuda")

    def step():
        b = g.bufs
        g.ctx.cocodc_outer_step_at(g.hyper(), b.w_now, b.w_snap, b.now_stride, b.snap_stride, g.pool_off, b.theta_g,
                                   b.momentum, None, g.ids, g.n_ids, clock[0:1], clock[1:2], g.last_sync, g.norms,
                                   g.scores)
        g.ctx.cocodc_select_fragments_at(g.scores, g.last_sync, None, clock[1:2], w.H, B.BUDGET_COUNT, w.budget,
                                         g.mask, g.ids, g.n_ids, g.pool_off)
        g.ctx.cocodc_snapshot(b.w_now, b.w_snap, b.now_stride, b.snap_stride, g.pool_off, w.M, g.ids, g.n_ids)
        clock.add_(tau)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()                                   # warm-up outside the capture (first-use set-up of the kernels)
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for _ in range(4):                           # one eager warm-up step + four replays (recording runs nothing)
        graph.replay()
    torch.cuda.synchronize()
    assert g.poll() == 0
    assert int(clock[0].item()) == 10 + 5 * tau
    for x, y in ((a.bufs.w_now, g.bufs.w_now), (a.bufs.theta_g, g.bufs.theta_g), (a.bufs.momentum, g.bufs.momentum),
                 (a.bufs.w_snap, g.bufs.w_snap), (a.scores, g.scores), (a.last_sync, g.last_sync), (a.ids, g.ids)):
        assert torch.equal(x, y)

    # the same schedule step as two launches (completion, initiation), again from a graph
    h = fresh()
    clock2 = torch.tensor([10, 10 + tau], dtype=torch.int64, device="cuda")

    def step2():
        b = h.bufs
        h.ctx.cocodc_outer_step_at(h.hyper(), b.w_now, b.w_snap, b.now_stride, b.snap_stride, h.pool_off, b.theta_g,
                                   b.momentum, None, h.ids, h.n_ids, clock2[0:1], clock2[1:2], h.last_sync, h.norms,
                                   h.scores)
        h.ctx.cocodc_initiate_at(h.scores, h.last_sync, None, clock2[1:2], w.H, B.BUDGET_COUNT, w.budget, h.mask,
                                 h.ids, h.n_ids, h.pool_off, b.w_now, b.w_snap, b.now_stride, b.snap_stride, w.M)
        clock2.add_(tau)

    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step2()
    torch.cuda.current_stream().wait_stream(side)
    graph2 = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph2):
        step2()
    for _ in range(4):
        graph2.replay()
    torch.cuda.synchronize()
    assert h.poll() == 0
    for x, y in ((a.bufs.w_now, h.bufs.w_now), (a.bufs.theta_g, h.bufs.theta_g), (a.bufs.momentum, h.bufs.momentum),
                 (a.bufs.w_snap, h.bufs.w_snap), (a.scores, h.scores), (a.last_sync, h.last_sync), (a.ids, h.ids)):
        assert torch.equal(x, y)


def test_selected_pool_places_keep_the_native_alignment():
    """Fragments whose native offsets are not multiples of 4: the places cocodc_select_fragments hands out in
    the snapshot pool are congruent to them mod 4 (so snapshot and completion run as vectors), do not overlap,
    fit the documented pool size, and the chain select -> snapshot -> step matches the oracle."""
    from helpers import check_step_against_oracle, orc_hyper
    frs = [[(1, 9_001)], [(9_003, 12_346)], [(21_350, 4_100), (40_003, 777)], [(25_451, 5)], [(25_457, 14_001)]]
    w = synth.small_workload((41_000, frs), M=3, seed=17, scale_kind="loguniform", tau=3)
    K = w.K
    sizes = w.partition.frag_sizes
    budget = 3
    pool_len = int(np.sort(sizes)[::-1][:budget].sum()) + 8 * K
    pool_len += (-pool_len) % 4
    prob = GpuProblem(w, synth.generate(w, "cuda", momentum_sigma=1e-3, snap_layout="pool", pool_ids=[],
                                        pool_len=pool_len))
    dev = "cuda"
    pool_off = prob.bufs.snap_offset
    rng = np.random.default_rng(3)
    for trial in range(4):
        scores = rng.random(K).astype(np.float32)
        prob.scores.copy_(torch.from_numpy(scores))
        prob.ctx.cocodc_select_fragments(prob.scores, prob.last_sync, None, 10, w.H, prob.B.BUDGET_COUNT, budget,
                                         prob.mask, prob.ids, prob.n_ids, pool_off)
        n = int(prob.n_ids.item())
        ids = np_(prob.ids)[:n].tolist()
        _, eids, en = orc.select_fragments(scores, np_(prob.last_sync), sizes, 10, w.H, orc.BUDGET_COUNT, budget)
        assert ids == eids.tolist()
        po = np_(pool_off)
        end = 0
        for p in ids:
            native = w.partition.fragments[p][0][0]
            assert (po[p] - native) % 4 == 0 and po[p] >= end and po[p] - end < 8
            end = po[p] + int(sizes[p])
        assert end <= pool_len
        prob.snapshot()
        prob.bufs.w_now.add_(torch.randn_like(prob.bufs.w_now) * 1e-3)
        before = prob.host_state()
        prob.outer_step(t_p=10, t_l=13)
        assert prob.poll() == 0
        check_step_against_oracle(prob, before, ids, 10, 13, orc_hyper(w))
        prob.last_sync.zero_()


def test_sums_of_squares_of_two_slices_give_the_whole_fragments_scores():
    """Parameter-range sharding on one GPU: two contexts each own one half of every fragment (all workers of that
    element range) over the same buffers.  Each completes its halves with COCODC_STAGE_SUMSQ, which stops Eq. 10
    at the per-fragment sums of squares; the two fp64 vectors are added (the all-reduce of a real deployment) and
    cocodc_scores_from_sumsq forms norms, scores and last_sync of the whole fragments from the totals.  Elements,
    norms and scores are compared with the oracle run on the whole fragments."""
    from paper_2504_17672_b200 import binding as B
    from helpers import check_step_against_oracle, orc_hyper
    frs = [[(4, 30_001)], [(30_009, 12_000), (60_000, 5_003)], [(42_012, 17_777)]]
    w = synth.small_workload((70_000, frs), M=3, seed=41, scale_kind="loguniform", tau=3)
    prob = GpuProblem(w, synth.generate(w, "cuda", momentum_sigma=1e-3))
    halves = ([], [])
    for f in frs:
        lo_half, hi_half = [], []
        for off, ln in f:
            cut = ln // 2 + 1
            lo_half.append((off, cut))
            hi_half.append((off + cut, ln - cut))
        halves[0].append(lo_half)
        halves[1].append(hi_half)
    ctxs = []
    for h in halves:
        wh = synth.small_workload((w.N, h), M=3, seed=41)
        ptr, off, ln = wh.partition.csr()
        ctxs.append(B.Context(w.N, ptr, off, ln, 3))
    ids = [2, 0]
    prob.set_ids(ids)
    prob.last_sync.copy_(torch.tensor([1, 0, 3], device="cuda"))
    before = prob.host_state()
    b = prob.bufs
    t_p, t_l = 9, 12
    sums = [torch.full((w.K,), -1.0, dtype=torch.float64, device="cuda") for _ in ctxs]
    for ctx, sq in zip(ctxs, sums):
        n0 = ctx.launch_count
        ctx.cocodc_outer_step(prob.hyper(), b.w_now, b.w_snap, b.now_stride, b.snap_stride, None, b.theta_g, b.momentum,
                              None, prob.ids, prob.n_ids, t_p, t_l, None, None, None,
                              stages=B.STAGE_OUTER | B.STAGE_MERGE | B.STAGE_SUMSQ, sumsq_out=sq)
        assert ctx.launch_count - n0 == 1               # plan, streaming pass and sums in one launch
        assert ctx.cocodc_poll_status() == 0
    assert float(sums[0][1]) == -1.0                    # a fragment that was not listed keeps its entry
    assert torch.equal(prob.last_sync, torch.tensor([1, 0, 3], device="cuda"))      # sums only: nothing stamped yet
    total = sums[0] + sums[1]                           # stands in for the all-reduce over the two devices
    prob.ctx.cocodc_scores_from_sumsq(total, prob.ids, prob.n_ids, None, t_p, t_l, prob.last_sync, prob.norms,
                                      prob.scores)
    assert prob.poll() == 0
    check_step_against_oracle(prob, before, ids, t_p, t_l, orc_hyper(w))
    # the sums themselves against the oracle's
    res, _ = orc.outer_step(fragments_of(w), orc_hyper(w), before["w_now"], before["w_snap"], before["theta_g"],
                            before["momentum"], ids, t_p, t_l, before["last_sync"])
    for p in ids:
        assert abs(float(total[p]) - res[p].sumsq) <= 2e-6 * res[p].sumsq
    # stand-alone form: sums of squares of a vector, then scores from them with intervals
    x = torch.randn(w.N, device="cuda", generator=torch.Generator(device="cuda").manual_seed(3)) * 1e-2
    sq = torch.zeros(w.K, dtype=torch.float64, device="cuda")
    n0 = prob.ctx.launch_count
    prob.ctx.cocodc_fragment_scores(x, None, None, None, sumsq_out=sq)
    assert prob.ctx.launch_count - n0 == 1
    exp_sq = orc.fragment_sumsq(fragments_of(w), np_(x))
    assert np.all(np.abs(np_(sq) - exp_sq) <= 2e-6 * exp_sq)
    iv = torch.tensor([4, 0, 9], dtype=torch.int64, device="cuda")
    norms = torch.zeros(w.K, device="cuda")
    scores = torch.zeros(w.K, device="cuda")
    prob.ctx.cocodc_scores_from_sumsq(sq, None, None, iv, 0, 0, None, norms, scores)
    en, es = orc.fragment_scores(fragments_of(w), np_(x), np_(iv))
    assert np.all(np.abs(np_(norms) - en) <= TOL_NORM * en) and np.all(np.abs(np_(scores) - es) <= TOL_NORM * es)
    assert prob.poll() == 0
    # a fragment table too large to travel as a kernel argument takes the plan kernel as well
    big = synth.small_workload([300] * 200, M=1, seed=1)
    ptr, off, ln = big.partition.csr()
    cbig = B.Context(big.N, ptr, off, ln, 1)
    xb = torch.ones(big.N, device="cuda")
    nb = torch.zeros(200, device="cuda")
    n0 = cbig.launch_count
    cbig.cocodc_fragment_scores(xb, None, nb, nb.clone())
    assert cbig.launch_count - n0 == 2 and cbig.cocodc_poll_status() == 0
    assert np.allclose(np_(nb), np.sqrt(300.0), rtol=1e-6)


@pytest.mark.parametrize("case", range(10))
def test_initiate_equals_selection_followed_by_snapshot(case):
    """cocodc_initiate (Algorithm 2 and the snapshot of what it picks in one launch) against the two separate calls
    and, through them, the oracle: bit for bit on mask, ids, count, pool places, in-flight marks and every word of
    the snapshot pool.  Random schedule states: overdue fragments, never-synced ones, ties, ineligible and in-flight
    fragments, both walked budgets, with and without a pool; the tenth case has a table too large for one launch."""
    from paper_2504_17672_b200 import binding as B
    rng = np.random.default_rng(700 + case)
    K = 150 if case == 9 else int(rng.integers(1, 41))
    sizes = rng.choice([3, 64, 1000, 1025, 4096, 9000, 20_001], size=K).tolist()
    frs, pos = [], int(rng.integers(0, 4))
    for s_ in sizes:
        frs.append([(pos, int(s_))])
        pos += int(s_) + int(rng.choice([0, 1, 2, 5]))
    M = int(rng.integers(1, 4))
    w = synth.small_workload((pos + 8 - pos % 4, frs), M=M, seed=case)
    ptr, off, ln = w.partition.csr()
    bufs = synth.generate(w, "cuda")
    scores_h = rng.choice([0.5, 1.0, 1.0, 2.5, 7.0, np.inf], size=K).astype(np.float32) * rng.choice([1.0, 1.0, 3.0], size=K).astype(np.float32)
    last_h = rng.integers(0, 160, size=K).astype(np.int64)
    inel_h = (rng.random(K) < 0.15).astype(np.uint8)
    flight_h = (rng.random(K) < 0.15).astype(np.uint8)
    t_now, H = 200, 100
    kind = int(rng.integers(0, 2))
    budget = int(rng.integers(1, 6)) if kind == 0 else int(rng.integers(1, max(2, sum(sizes) // 2)))
    use_pool = bool(rng.integers(0, 2)) or True if case % 3 else False
    pool_len = (sum(sizes) + 8 * K + 1023) // 1024 * 1024
    out = {}
    for name in ("two_calls", "initiate"):
        ctx = B.Context(w.N, ptr, off, ln, M)
        scores = torch.from_numpy(scores_h).cuda()
        last = torch.from_numpy(last_h).cuda()
        inel = torch.from_numpy(inel_h).cuda()
        flight = torch.from_numpy(flight_h.copy()).cuda()
        ctx.cocodc_bind_in_flight(flight)
        mask = torch.full((K,), 9, dtype=torch.uint8, device="cuda")
        ids = torch.full((K,), 77, dtype=torch.int32, device="cuda")
        n_sel = torch.full((1,), -5, dtype=torch.int32, device="cuda")
        pool_off = torch.full((K,), 123, dtype=torch.int64, device="cuda") if use_pool else None
        snap = (torch.full((M, pool_len), -3.0, device="cuda") if use_pool
                else torch.full((M, w.N), -3.0, device="cuda"))
        n0 = ctx.launch_count
        if name == "two_calls":
            ctx.cocodc_select_fragments(scores, last, inel, t_now, H, kind, budget, mask, ids, n_sel, pool_off)
            ctx.cocodc_snapshot(bufs.w_now, snap, bufs.now_stride, snap.stride(0), pool_off, M, ids, n_sel)
        else:
            ctx.cocodc_initiate(scores, last, inel, t_now, H, kind, budget, mask, ids, n_sel, pool_off, bufs.w_now, snap,
                                bufs.now_stride, snap.stride(0), M)
            assert ctx.launch_count - n0 == (1 if K <= 128 else 3)      # beyond the limit: select, plan, snapshot
        assert ctx.cocodc_poll_status() == 0
        out[name] = dict(mask=np_(mask), ids=np_(ids), n=int(n_sel.item()), flight=np_(flight),
                         pool_off=None if pool_off is None else np_(pool_off), snap=np_(snap))
        ctx.close()
    a, b = out["two_calls"], out["initiate"]
    assert a["n"] == b["n"] and np.array_equal(a["mask"], b["mask"]) and np.array_equal(a["ids"], b["ids"])
    assert np.array_equal(a["flight"], b["flight"])
    if use_pool:
        assert np.array_equal(a["pool_off"], b["pool_off"])
    assert np.array_equal(a["snap"], b["snap"])
    # and against the oracle
    emask, eids, en = orc.select_fragments(scores_h, last_h, np.array(sizes), t_now, H, kind, budget,
                                           ineligible=np.maximum(inel_h, flight_h))
    assert b["n"] == en and b["ids"][:en].tolist() == eids.tolist() and np.array_equal(b["mask"], emask)
    assert np.array_equal(b["flight"], np.maximum(flight_h, emask))
    exp = orc.snapshot(fragments_of(w), np_(bufs.w_now), eids, M, b["pool_off"],
                       np.full(b["snap"].shape, -3.0, dtype=np.float32))
    assert np.array_equal(b["snap"], exp)


def test_initiate_rejects_nan_scores_and_takes_the_enumerating_budget_in_two_launches():
    from paper_2504_17672_b200 import binding as B
    w = synth.small_workload([4096, 5000, 776], M=2, seed=4)
    ptr, off, ln = w.partition.csr()
    ctx = B.Context(w.N, ptr, off, ln, 2)
    bufs = synth.generate(w, "cuda")
    K = 3
    scores = torch.tensor([1.0, float("nan"), 2.0], device="cuda")
    last = torch.zeros(K, dtype=torch.int64, device="cuda")
    mask = torch.zeros(K, dtype=torch.uint8, device="cuda")
    ids = torch.zeros(K, dtype=torch.int32, device="cuda")
    n_sel = torch.ones(1, dtype=torch.int32, device="cuda")
    snap = torch.full((2, w.N), -1.0, device="cuda")
    ctx.cocodc_initiate(scores, last, None, 5, 100, B.BUDGET_COUNT, 2, mask, ids, n_sel, None, bufs.w_now, snap,
                        bufs.now_stride, snap.stride(0), 2)
    assert ctx.cocodc_poll_status() == B.ERR_NONFINITE
    assert int(n_sel.item()) == 0 and bool((snap == -1.0).all())
    scores[1] = 0.5
    n0 = ctx.launch_count
    ctx.cocodc_initiate(scores, last, None, 5, 100, B.BUDGET_PARAMS_EXACT, 6000, mask, ids, n_sel, None, bufs.w_now,
                        snap, bufs.now_stride, snap.stride(0), 2)
    assert ctx.launch_count - n0 == 2 and ctx.cocodc_poll_status() == 0
    _, eids, en = orc.select_fragments(np_(scores), np_(last), w.partition.frag_sizes, 5, 100,
                                       orc.BUDGET_PARAMS_EXACT, 6000)
    assert np_(ids)[:en].tolist() == eids.tolist()
