"""A completion that leaves Eq. 10's last steps to the next selection (COCODC_STAGE_DEFER): whatever forms the scores
afterwards - the prologue of cocodc_initiate, the small launch placed before other calls, cocodc_flush_scores - the
results are bit for bit those of the undeferred stage, which the other parity tests hold to the oracle; the first
test also checks the deferred route against the oracle directly."""

import numpy as np
import pytest
import torch

import synth
from oracle import reference as orc
from helpers import GpuProblem, check_step_against_oracle, np_, orc_hyper

pytestmark = pytest.mark.gpu

RAGGED = (60_000, [[(3, 9_001), (40_010, 4_097)], [(9_004, 12_345)], [(21_349, 5)], [(21_360, 18_640)],
                   [(44_111, 15_000)]])
MANY_TILES = (1_300_000, [[(4, 600_001)], [(600_008, 650_000)], [(1_250_009, 40_000)]])
DEFER = 7 | 16          # COCODC_STAGE_ALL | COCODC_STAGE_DEFER


def make(M, seed, frs=RAGGED, **kw):
    w = synth.small_workload(frs, M=M, seed=seed, scale_kind="loguniform")
    prob = GpuProblem(w, synth.generate(w, "cuda", momentum_sigma=1e-3, **kw))
    prob.flight = torch.zeros(w.K, dtype=torch.uint8, device="cuda")
    prob.ctx.cocodc_bind_in_flight(prob.flight)
    return prob


def schedule_state(prob):
    return [np_(x).copy() for x in (prob.norms, prob.scores, prob.last_sync, prob.flight)]


@pytest.mark.parametrize("M,frs,same", [(4, RAGGED, False), (2, MANY_TILES, False), (4, MANY_TILES, True),
                                         (1, RAGGED, True), (9, MANY_TILES, False), (49, RAGGED, False)])
def test_flush_forms_what_the_undeferred_stage_forms(M, frs, same):
    """Staged kernel, in-place kernel, staged kernel at zero delay, chunk-ring kernel, element loop."""
    ids = [2, 0] if frs is MANY_TILES else [3, 0, 4]
    out = {}
    for name, stages in (("plain", 7), ("deferred", DEFER)):
        prob = make(M, seed=900 + M, frs=frs)
        prob.set_ids(ids)
        prob.flight[ids] = 1
        prob.last_sync.copy_(torch.arange(prob.w.K, dtype=torch.int64, device="cuda"))
        before = prob.host_state()
        was = schedule_state(prob)
        n0 = prob.ctx.launch_count
        kw = dict(hyper=prob.hyper(tau=0), w_snap=prob.bufs.w_now) if same else {}
        t_p, t_l = (30, 30) if same else (30, 34)
        prob.outer_step(t_p, t_l, stages=stages, **kw)
        if name == "deferred":
            torch.cuda.synchronize()
            for x, y in zip(was, schedule_state(prob)):       # nothing of the schedule state has moved yet
                assert np.array_equal(x, y)
            prob.ctx.cocodc_flush_scores()
            assert prob.ctx.launch_count - n0 == 2
            prob.ctx.cocodc_flush_scores()                    # nothing outstanding: no launch
            assert prob.ctx.launch_count - n0 == 2
            ohp = orc_hyper(prob.w, tau=0) if same else orc_hyper(prob.w)
            check_step_against_oracle(prob, before, ids, t_p, t_l, ohp, same=same)
        assert prob.poll() == 0
        out[name] = schedule_state(prob) + [np_(prob.bufs.w_now), np_(prob.bufs.theta_g), np_(prob.bufs.momentum)]
        assert not out[name][3][ids].any()                    # the completion clears its in-flight marks
        assert (out[name][2][ids] == t_l).all()
    for x, y in zip(out["plain"], out["deferred"]):
        assert np.array_equal(x, y)


@pytest.mark.parametrize("case", range(8))
def test_initiate_after_a_deferred_completion_equals_the_undeferred_pair(case):
    """Completion + initiation as two launches, the scores formed in the second one's prologue: every output of both
    calls bit-identical to the undeferred pair, and the selection equal to the oracle's on the oracle's own scores."""
    from paper_2504_17672_b200 import binding as B
    rng = np.random.default_rng(4000 + case)
    K = int(rng.integers(3, 30))
    sizes = rng.choice([64, 1000, 1025, 4096, 9000, 20_001], size=K).tolist()
    frs, pos = [], 0
    for s_ in sizes:
        frs.append([(pos, int(s_))])
        pos += int(s_) + int(rng.choice([0, 4, 8]))
    M = int(rng.integers(1, 5))
    n_done = int(rng.integers(1, min(K, 5)))
    done = [int(x) for x in rng.choice(K, size=n_done, replace=False)]
    scores_h = rng.choice([1e-4, 1e-3, 1e-2, np.inf], size=K).astype(np.float32)
    last_h = rng.integers(0, 120, size=K).astype(np.int64)
    flight_h = (rng.random(K) < 0.2).astype(np.uint8)
    flight_h[done] = 1
    kind = int(rng.integers(0, 2))
    budget = int(rng.integers(1, 5)) if kind == 0 else int(rng.integers(1, max(2, sum(sizes) // 2)))
    t_p, t_l, H = 130, 134, 100
    pool_len = (sum(sizes) + 8 * K + 1023) // 1024 * 1024
    out = {}
    for name, stages in (("plain", 7), ("deferred", DEFER)):
        w = synth.small_workload(((pos + 11) // 4 * 4, frs), M=M, seed=case, scale_kind="loguniform")
        prob = GpuProblem(w, synth.generate(w, "cuda", snap_layout="pool", pool_ids=done, momentum_sigma=1e-3))
        prob.flight = torch.from_numpy(flight_h.copy()).cuda()
        prob.ctx.cocodc_bind_in_flight(prob.flight)
        prob.scores.copy_(torch.from_numpy(scores_h))
        prob.last_sync.copy_(torch.from_numpy(last_h))
        prob.set_ids(done)
        before = prob.host_state()
        b = prob.bufs
        n0 = prob.ctx.launch_count
        prob.outer_step(t_p, t_l, stages=stages)
        # the next set is recorded into a second pool, so that the first one can still be compared
        pool2 = torch.full((M, pool_len), -3.0, device="cuda")
        off2 = torch.full((K,), 123, dtype=torch.int64, device="cuda")
        ids2 = torch.full((K,), 77, dtype=torch.int32, device="cuda")
        n2 = torch.full((1,), -5, dtype=torch.int32, device="cuda")
        prob.ctx.cocodc_initiate(prob.scores, prob.last_sync, None, t_l, H, kind, budget, prob.mask, ids2, n2, off2,
                                 b.w_now, pool2, b.now_stride, pool2.stride(0), M)
        assert prob.ctx.launch_count - n0 == 2
        assert prob.poll() == 0
        out[name] = dict(norms=np_(prob.norms), scores=np_(prob.scores), last=np_(prob.last_sync),
                         flight=np_(prob.flight), mask=np_(prob.mask), ids=np_(ids2), n=int(n2.item()), off=np_(off2),
                         pool=np_(pool2), w_now=np_(b.w_now), theta_g=np_(b.theta_g), momentum=np_(b.momentum))
        if name == "deferred":
            check_step_against_oracle(prob, before, done, t_p, t_l, orc_hyper(w))
    a, d = out["plain"], out["deferred"]
    for k in a:
        assert np.array_equal(a[k], d[k]), k
    # the decision itself, from the device's scores (their parity with the oracle is checked above)
    inel = flight_h.copy()
    inel[done] = 0
    emask, eids, en = orc.select_fragments(d["scores"], d["last"], np.array(sizes), t_l, H, kind, budget, ineligible=inel)
    assert d["n"] == en and d["ids"][:en].tolist() == eids.tolist() and np.array_equal(d["mask"], emask)
    assert np.array_equal(d["flight"], np.maximum(inel, emask))
    assert (d["last"][done] == t_l).all()


def test_calls_that_do_not_consume_a_deferred_completion_form_its_scores_first():
    """A second completion, a selection given other arrays, the stand-alone selection, stand-alone scoring: each is
    preceded by the one small launch, and the results equal the undeferred sequence."""
    from paper_2504_17672_b200 import binding as B
    out = {}
    for name, stages in (("plain", 7), ("deferred", DEFER)):
        prob = make(4, seed=77, frs=MANY_TILES)
        b = prob.bufs
        extra = 1 if name == "deferred" else 0
        # two completions in a row
        prob.set_ids([1])
        n0 = prob.ctx.launch_count
        prob.outer_step(10, 14, stages=stages)
        prob.set_ids([2, 0])
        prob.outer_step(14, 18, stages=stages)
        assert prob.ctx.launch_count - n0 == 2 + extra
        # a selection that reads a copy of the scores: not the consumer of the pending completion
        other = torch.tensor([0.1, 0.5, 0.3], device="cuda")
        ids2 = torch.full((prob.w.K,), -1, dtype=torch.int32, device="cuda")
        n2 = torch.zeros(1, dtype=torch.int32, device="cuda")
        n0 = prob.ctx.launch_count
        prob.ctx.cocodc_initiate(other, prob.last_sync, None, 18, 100, B.BUDGET_COUNT, 1, prob.mask, ids2, n2,
                                 None, b.w_now, b.w_snap, b.now_stride, b.snap_stride, 4)
        assert prob.ctx.launch_count - n0 == 1 + extra
        first = dict(scores=np_(prob.scores).copy(), last=np_(prob.last_sync).copy(), ids=np_(ids2).copy())
        # the stand-alone selection after a deferred completion of what was just recorded
        prob.set_ids([int(ids2[0].item())])
        n0 = prob.ctx.launch_count
        prob.outer_step(18, 22, stages=stages)
        prob.ctx.cocodc_select_fragments(prob.scores, prob.last_sync, None, 22, 100, B.BUDGET_COUNT, 2, prob.mask,
                                         ids2, n2)
        assert prob.ctx.launch_count - n0 == 2 + extra
        # stand-alone scoring writes the same arrays
        prob.set_ids([0])
        prob.outer_step(22, 26, stages=stages)
        delta = torch.randn(prob.w.N, generator=torch.Generator().manual_seed(11)).cuda()
        n0 = prob.ctx.launch_count
        prob.ctx.cocodc_fragment_scores(delta, None, prob.norms, prob.scores)
        assert prob.ctx.launch_count - n0 == 1 + extra
        assert prob.poll() == 0
        out[name] = dict(first, norms=np_(prob.norms), scores2=np_(prob.scores), last2=np_(prob.last_sync),
                         flight=np_(prob.flight), ids2=np_(ids2), w_now=np_(b.w_now), theta_g=np_(b.theta_g))
    for k in out["plain"]:
        assert np.array_equal(out["plain"][k], out["deferred"][k]), k


def test_deferred_completion_with_a_table_too_large_for_one_launch():
    """150 fragments: the plan comes from its own kernel and cocodc_initiate takes its three-launch route, which forms
    the outstanding scores before it selects."""
    from paper_2504_17672_b200 import binding as B
    rng = np.random.default_rng(5)
    sizes = rng.choice([64, 1000, 4096], size=150).tolist()
    frs, pos = [], 0
    for s_ in sizes:
        frs.append([(pos, int(s_))])
        pos += int(s_)
    out = {}
    for name, stages in (("plain", 7), ("deferred", DEFER)):
        w = synth.small_workload((pos, frs), M=2, seed=3, scale_kind="loguniform")
        prob = GpuProblem(w, synth.generate(w, "cuda", momentum_sigma=1e-3))
        b = prob.bufs
        done = [149, 3, 77]
        prob.set_ids(done)
        before = prob.host_state()
        n0 = prob.ctx.launch_count
        prob.outer_step(5, 9, stages=stages)
        ids2 = torch.full((150,), -1, dtype=torch.int32, device="cuda")
        n2 = torch.zeros(1, dtype=torch.int32, device="cuda")
        snap2 = torch.zeros_like(b.w_snap)
        prob.ctx.cocodc_initiate(prob.scores, prob.last_sync, None, 9, 100, B.BUDGET_COUNT, 3, prob.mask, ids2, n2, None,
                                 b.w_now, snap2, b.now_stride, b.snap_stride, 2)
        assert prob.ctx.launch_count - n0 == 2 + 3 + (1 if name == "deferred" else 0)
        assert prob.poll() == 0
        if name == "deferred":
            check_step_against_oracle(prob, before, done, 5, 9, orc_hyper(w))
        out[name] = [np_(x) for x in (prob.norms, prob.scores, prob.last_sync, ids2, n2, snap2)]
    for x, y in zip(out["plain"], out["deferred"]):
        assert np.array_equal(x, y)


def test_deferred_schedule_step_replayed_from_a_cuda_graph_equals_eager_undeferred_steps():
    """[completion with its scores deferred, initiation] recorded once with device-resident step numbers and replayed."""
    w = synth.get_workload("tiny")
    from paper_2504_17672_b200 import binding as B

    def fresh():
        prob = GpuProblem(w, synth.generate(w, "cuda", snap_layout="pool", pool_ids=[0, 1], momentum_sigma=1e-3))
        prob.pool_off = prob.bufs.snap_offset
        prob.flight = torch.zeros(w.K, dtype=torch.uint8, device="cuda")
        prob.flight[:2] = 1
        prob.ctx.cocodc_bind_in_flight(prob.flight)
        prob.scores.copy_(torch.arange(w.K, 0, -1, dtype=torch.float32, device="cuda"))
        prob.set_ids([0, 1])
        return prob

    tau = w.tau
    a = fresh()
    t = 10
    for _ in range(5):
        b = a.bufs
        a.ctx.cocodc_outer_step(a.hyper(), b.w_now, b.w_snap, b.now_stride, b.snap_stride, a.pool_off, b.theta_g,
                                b.momentum, None, a.ids, a.n_ids, t, t + tau, a.last_sync, a.norms, a.scores)
        t += tau
        a.ctx.cocodc_initiate(a.scores, a.last_sync, None, t, w.H, B.BUDGET_COUNT, w.budget, a.mask, a.ids, a.n_ids,
                              a.pool_off, b.w_now, b.w_snap, b.now_stride, b.snap_stride, w.M)
    assert a.poll() == 0

    g = fresh()
    clock = torch.tensor([10, 10 + tau], dtype=torch.int64, device="cuda")

    def step():
        b = g.bufs
        g.ctx.cocodc_outer_step_at(g.hyper(), b.w_now, b.w_snap, b.now_stride, b.snap_stride, g.pool_off, b.theta_g,
                                   b.momentum, None, g.ids, g.n_ids, clock[0:1], clock[1:2], g.last_sync, g.norms,
                                   g.scores, DEFER)
        g.ctx.cocodc_initiate_at(g.scores, g.last_sync, None, clock[1:2], w.H, B.BUDGET_COUNT, w.budget, g.mask,
                                 g.ids, g.n_ids, g.pool_off, b.w_now, b.w_snap, b.now_stride, b.snap_stride, w.M)
        clock.add_(tau)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    n0 = g.ctx.launch_count
    with torch.cuda.graph(graph):
        step()
    assert g.ctx.launch_count - n0 == 2
    for _ in range(4):
        graph.replay()
    torch.cuda.synchronize()
    assert g.poll() == 0
    for x, y in ((a.bufs.w_now, g.bufs.w_now), (a.bufs.theta_g, g.bufs.theta_g), (a.bufs.momentum, g.bufs.momentum),
                 (a.bufs.w_snap, g.bufs.w_snap), (a.scores, g.scores), (a.norms, g.norms), (a.last_sync, g.last_sync),
                 (a.ids, g.ids), (a.flight, g.flight)):
        assert torch.equal(x, y)


def test_deferring_is_refused_where_it_has_no_meaning():
    prob = make(4, seed=1)
    prob.set_ids([0])
    B = prob.B
    b = prob.bufs
    sums = torch.zeros(prob.w.K, dtype=torch.float64, device="cuda")

    def code(stages, sumsq_out=None):
        try:
            prob.ctx.cocodc_outer_step(prob.hyper(), b.w_now, b.w_snap, b.now_stride, b.snap_stride, None, b.theta_g,
                                       b.momentum, None, prob.ids, prob.n_ids, 1, 3, prob.last_sync, prob.norms,
                                       prob.scores, stages, sumsq_out=sumsq_out)
        except B.CocodcError as e:
            return e.code
        return 0

    assert code(1 | 2 | 16) == B.ERR_INVALID_ARG              # nothing to defer without the SCORE stage
    assert code(7 | 8 | 16, sums) == B.ERR_INVALID_ARG         # the sums themselves are not handed out
    assert code(7 | 16, sums) == B.ERR_INVALID_ARG
    assert code(7 | 32) == B.ERR_INVALID_ARG
    assert prob.ctx.launch_count == 0
    assert code(7 | 16) == 0
    prob.ctx.cocodc_flush_scores()
    assert prob.poll() == 0
    assert float(prob.norms[0].item()) > 0.0


def test_a_status_poll_that_reports_an_error_drops_the_outstanding_completion():
    """After an error the outputs of the launches before the poll are undefined; the scores a deferred completion left
    unformed are then not formed later either (the error here is the self-test's bounded wait running out)."""
    prob = make(4, seed=2)
    prob.set_ids([1, 3])
    prob.outer_step(4, 8, stages=DEFER)
    was = schedule_state(prob)
    prob.ctx.cocodc_selftest_bounded_wait(2000)
    assert prob.poll() == prob.B.ERR_TIMEOUT
    n0 = prob.ctx.launch_count
    prob.ctx.cocodc_flush_scores()
    assert prob.ctx.launch_count == n0
    torch.cuda.synchronize()
    for x, y in zip(was, schedule_state(prob)):
        assert np.array_equal(x, y)
    # the context is usable as before
    before = prob.host_state()
    prob.outer_step(8, 12, stages=DEFER)
    prob.ctx.cocodc_flush_scores()
    assert prob.poll() == 0
    check_step_against_oracle(prob, before, [1, 3], 8, 12, orc_hyper(prob.w))
