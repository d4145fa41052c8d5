"""The N > 1 host logic of the benchmark on CPU: two gloo ranks, no GPU.

Ranks own independent shards (weak scaling, no data-path collective); what crosses ranks is only the
timing reduction: units are summed, time is the maximum."""

import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    import synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.dist_env() == (rank, world, rank)
        # each rank reports different local figures; the job figure is (sum of units, max of seconds)
        units, seconds = bench.aggregate(100.0 * (rank + 1), 2.0 + rank, world, True)
        assert units == 300.0 and seconds == 3.0
        # a fixed list of problems splits into disjoint contiguous blocks that cover it
        lo, hi = bench.shard_units(13, world, rank)
        spans = [None] * world
        dist.all_gather_object(spans, (lo, hi))
        assert spans[0][0] == 0 and spans[-1][1] == 13 and all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
        # ranks own different shards of the same shape: same fragment table, different seeded values
        w = synth.small_workload([1000, 2000], M=2, seed=7)
        mine = synth.generate(w.with_(seed=w.seed + 1000 * rank), "cpu")
        sums = [None] * world
        dist.all_gather_object(sums, float(mine.theta_g.double().sum()))
        assert sums[0] != sums[1]
        # the selection decision is deterministic on every rank given the same history (Section 3.2)
        from oracle import reference as orc
        sel = orc.select_fragments([1.0, 2.0], [0, 0], [1000, 2000], 5, 100, 0, 1)[1].tolist()
        allsel = [None] * world
        dist.all_gather_object(allsel, sel)
        assert allsel[0] == allsel[1] == [1]
        # worker-per-device deployment: the listed fragments' ranges of the per-rank sums are all-reduced in place
        from paper_2504_17672_b200 import distributed as D
        frs = [[(3, 100), (700, 57)], [(103, 250)], [(400, 299)]]
        ranges = D.fragment_ranges(frs, [2, 0])
        assert ranges == [(400, 299), (3, 100), (700, 57)]
        buf = torch.full((1000,), float(rank + 1))
        calls = D.allreduce_ranges(buf, ranges, bucket_elems=128)
        assert calls == 3 + 1 + 1
        exp = torch.full((1000,), float(rank + 1))
        for o, l in ranges:
            exp[o:o + l] = 3.0                                    # 1 + 2 summed over the two ranks
        assert torch.equal(buf, exp)
        # parameter-range sharding: every rank holds a slice of each fragment; what crosses ranks is one all-reduce
        # of the K fp64 sums of squares, after which the library forms the scores (a recording stand-in here)
        full = torch.arange(1, 13, dtype=torch.float64).reshape(3, 4)          # 3 fragments of 4 elements
        mine = (full[:, 2 * rank:2 * rank + 2] ** 2).sum(dim=1)                # this rank's half of every sum
        seen = {}

        class Recorder:
            def cocodc_scores_from_sumsq(self, sumsq, ids, n_ids, interval, t_p, t_l, last_sync, norms, scores):
                seen.update(sumsq=sumsq.clone(), args=(ids, n_ids, interval, t_p, t_l, last_sync, norms, scores))

        D.scores_from_sharded_sumsq(Recorder(), mine, "ids", "n", 7, 11, "last", "norms", "scores")
        assert torch.equal(seen["sumsq"], (full ** 2).sum(dim=1))
        assert seen["args"] == ("ids", "n", None, 7, 11, "last", "norms", "scores")
        out.put((rank, "ok"))
    except Exception as e:  # pragma: no cover
        out.put((rank, repr(e)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_aggregate_like_the_benchmark():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=120)
    results = sorted(out.get(timeout=5) for _ in range(2))
    assert results == [(0, "ok"), (1, "ok")], results


def test_reference_arm_runs_only_on_rank_zero(monkeypatch, capsys):
    import bench

    class A:
        workload = "tiny"; steps = 1; warmup = 0; reference_sample = 20_000

    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")
    bench.run_reference(A)
    assert capsys.readouterr().out == ""
    monkeypatch.setenv("RANK", "0")
    bench.run_reference(A)
    import json
    line = json.loads(capsys.readouterr().out)
    assert line["impl"] == "reference" and line["value"] > 0 and line["e2e"]["h2d_bytes_per_step"] == 0


def test_peer_glue_orders_sum_barrier_step_barrier():
    """complete_fragments_peers (host logic only, a recording stand-in for the context): this rank's sum goes to its
    own buffer, a barrier separates it from the step that reads every rank's buffer in rank order, and a second
    barrier keeps the buffers alive until every rank has read them."""
    from types import SimpleNamespace
    import torch
    from paper_2504_17672_b200 import distributed as D
    log = []

    class Recorder:
        def cocodc_pseudo_gradient_sum(self, w_snap, stride, snap_offset, theta_g, M, out, ids, n_ids):
            log.append(("sum", out, M))

        def cocodc_outer_step_received_peers(self, hyper, M_total, w_now, w_snap, ns, ss, so, thg, mom, sums, dout,
                                             ids, n_ids, t_p, t_l, last, norms, scores):
            log.append(("step", list(sums), M_total, t_p, t_l))

    bufs = ["rank0-buffer", "rank1-buffer", "rank2-buffer"]
    t = torch.zeros(2, 8)
    D.complete_fragments_peers(Recorder(), SimpleNamespace(M=2), 6, 1, bufs, None, None, t, t, None, None, None, 4, 7,
                               None, None, None, lambda: log.append(("barrier",)))
    assert [x[0] for x in log] == ["sum", "barrier", "step", "barrier"]
    assert log[0][1] == "rank1-buffer" and log[0][2] == 2
    assert log[2][1] == bufs and log[2][2:] == (6, 4, 7)


def _run_bench(*argv, timeout=300):
    import subprocess
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *argv], capture_output=True, text=True,
                          timeout=timeout)


def test_gpus_flag_launches_that_many_ranks():
    """`python bench.py --gpus 2` started plainly launches two ranks itself; with the CPU stand-in step the whole
    launch path (launcher, process group, barrier, reduction, rank 0's line) runs here over gloo."""
    import json
    r = _run_bench("--gpus", "2", "--stub-step", "--steps", "4")
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][-1])
    assert line["n_gpus"] == 2 and line["units"] == 4 * 1000.0 * (1 + 2)


def test_gpus_flag_reaches_the_device_check_in_every_rank():
    """Without CUDA devices the real benchmark must fail loudly in BOTH ranks (no rank silently runs elsewhere)."""
    if torch.cuda.is_available():
        pytest.skip("this box has a GPU")
    r = _run_bench("--gpus", "2", "--steps", "1", "--no-e2e", "--no-cpu-baseline")
    assert r.returncode != 0
    assert "rank 0: no CUDA device" in r.stderr and "rank 1: no CUDA device" in r.stderr
