"""The synthetic workloads: fragment tables and seeded buffers (no method arithmetic here)."""

import numpy as np
import torch

import synth


def test_workload_shapes():
    expect = {
        "tiny": (1_048_576, 8, 2),
        "gpt2_small": (124_439_808, 13, 4),
        "llama_1b": (953_223_168, 16, 4),
        "sweep_1b": (953_223_168, 32, 4),
        "llama_3b": (3_426_473_600, 27, 4),
        "paper_150m": (154_165_248, 4, 4),
    }
    for name, (N, K, M) in expect.items():
        w = synth.get_workload(name)
        assert (w.N, w.K, w.M) == (N, K, M)
        assert int(w.partition.frag_sizes.sum()) == N
        ptr, off, ln = w.partition.csr()
        assert ptr[-1] == len(off) == len(ln) == w.partition.n_segments
    g = synth.get_workload("gpt2_small")
    assert g.partition.frag_size(0) == 39_385_344 and g.partition.frag_size(1) == 7_087_872
    assert g.budget == 31_109_952
    l1 = synth.get_workload("llama_1b").partition
    assert l1.frag_size(0) == 116_920_320 and l1.frag_size(1) == 51_384_320 and l1.frag_size(15) == 116_922_368
    l3 = synth.get_workload("llama_3b")
    assert l3.partition.frag_size(0) == 123_910_400 and l3.partition.frag_size(26) == 204_803_200
    assert l3.budget == 1_027_942_080
    assert synth.get_workload("sweep_1b").partition.frag_size(7) == 29_788_224


def test_named_workloads_have_no_tiny_fragments():
    """The parity helpers measure fragments of fewer than 64 elements against their operands (test partitions
    only); every named workload stays far above that, so its parity is always relative to the outputs."""
    for name in synth.WORKLOAD_NAMES:
        assert int(synth.get_workload(name).partition.frag_sizes.min()) >= 131_072, name


def test_generate_is_seeded_and_layout_independent():
    w = synth.small_workload((1000, [[(3, 100), (700, 57)], [(103, 250)], [(400, 299)]]), M=3, seed=5,
                             scale_kind="loguniform")
    a = synth.generate(w, "cpu", momentum_sigma=1e-3)
    b = synth.generate(w, "cpu", momentum_sigma=1e-3)
    for x, y in ((a.theta_g, b.theta_g), (a.w_now, b.w_now), (a.w_snap, b.w_snap), (a.momentum, b.momentum)):
        assert torch.equal(x, y)
    c = synth.generate(w.with_(seed=6), "cpu")
    assert not torch.equal(a.theta_g, c.theta_g)
    pool = synth.generate(w, "cpu", snap_layout="pool", pool_ids=[2, 0], momentum_sigma=1e-3)
    assert torch.equal(pool.w_now, a.w_now) and torch.equal(pool.theta_g, a.theta_g)
    off = pool.snap_offset.tolist()
    assert off[1] == -1 and off[2] == 0 and off[0] == 300
    assert torch.equal(pool.w_snap[:, 0:299], a.w_snap[:, 400:699])
    assert torch.equal(pool.w_snap[:, 300:400], a.w_snap[:, 3:103])
    assert torch.equal(pool.w_snap[:, 400:457], a.w_snap[:, 700:757])


def test_value_scales_follow_the_recipe():
    w = synth.small_workload([200_000, 200_000], M=2, seed=1)
    d = synth.generate(w, "cpu")
    assert abs(float(d.theta_g.std()) - 0.02) < 5e-4
    assert abs(float((d.w_snap[0] - d.theta_g).std()) - 1e-3) < 5e-5
    drift = d.w_now - d.w_snap
    assert abs(float(drift[0].std()) - 1e-3 * np.sqrt(1.01)) < 5e-5
    # the common movement dominates: workers' changes over the delay are strongly correlated
    assert float(torch.corrcoef(drift)[0, 1]) > 0.95
    s = synth.fragment_scales(synth.get_workload("llama_3b"))
    assert s.shape == (27,) and s.min() >= 1e-6 and s.max() <= 1.0
    s2 = synth.fragment_scales(synth.get_workload("gpt2_small"))
    assert s2.min() >= 1e-4 and s2.max() <= 1e-2
