"""cocodc_fragment_scores_noalloc against the CPU oracle and against cocodc_fragment_scores.

The no-allocation entry point serves callers that are not allowed to allocate device memory (code
inside an allocator hook, processes with a closed device heap, allocation-free hot paths): it keeps
its scratch in a fixed array inside the library instead of context memory.  This file is collected
last on purpose, so that a run that stops at the first failure has already run every other test.
"""

import numpy as np
import pytest
import torch

import synth
from oracle import reference as orc
from helpers import TOL_NORM, np_

pytestmark = pytest.mark.gpu

FRAGMENTS = (700_000, [[(1, 170_001), (500_003, 999)], [(170_002, 229_998)], [(400_000, 100_000)], [(501_002, 98_000)],
                       [(650_000, 7)]])


def test_noalloc_scores_match_the_context_entry_point_on_two_calls_in_a_row():
    from paper_2504_17672_b200 import binding as B
    w = synth.small_workload(FRAGMENTS, M=1, seed=9)
    ptr, off, ln = w.partition.csr()
    K = w.K
    ctx = B.Context(w.N, ptr, off, ln, 1)
    gen = torch.Generator(device="cuda").manual_seed(21)
    interval = torch.tensor([0, 3, 100, 7, 1], dtype=torch.int64, device="cuda")
    frs = [list(f) for f in w.partition.fragments]
    # the second call sees different data and a fragment of zeros: nothing of the first call may leak through
    for call in range(2):
        x = torch.randn(w.N, generator=gen, device="cuda") * (1e-3 if call == 0 else 5e-2)
        if call == 1:
            x[400_000:500_000] = 0.0
        ref_n = torch.zeros(K, device="cuda")
        ref_s = torch.zeros(K, device="cuda")
        ctx.cocodc_fragment_scores(x, interval, ref_n, ref_s)
        assert ctx.cocodc_poll_status() == 0
        got_n = torch.full((K,), -1.0, device="cuda")
        got_s = torch.full((K,), -1.0, device="cuda")
        # The device's free memory as the driver reports it (torch's own counters see only torch's allocator, not a
        # cudaMalloc inside the library).  The first call on a device may load the module that holds the scratch
        # array when it looks up its address, so the comparison is made around a later call.
        if call == 1:
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
        before = torch.cuda.memory_allocated()
        B.cocodc_fragment_scores_noalloc(w.N, ptr, off, ln, x, interval, got_n, got_s)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        if call == 1:
            assert torch.cuda.mem_get_info()[0] == free_before, "device memory was allocated during the call"
        rn, rs, gn, gs = np_(ref_n), np_(ref_s), np_(got_n), np_(got_s)
        en, es = orc.fragment_scores(frs, np_(x), np_(interval))          # Eq. 10 by the CPU oracle
        assert np.all(np.abs(gn - en) <= TOL_NORM * np.abs(en)), (call, gn, en)
        assert np.all(np.abs(gs - es) <= TOL_NORM * np.abs(es)), (call, gs, es)
        assert np.all(np.abs(gn - rn) <= TOL_NORM * np.abs(rn)), (call, gn, rn)
        assert np.all(np.abs(gs - rs) <= TOL_NORM * np.abs(rs)), (call, gs, rs)
        if call == 1:
            assert gn[2] == 0.0 and gs[2] == 0.0
        # without intervals the score is the norm
        B.cocodc_fragment_scores_noalloc(w.N, ptr, off, ln, x, None, got_n, got_s)
        torch.cuda.synchronize()
        assert np.array_equal(np_(got_n), np_(got_s))


def test_noalloc_rejects_what_its_fixed_scratch_cannot_hold():
    from paper_2504_17672_b200 import binding as B
    x = torch.zeros(1 << 16, device="cuda")
    out = torch.zeros(128, device="cuda")
    K = B.NOALLOC_MAX_K + 1
    ptr = np.arange(K + 1, dtype=np.int32)
    off = np.arange(K, dtype=np.int64) * 16
    ln = np.full(K, 16, dtype=np.int64)
    with pytest.raises(B.CocodcError) as e:
        B.cocodc_fragment_scores_noalloc(1 << 16, ptr, off, ln, x, None, out, out)
    assert e.value.code == B.ERR_INVALID_ARG
    # one fragment with too many segments
    S = B.NOALLOC_MAX_SEGMENTS + 1
    with pytest.raises(B.CocodcError) as e:
        B.cocodc_fragment_scores_noalloc(1 << 16, [0, S], np.arange(S) * 16, np.full(S, 8), x, None, out, out)
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.CocodcError) as e:       # overlapping segments
        B.cocodc_fragment_scores_noalloc(1 << 16, [0, 1, 2], [0, 8], [16, 16], x, None, out, out)
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.CocodcError) as e:       # misaligned vector
        B.cocodc_fragment_scores_noalloc(1 << 15, [0, 1], [0], [100], x[1:], None, out, out)
    assert e.value.code == B.ERR_ALIGNMENT
    # at the limits it works
    K = B.NOALLOC_MAX_K
    x.fill_(0.5)
    B.cocodc_fragment_scores_noalloc(1 << 16, np.arange(K + 1), np.arange(K) * 1024, np.full(K, 1000), x, None,
                                     out[:K], out[K:2 * K].clone())
    torch.cuda.synchronize()
    assert np.allclose(np_(out[:K]), 0.5 * np.sqrt(1000.0), rtol=1e-6)
