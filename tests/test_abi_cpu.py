"""Host-only checks of the C-ABI library: it loads, exports what the header declares, and validates arguments.

No kernel is launched here; these run without a GPU.
"""

import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2504_17672_b200 import build
    build.build()
    from paper_2504_17672_b200 import binding
    return binding


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(cocodc_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol(B):
    lib = B.library()
    names = declared_functions()
    assert {"cocodc_fragment_scores", "cocodc_select_fragments", "cocodc_outer_step", "cocodc_merge"} <= names
    for name in names:
        assert hasattr(lib, name), name
    assert names == set(B.EXPORTS)


def rows(name):
    out = []
    for line in open(os.path.join(ROOT, "tests", "golden", name)):
        line = line.strip()
        if line and not line.startswith("#"):
            out.append([float(x) for x in line.split()])
    return out


@pytest.mark.parametrize("row", rows("schedule_sizing.txt"))
def test_sync_budget_matches_paper_values(B, row):
    K, H, gamma, Tc, Ts, N, h = row
    assert B.cocodc_sync_budget(int(K), int(H), gamma, Tc, Ts) == (int(N), int(h))


def test_sync_budget_agrees_with_oracle_and_rejects_bad_input(B):
    from oracle import reference as orc
    rng = np.random.default_rng(0)
    for _ in range(200):
        K = int(rng.integers(1, 40)); H = int(rng.integers(1, 500))
        gamma = float(rng.uniform(0.01, 1.0)); Tc = float(rng.uniform(0.01, 3)); Ts = float(rng.uniform(0.01, 30))
        assert B.cocodc_sync_budget(K, H, gamma, Tc, Ts) == orc.sync_budget(K, H, gamma, Tc, Ts)
    for bad in ((0, 100, 0.4, 1, 1), (4, 0, 0.4, 1, 1), (4, 100, 0.0, 1, 1), (4, 100, 1.5, 1, 1),
                (4, 100, 0.4, 0.0, 1), (4, 100, 0.4, 1, -1.0), (4, 100, float("nan"), 1, 1)):
        with pytest.raises(B.CocodcError) as e:
            B.cocodc_sync_budget(*bad)
        assert e.value.code == B.ERR_INVALID_ARG


def test_status_strings(B):
    seen = {B.status_string(c) for c in range(8)}
    assert len(seen) == 8 and "ok" in seen
    assert "unknown" in B.status_string(99)


def test_create_rejects_bad_partitions_before_touching_the_device(B):
    def create(N, ptr, off, ln, max_M=4):
        return B.Context(N, ptr, off, ln, max_M, device=0)

    cases = [
        (100, [0, 1, 2], [0, 40], [50, 50]),      # overlapping segments
        (100, [0, 1, 2], [0, 60], [50, 50]),      # runs past N
        (100, [0, 1, 1], [0], [50]),              # empty fragment
        (100, [0, 1], [-4], [50]),                # negative offset
        (100, [0, 1], [0], [0]),                  # empty segment
        (100, [1, 2], [0, 50], [50, 50]),         # CSR does not start at 0
        (100, [0, 1000, 2], [0, 50], [50, 50]),   # a pointer beyond the segment arrays, although the last one equals S
    ]
    for N, ptr, off, ln in cases:
        with pytest.raises(B.CocodcError) as e:
            create(N, ptr, off, ln)
        assert e.value.code == B.ERR_INVALID_ARG, (ptr, off, ln)
    for bad_M in (0, 65):
        with pytest.raises(B.CocodcError) as e:
            create(100, [0, 1], [0], [100], max_M=bad_M)
        assert e.value.code == B.ERR_INVALID_ARG


def test_noalloc_entry_point_checks_its_table_before_touching_the_device(B):
    """The table is host data validated on every call; a pointer array that is not monotone must not make the
    host loop read past the segment arrays (the addresses below are never dereferenced: validation fails first)."""
    fake = ctypes.c_void_p(0x10000)

    def call(N, ptr, off, ln):
        ptr = np.ascontiguousarray(ptr, dtype=np.int32)
        off = np.ascontiguousarray(off, dtype=np.int64)
        ln = np.ascontiguousarray(ln, dtype=np.int64)
        part = B._Partition(N, len(ptr) - 1, len(off), ptr.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                            off.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)),
                            ln.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)))
        return B.library().cocodc_fragment_scores_noalloc(ctypes.byref(part), fake, None, fake, fake, 0, None)

    assert call(100, [0, 1000, 2], [0, 50], [50, 50]) == B.ERR_INVALID_ARG
    assert call(100, [0, 2, 2], [0, 50], [50, 50]) == B.ERR_INVALID_ARG        # empty second fragment
    assert call(100, [0, 1, 2], [0, 40], [50, 50]) == B.ERR_INVALID_ARG        # overlap
    assert call(100, [0, 1, 2], [0, 60], [50, 50]) == B.ERR_INVALID_ARG        # past N


def test_null_context_is_rejected(B):
    lib = B.library()
    assert lib.cocodc_poll_status(None, None) == B.ERR_INVALID_ARG
    assert lib.cocodc_fragment_scores(None, None, None, None, None, None, None) == B.ERR_INVALID_ARG
    assert lib.cocodc_scores_from_sumsq(None, None, None, None, None, 0, 0, None, None, None, None) == B.ERR_INVALID_ARG
    assert lib.cocodc_bind_in_flight(None, None) == B.ERR_INVALID_ARG
    assert lib.cocodc_flush_scores(None, None) == B.ERR_INVALID_ARG
    assert lib.cocodc_destroy(None) == B.OK
    assert lib.cocodc_launch_count(None) == 0


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    """The binding has no fallback: without the built library the import raises."""
    import importlib
    from paper_2504_17672_b200 import build
    monkeypatch.setattr(build, "LIBRARY", str(tmp_path / "libcocodc.so"))
    import paper_2504_17672_b200.binding as binding
    with pytest.raises(ImportError):
        binding._load()


def test_plain_c_client_compiles_links_and_runs(B, tmp_path):
    """The header is C99 and the library needs nothing but itself: gcc builds tests/abi_client.c against both."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no gcc")
    from paper_2504_17672_b200 import build
    lib_dir = os.path.dirname(build.LIBRARY)
    exe = str(tmp_path / "abi_client")
    subprocess.run([gcc, "-std=c99", "-pedantic", "-Wall", "-Wextra", "-Werror", "-I", os.path.join(ROOT, "include"),
                    os.path.join(ROOT, "tests", "abi_client.c"), "-o", exe, "-L", lib_dir, "-lcocodc",
                    "-Wl,-rpath," + lib_dir], check=True)
    out = subprocess.run([exe], check=True, capture_output=True, text=True).stdout
    assert out.strip() == "abi client ok: N=8 h=12"
