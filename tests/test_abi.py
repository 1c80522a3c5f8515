"""The C-ABI library loads and exports every symbol the public header declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared(header):
    text = open(os.path.join(ROOT, "include", header)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(distsim_[a-z_0-9]+)\s*\(", text)))


def test_every_header_is_covered():
    assert sorted(os.listdir(os.path.join(ROOT, "include"))) == ["distsim.h", "distsim_bench.h", "distsim_testing.h"]


def test_libraries_export_every_declared_symbol():
    from paper_2306_08423_b200 import build as B
    lib = ctypes.CDLL(B.build())
    names = _declared("distsim.h")
    assert {"distsim_load_event_table", "distsim_eval_strategies", "distsim_emit_timelines",
            "distsim_argmin"} <= set(names)
    for name in names + _declared("distsim_testing.h"):
        assert hasattr(lib, name), name
    bench = ctypes.CDLL(B.BENCH_LIB)
    for name in _declared("distsim_bench.h"):
        assert hasattr(bench, name), name
        assert not hasattr(lib, name), f"{name}: measurement code inside the engine's library"


def test_binding_names_match_headers():
    from paper_2306_08423_b200.build import build
    build()
    from paper_2306_08423_b200 import engine, probes
    assert sorted(engine.EXPORTS) == _declared("distsim.h")
    assert sorted(engine.TESTING_EXPORTS) == _declared("distsim_testing.h")
    assert sorted(probes.EXPORTS) == _declared("distsim_bench.h")
    for name in engine.EXPORTS + engine.TESTING_EXPORTS:
        if name not in ("distsim_create", "distsim_destroy", "distsim_last_error"):
            assert callable(getattr(engine, name)), name
    for name in probes.EXPORTS:
        assert callable(getattr(probes, name)), name


def test_create_fails_loudly_without_a_gpu():
    import pytest
    import torch
    from paper_2306_08423_b200 import engine
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(engine.DistsimError) as ei:
        engine.Context(0)
    assert ei.value.code == engine.E_CUDA


def test_long_pipeline_ranges_are_cut_into_launchable_pieces():
    # host arithmetic only: block counts in 64 bits, pieces cover the range exactly once
    from paper_2306_08423_b200 import engine
    for pp, cpb in ((64, 2), (32, 2), (16, 4), (1, 64)):
        for lo, hi in ((0, 1), (5, 5), (3, 1000), (0, 8_600_000_000), (7, 2**40 + 11)):
            max_blocks = 1 << 24
            n, pieces = engine.distsim_testing_lockstep_pieces(pp, lo, hi, max_blocks, 4096)
            assert n == -(-(hi - lo) // (max_blocks * cpb))
            pos = lo
            for a, b, blocks in pieces:
                assert a == pos and a < b <= hi and blocks == -(-(b - a) // cpb) and 1 <= blocks <= max_blocks
                pos = b
            if n <= 4096:
                assert pos == (hi if hi > lo else lo)
    with __import__("pytest").raises(engine.DistsimError):
        engine.distsim_testing_lockstep_pieces(3, 0, 10, 16)


def test_bidirectional_item_order_built_on_the_host():
    # the merged order the library builds for the bidirectional schedule (host code, no device)
    # against the token game restated in Python for the oracle's pins, and the schedule's slot count
    from paper_2306_08423_b200 import engine as E
    from tests.dag_bruteforce import bidirectional_order
    for pp in (2, 4, 6, 8, 16, 32):
        for m in (2, 4, 6, 8, 16, 34, 64, 128):
            got, kept = E.distsim_testing_bidirectional_order(pp, m)
            want, slots = bidirectional_order(pp, m)
            assert got == [want[d] for d in range(pp)], (pp, m)
            if m % pp == 0:
                assert slots == 2 * m + pp - 2
            # the kept tail: from the last backward item of the device's later stage on
            longest = 2
            for d in range(pp):
                u_first = 0 if d > pp - 1 - d else 1
                last = m // 2 - 1 + u_first * (m // 2)
                longest = max(longest, 2 * m - want[d].index(("B", last, u_first)))
            assert kept == longest <= pp // 2 + 2, (pp, m, kept, longest)
    import pytest
    for bad in ((3, 4), (4, 3), (34, 4), (0, 2)):
        with pytest.raises(E.DistsimError):
            E.distsim_testing_bidirectional_order(*bad)
