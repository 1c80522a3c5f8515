"""The C-ABI library loads and exports every symbol the public header declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "distsim.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(distsim_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2306_08423_b200.build import build
    lib = ctypes.CDLL(build())
    names = _declared()
    assert {"distsim_load_event_table", "distsim_eval_strategies", "distsim_emit_timelines",
            "distsim_argmin"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_binding_names_match_header():
    from paper_2306_08423_b200.build import build
    build()
    from paper_2306_08423_b200 import engine
    assert sorted(engine.EXPORTS) == _declared()
    for name in engine.EXPORTS:
        if name not in ("distsim_create", "distsim_destroy", "distsim_last_error", "distsim_launch_count"):
            assert callable(getattr(engine, name)), name


def test_create_fails_loudly_without_a_gpu():
    import pytest
    import torch
    from paper_2306_08423_b200 import engine
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(engine.DistsimError) as ei:
        engine.Context(0)
    assert ei.value.code == engine.E_CUDA
