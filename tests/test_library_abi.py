"""The C-ABI library loads without a GPU and exports every function the header declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    import __graft_entry__
    __graft_entry__.build()
    header = open(os.path.join(ROOT, "include", "straggler_sim.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = sorted(set(re.findall(r"\b(sim_[a-z_0-9]+)\s*\(", header)))
    assert "sim_create" in declared and "sim_run" in declared and "sim_get_trace" in declared
    lib = ctypes.CDLL(os.path.join(ROOT, "paper_2003_10579_b200", "libstraggler_sim.so"))
    for name in declared:
        assert hasattr(lib, name), name
    from paper_2003_10579_b200 import binding
    assert sorted(binding.EXPORTS) == declared


def test_binding_refuses_to_work_without_the_library(tmp_path, monkeypatch):
    import importlib
    from paper_2003_10579_b200 import binding
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    try:
        binding._load()
    except ImportError as e:
        assert "no CPU fallback" in str(e)
    else:
        raise AssertionError("loading a missing library must fail")
    importlib.reload(binding)
