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


def test_argument_errors_are_found_on_the_host_before_any_device_call():
    """sim_create refuses bad sizes before it touches the device, so the refusals can be checked without a GPU:
    an m beyond the index stream's chunk field, an m whose index table cannot sit in shared memory beside the
    row tiles, and the no-allocation entry point's buffer checks in the binding."""
    import __graft_entry__
    __graft_entry__.build()
    from paper_2003_10579_b200 import binding as B
    import ctypes as C
    fake = 0x10000                      # never dereferenced: every case below fails validation first
    prob = B.SimProblem(B.MODELS["lsq"], 4096, 64, 1, 0, fake, fake, None, None)
    h = C.c_void_p()

    def create(m, P=4, K=2):
        return B.lib.sim_create(C.byref(prob), P, K, 0, B.SimDelay(0, 1.0, 0.0), 0.01, m, 0, 8, 0, None, C.byref(h))

    assert create((1 << 26) + 1) == 1 and b"2^26" in B.lib.sim_last_error(None)
    assert create(60000) == 1 and b"m is too large" in B.lib.sim_last_error(None)
    assert create(0) == 1 and create(16, P=4, K=5) == 1 and create(16, P=129, K=1) == 1
    assert not h.value


def test_noalloc_binding_checks_the_callers_buffers():
    import pytest
    import torch
    from paper_2003_10579_b200 import binding as B
    out = {k: torch.zeros(4) for k in ("t", "K", "worker", "stale", "seq")}    # CPU tensors of the wrong type
    with pytest.raises(ValueError):
        B.schedule_noalloc(out, P=4, K=2, variant="ksync", delay_kind="exp", mu=1.0, seed=0, n_replicas=2, iters=2)
