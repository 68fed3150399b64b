"""The entry point for callers that cannot allocate device memory (its worker state lives in a
fixed array inside the library) must give exactly the schedule of the regular entry points.

Collected last on purpose: a run that stops at the first failure has then already run every other
test.  Two calls in a row are checked because the fixed array keeps the first call's contents:
the second call must not see them."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

_U16, _U32 = torch.uint16, torch.uint32


def _regular(B, kw, R, J, K0=0, ti=0.0):
    sim = B.Simulation(None, eta=0.0, m=1, n_replicas=R, **kw)
    if ti > 0:
        sim.set_adasync(K0, ti)
    sim.run(J)
    tr = sim.trace()
    sim.close()
    return tr


def _noalloc(B, kw, R, J, K0=0, ti=0.0):
    Ks = kw["P"] if ti > 0 else kw["K"]
    # the caller owns every buffer; poison them so that unwritten entries would show
    out = {"t": torch.full((R, J), -1.0, dtype=torch.float64, device="cuda"),
           "K": torch.full((R, J), 777, dtype=torch.int32, device="cuda").to(_U16),
           "worker": torch.full((R, J, Ks), 555, dtype=torch.int32, device="cuda").to(_U16),
           "stale": torch.full((R, J, Ks), 12345, dtype=torch.int64, device="cuda").to(_U32),
           "seq": torch.full((R, J, Ks), 12345, dtype=torch.int64, device="cuda").to(_U32)}
    B.schedule_noalloc(out, n_replicas=R, iters=J, K0=K0, t_interval=ti, stream=torch.cuda.current_stream(), **kw)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def test_no_alloc_entry_point_matches_regular_path_twice_in_a_row():
    from paper_2003_10579_b200 import binding as B
    calls = [
        (dict(P=16, K=5, variant="kbatchasync", delay_kind="shifted_exp", mu=1.0, shift=0.5, seed=11, replica_base=3), 200, 300, 0, 0.0),
        (dict(P=8, K=3, variant="kasync", delay_kind="exp", mu=2.0, seed=12, replica_base=0), 64, 150, 0, 0.0),
        (dict(P=8, K=1, variant="ksync", delay_kind="shifted_exp", mu=2.0, shift=1.0, seed=13), 33, 120, 1, 20.0),
        (dict(P=6, K=4, variant="kbatchsync", delay_kind="exp", mu=1.0, seed=14), 5, 9000, 0, 0.0),   # > one launch
    ]
    for kw, R, J, K0, ti in calls:
        want = _regular(B, kw, R, J, K0, ti)
        got = _noalloc(B, kw, R, J, K0, ti)
        for k in ("t", "K", "worker", "stale", "seq"):
            a = got[k].view(np.int64) if k == "t" else got[k]
            b = want[k].view(np.int64) if k == "t" else want[k]
            assert np.array_equal(a, b), (kw["variant"], k)


def test_no_alloc_entry_point_refuses_what_the_fixed_array_cannot_hold():
    from paper_2003_10579_b200 import binding as B
    kw = dict(P=32, K=1, variant="ksync", delay_kind="exp", mu=1.0, seed=0)
    types = {"t": torch.float64, "K": _U16, "worker": _U16, "stale": _U32, "seq": _U32}
    out = {k: torch.zeros(4097, dtype=torch.int64, device="cuda").to(dt) for k, dt in types.items()}
    for R in (4097, 2049):          # too many replicas; too many replica x worker pairs
        with pytest.raises(B.SimError) as e:
            B.schedule_noalloc(out, n_replicas=R, iters=1, **kw)
        assert e.value.status == 1 and "SIM_NOALLOC_MAX" in str(e.value)


def test_no_alloc_binding_refuses_buffers_the_library_would_overrun():
    from paper_2003_10579_b200 import binding as B
    kw = dict(P=4, K=2, variant="ksync", delay_kind="exp", mu=1.0, seed=0)
    types = {"t": torch.float64, "K": _U16, "worker": _U16, "stale": _U32, "seq": _U32}
    out = {k: torch.zeros(16, dtype=torch.int64, device="cuda").to(dt) for k, dt in types.items()}
    with pytest.raises(ValueError):          # worker / stale / seq need 4 x 4 x 2 = 32 entries
        B.schedule_noalloc(out, n_replicas=4, iters=4, **kw)
