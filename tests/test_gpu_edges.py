"""GPU parity at the degenerate ends of the parameter ranges: one sample, one feature block, one
worker, minibatch of one, 32 workers with K = 32, replica ids at the top of the 32-bit range, a single
replica, and zero-length / repeated runs."""
import numpy as np
import pytest
import torch

from oracle import core
from paper_2003_10579_b200 import inputs
from parity import assert_schedule_equal, to_device
from test_gpu_linear import run_case

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2003_10579_b200 import binding
    return binding


@pytest.mark.parametrize("variant", list(core.VARIANTS))
def test_smallest_shapes(B, variant):
    run_case(B, inputs.make_lsq(1, 4, 0.0, 50), variant=variant, P=1, K=1, m=1, eta=0.05, R=1, J=12, chunks=[3])     # one sample
    run_case(B, inputs.make_lsq(7, 4, 0.1, 51), variant=variant, P=3, K=2, m=1, eta=0.05, R=2, J=15, chunks=[4])
    run_case(B, inputs.make_logistic(33, 8, 0.1, 52), variant=variant, P=2, K=2, m=3, eta=0.1, R=3, J=15, use_ref=False)
    run_case(B, inputs.make_mixture(40, 4, 2, 0.5, 53), variant=variant, P=2, K=1, m=5, eta=0.1, R=2, J=12, use_ref=False)


@pytest.mark.parametrize("variant", list(core.VARIANTS))
def test_all_32_workers_contribute(B, variant):
    run_case(B, inputs.make_lsq(500, 32, 0.1, 54), variant=variant, P=32, K=32, m=2, eta=0.05, R=3, J=10, chunks=[2])


def test_replica_ids_at_the_top_of_the_range(B):
    base = 2**32 - 5
    run_case(B, inputs.make_lsq(300, 16, 0.1, 55), variant="kbatchasync", P=4, K=2, m=4, eta=0.05, R=5, J=20, base=base)
    sim = B.Simulation(None, P=4, K=2, variant="kasync", delay_kind="exp", mu=1.0, eta=0.0, m=1, seed=7, n_replicas=5, replica_base=base)
    sim.run(40)
    ora = core.BulkSchedule("kasync", 4, 2, "exp", 1.0, 0.0, 7, 5, replica_base=base).run(40)
    assert_schedule_equal(sim.trace(), ora)
    sim.close()


def test_zero_length_and_many_short_runs(B):
    data = inputs.make_lsq(200, 16, 0.1, 56)
    dev = to_device(data)
    kw = dict(P=4, K=2, variant="kasync", delay_kind="exp", mu=1.0, eta=0.05, m=4, seed=3, n_replicas=4)
    a, b = B.Simulation(dev, **kw), B.Simulation(dev, **kw)
    assert a.trace_size()[0] == 0 and a.trace()["t"].shape == (4, 0)
    a.run(0)
    a.run(30)
    for _ in range(30):
        b.run(1)           # thirty growths of the trace from capacity 1
    ta, tb = a.trace(), b.trace()
    for k in ta:
        assert np.array_equal(ta[k], tb[k]), k
    assert np.array_equal(a.params(), b.params())
    a.close(); b.close()


def test_seed_uses_all_64_bits(B):
    kw = dict(P=4, K=2, variant="ksync", delay_kind="exp", mu=1.0, eta=0.0, m=1, n_replicas=2)
    out = []
    for seed in (1, 1 + 2**32, 2**63 + 1):
        sim = B.Simulation(None, seed=seed, **kw)
        sim.run(5)
        out.append(sim.trace()["t"])
        assert_schedule_equal(sim.trace(), core.BulkSchedule("ksync", 4, 2, "exp", 1.0, 0.0, seed, 2).run(5))
        sim.close()
    assert not np.array_equal(out[0], out[1]) and not np.array_equal(out[0], out[2])


@pytest.mark.parametrize("variant", list(core.VARIANTS))
def test_more_workers_than_warp_lanes(B, variant):
    """P = 40 and P = 128 workers (two / four per lane of the arrival kernel; 42 / 130 parameter versions):
    parameters and losses of every model family against the oracle."""
    run_case(B, inputs.make_lsq(600, 24, 0.1, 61), variant=variant, P=40, K=9, m=4, eta=0.02, R=3, J=40)
    run_case(B, inputs.make_logistic(500, 12, 0.05, 62), variant=variant, P=128, K=17, m=3, eta=0.05, R=2, J=30, use_ref=False)
    run_case(B, inputs.make_mixture(400, 20, 4, 0.5, 63, "softmax"), variant=variant, P=70, K=33, m=2, eta=0.05, R=2, J=20,
             use_ref=False)


def test_a_wait_that_runs_out_is_reported_and_poisons_only_its_handle(B):
    """The timeout path end to end, without hanging anything: the library's self-test kernel waits about a thousand
    polls on a barrier nobody arrives at and gives up; the handle's next synchronising call must return
    SIM_ERR_TIMEOUT, the handle must then refuse to run, and another handle on the same device must be unaffected."""
    data = to_device(inputs.make_lsq(300, 16, 0.1, 56))
    kw = dict(P=4, K=2, variant="ksync", delay_kind="exp", mu=1.0, eta=0.05, m=4, seed=1, n_replicas=3)
    bad, good = B.Simulation(data, **kw), B.Simulation(data, **kw)
    bad.run(5)
    good.run(5)
    bad.selftest_wait_timeout()
    with pytest.raises(B.SimError) as e:
        bad.trace_size()
    assert e.value.status == 4 and "wait ran out" in str(e.value)          # SIM_ERR_TIMEOUT
    with pytest.raises(B.SimError) as e:
        bad.run(1)
    assert e.value.status == 5                                             # SIM_ERR_STATE: the handle is poisoned
    with pytest.raises(B.SimError) as e:
        bad.params()
    assert e.value.status == 4
    bad.close()
    good.run(5)                                                            # the device and other handles carry on
    tr = good.trace()
    assert tr["t"].shape == (3, 10) and np.isfinite(tr["loss"]).all()
    good.close()


def test_switching_the_k_schedule_off_also_leaves_the_loss_driven_mode(B):
    """sim_set_adasync_loss followed by sim_set_adasync(0, 0): fixed K again, trace rows K wide, the fixed-K schedule."""
    data = to_device(inputs.make_lsq(300, 16, 0.1, 57))
    kw = dict(P=6, K=2, variant="kasync", delay_kind="exp", mu=1.0, eta=0.05, m=4, seed=2, n_replicas=4)
    a, b = B.Simulation(data, **kw), B.Simulation(data, **kw)
    a.set_adasync_loss(1, 3.0)
    a.set_adasync(0, 0.0)
    a.run(30)
    b.run(30)
    assert a.trace_size() == (30, 2)
    ta, tb = a.trace(), b.trace()
    for k in ta:
        assert np.array_equal(ta[k], tb[k]), k
    a.close(); b.close()
