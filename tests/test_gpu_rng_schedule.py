"""GPU parity, integer / fp64 side: the random draws and the arrival process of every variant
must be bit-identical to the oracle's."""
import numpy as np
import pytest

from oracle import core

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2003_10579_b200 import binding
    return binding


@pytest.mark.parametrize("kind,mu,shift", [("exp", 1.0, 0.0), ("shifted_exp", 2.0, 1.0), ("exp", 0.37, 0.0), ("pareto2", 2.0, 1.0), ("pareto2", 2.0, 0.3)])
def test_delay_draws_bit_exact(B, kind, mu, shift):
    R, P, S, base, seed = 5, 7, 300, 3, 12345678901234
    got = B.draw_delays(kind, mu, shift, seed, base, R, P, S)
    want = np.array([[[core.delay(kind, mu, shift, seed, base + r, i, s) for s in range(S)] for i in range(P)]
                     for r in range(R)])
    assert np.array_equal(got.view(np.int64), want.view(np.int64))


def test_index_draws_bit_exact(B):
    R, P, S, base, seed, n, m = 3, 4, 20, 1, 99, 65536, 37
    got = B.draw_indices(seed, base, R, P, S, n, m)
    for r in range(R):
        for i in range(P):
            for s in range(S):
                assert np.array_equal(got[r, i, s], core.minibatch_indices(seed, base + r, i, s, n, m))
    got = B.draw_indices(7, 0, 2, 2, 3, 1000003, 16)        # n not a power of two
    assert np.array_equal(got[1, 1, 2], core.minibatch_indices(7, 1, 1, 2, 1000003, 16))
    got = B.draw_indices(7, 0, 1, 1, 1, 2**32, 8)           # the largest n
    assert np.array_equal(got[0, 0, 0], core.minibatch_indices(7, 0, 0, 0, 2**32, 8))


def run_gpu_schedule(B, variant, P, K, kind, mu, shift, seed, R, J, base=0, K0=0, ti=0.0, chunks=None):
    sim = B.Simulation(None, P=P, K=K, variant=variant, delay_kind=kind, mu=mu, shift=shift, eta=0.0, m=1,
                       seed=seed, n_replicas=R, replica_base=base)
    if ti > 0:
        sim.set_adasync(K0, ti)
    for c in (chunks or [J]):
        sim.run(c)
    tr = sim.trace()
    sim.close()
    return tr


def check(B, variant, P, K, kind="exp", mu=1.0, shift=0.0, seed=0, R=33, J=150, base=0, K0=0, ti=0.0, chunks=None):
    from parity import assert_schedule_equal
    gpu = run_gpu_schedule(B, variant, P, K, kind, mu, shift, seed, R, J, base, K0, ti, chunks)
    ora = core.BulkSchedule(variant, P, K, kind, mu, shift, seed, R, replica_base=base, K0=K0, t_interval=ti).run(J)
    assert_schedule_equal(gpu, ora)
    assert np.all(gpu["loss"] == 0) and np.all(gpu["dist2"] == 0)


@pytest.mark.parametrize("variant", list(core.VARIANTS))
@pytest.mark.parametrize("P,K", [(1, 1), (4, 2), (7, 7), (16, 5), (32, 1), (32, 32), (31, 8)])
def test_schedule_bit_exact(B, variant, P, K):
    check(B, variant, P, K, "shifted_exp", 1.3, 0.25, seed=5, base=11)


@pytest.mark.parametrize("variant", list(core.VARIANTS))
@pytest.mark.parametrize("P,K", [(33, 1), (33, 33), (48, 7), (64, 64), (64, 20), (65, 9), (100, 31), (128, 128), (128, 5)])
def test_schedule_bit_exact_more_than_a_lane_per_worker(B, variant, P, K):
    """P > 32: two or four workers per lane in the arrival kernel, up to 130 version-pool slots."""
    check(B, variant, P, K, "shifted_exp", 0.9, 0.1, seed=15, R=7, J=60 if K > 40 else 120, base=3)


@pytest.mark.parametrize("variant", list(core.VARIANTS))
def test_schedule_wide_growing_K_ties_and_resume(B, variant):
    check(B, variant, 80, 1, "exp", 1.0, 0.0, seed=16, R=5, J=150, K0=2, ti=1.5, chunks=[1, 49, 100])
    check(B, variant, 40, 35, "shifted_exp", float("inf"), 0.5, R=2, J=6)          # all delays equal: ties by worker id
    check(B, variant, 96, 12, "pareto2", 2.0, 1.0, seed=17, R=4, J=80)


@pytest.mark.parametrize("variant", list(core.VARIANTS))
def test_schedule_growing_K_and_resume(B, variant):
    check(B, variant, 8, 1, "shifted_exp", 2.0, 1.0, seed=6, R=20, J=260, K0=1, ti=30.0, chunks=[1, 59, 200])
    check(B, variant, 12, 1, "exp", 1.0, 0.0, seed=7, R=9, J=120, K0=3, ti=4.0)


@pytest.mark.parametrize("variant", list(core.VARIANTS))
def test_schedule_ties(B, variant):
    check(B, variant, 5, 3, "shifted_exp", float("inf"), 0.5, R=2, J=12)


@pytest.mark.parametrize("variant", list(core.VARIANTS))
def test_schedule_under_pareto_delays(B, variant):
    check(B, variant, 16, 5, "pareto2", 2.0, 1.0, seed=8, R=17, J=200, base=4)


def test_first_workload_schedule_all_replicas(B):
    """K-sync, P=4, K=2, Exp(1), 64 replicas x 200 iterations, seed 0."""
    check(B, "ksync", 4, 2, R=64, J=200)


def test_bad_arguments_are_refused(B):
    S = B.Simulation
    base = dict(P=4, K=2, variant="ksync", delay_kind="exp", mu=1.0, eta=0.1, m=4, seed=0, n_replicas=2)
    for bad in (dict(P=0), dict(P=129), dict(K=0), dict(K=5), dict(m=0), dict(n_replicas=0), dict(mu=0.0),
                dict(mu=float("nan")), dict(delay_kind="shifted_exp", shift=-1.0), dict(replica_base=2**32),
                dict(delay_kind="pareto2", mu=3.0, shift=1.0), dict(delay_kind="pareto2", mu=2.0, shift=0.0)):
        with pytest.raises(B.SimError) as e:
            S(None, **{**base, **bad})
        assert e.value.status == 1
    sim = S(None, **base)
    with pytest.raises(B.SimError):
        sim.set_adasync(9, 1.0)
    sim.run(3)
    with pytest.raises(B.SimError) as e:
        sim.set_adasync(1, 1.0)
    assert e.value.status == 5
    sim.close()
