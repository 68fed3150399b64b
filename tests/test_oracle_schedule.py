"""Pins for the oracle's arrival processes against the runtime results of Section 3 and
Appendix B, plus identities between variants.  CPU only."""
import math

import numpy as np
import pytest

from oracle import core
from oracle.sim import OracleReplica


def H(n):
    return sum(1.0 / i for i in range(1, n + 1))


def bulk(variant, P, K, kind="exp", mu=1.0, shift=0.0, seed=0, R=64, J=400, **kw):
    b = core.BulkSchedule(variant, P, K, kind, mu, shift, seed, R, **kw)
    return b.run(J)


def iteration_times(tr):
    t = tr["t"]
    return np.diff(np.concatenate([np.zeros((t.shape[0], 1)), t], axis=1), axis=1)


def z_ok(sample, mean, var, z=4.5):
    n = sample.size
    return abs(sample.mean() - mean) <= z * math.sqrt(var / n)


# ---- Lemma 1 / Appendix B.1: K-sync, T = X_{K:P}; Exp: (H_P - H_{P-K})/mu, variance sum 1/(i mu)^2
@pytest.mark.parametrize("P,K,mu,shift", [(4, 2, 1.0, 0.0), (16, 5, 2.0, 0.0), (16, 16, 1.0, 0.0),
                                          (8, 3, 2.0, 1.0), (16, 1, 1.0, 0.5), (64, 40, 1.0, 0.0), (128, 9, 1.5, 0.25)])
def test_ksync_mean_and_variance(P, K, mu, shift):
    kind = "shifted_exp" if shift else "exp"
    T = iteration_times(bulk("ksync", P, K, kind, mu, shift, seed=3, R=64, J=400))
    mean = shift + (H(P) - H(P - K)) / mu
    var = sum(1.0 / (i * mu) ** 2 for i in range(P - K + 1, P + 1))
    assert z_ok(T, mean, var)
    assert abs(T.var() - var) < 0.08 * var + 1e-3
    assert T.min() >= shift


def test_ksync_first_workload_shape():
    """P=4, K=2, Exp(1), 64 replicas x 200 iterations: mean 7/12 = 0.58333."""
    T = iteration_times(bulk("ksync", 4, 2, seed=0, R=64, J=200))
    assert z_ok(T, 7.0 / 12.0, 1 / 16 + 1 / 9, z=4.0)


def test_ksync_each_worker_selected_with_frequency_K_over_P():
    tr = bulk("ksync", 8, 3, seed=5, R=64, J=500)
    cnt = np.bincount(tr["worker"].ravel(), minlength=8) / (64 * 500)
    assert np.all(np.abs(cnt - 3 / 8) < 0.02)
    assert np.all(tr["stale"] == 0)
    # all P workers launch once per iteration, so the contributing task of iteration j has seq j
    assert np.all(tr["seq"] == np.arange(500, dtype=np.uint32)[None, :, None])


# ---- Lemma 2 / Appendix B.2: K-batch-sync; Exp: T ~ Erlang(K, P mu)
@pytest.mark.parametrize("P,K,mu", [(4, 2, 1.0), (16, 7, 1.0), (16, 16, 3.0), (100, 33, 1.0)])
def test_kbatchsync_erlang(P, K, mu):
    T = iteration_times(bulk("kbatchsync", P, K, "exp", mu, seed=6, R=64, J=400))
    assert z_ok(T, K / (P * mu), K / (P * mu) ** 2)
    assert abs(T.var() - K / (P * mu) ** 2) < 0.08 * K / (P * mu) ** 2


def test_kbatchsync_shifted_bound():
    """New-longer-than-used: Delta <= E[T] <= K E[X_{1:P}] = K (Delta + 1/(P mu))."""
    P, K, mu, D = 16, 6, 1.0, 0.5
    T = iteration_times(bulk("kbatchsync", P, K, "shifted_exp", mu, D, seed=7, R=64, J=400))
    assert T.min() >= D
    assert T.mean() <= K * (D + 1 / (P * mu))
    # a worker needs at least Delta per minibatch: with K <= P the K-th finish is below Delta + X_{K:P}
    assert T.mean() <= D + (H(P) - H(P - K)) / mu


# ---- Lemma 3: K-async; Exp: equality with E[X_{K:P}]; new-longer-than-used: upper bound
@pytest.mark.parametrize("P,K", [(8, 1), (8, 3), (16, 8), (32, 4), (96, 20)])
def test_kasync_exp_mean(P, K):
    T = iteration_times(bulk("kasync", P, K, seed=8, R=64, J=600))
    mean = H(P) - H(P - K)
    var = sum(1.0 / i ** 2 for i in range(P - K + 1, P + 1))
    assert z_ok(T, mean, var)


def test_kasync_shifted_is_below_ksync_and_lemma4():
    P, K, mu, D = 16, 4, 1.0, 0.5
    Ta = iteration_times(bulk("kasync", P, K, "shifted_exp", mu, D, seed=9, R=64, J=800))
    assert Ta.mean() < D + (H(P) - H(P - K)) / mu
    # Lemma 4 (P = nK): n consecutive iterations take at most Delta + sum_i E[Exp_{K:(P-iK)}]
    n = P // K
    bound = D + sum((H(P - i * K) - H(P - (i + 1) * K)) / mu for i in range(n))
    blocks = Ta[:, : (Ta.shape[1] // n) * n].reshape(Ta.shape[0], -1, n).sum(axis=2)
    assert blocks.mean() < bound * 1.02


# ---- Lemma 5: K-batch-async, long-run K E[X]/P for any distribution
@pytest.mark.parametrize("kind,mu,D", [("exp", 1.0, 0.0), ("shifted_exp", 2.0, 1.0)])
def test_kbatchasync_renewal_rate(kind, mu, D):
    P, K, J = 16, 4, 3000
    tr = bulk("kbatchasync", P, K, kind, mu, D, seed=10, R=32, J=J)
    J0 = 500
    rate = (tr["t"][:, -1] - tr["t"][:, J0 - 1]) / (J - J0)
    want = K * (D + 1 / mu) / P
    assert abs(rate.mean() - want) < 0.01 * want


def test_theorem1_and_theorem2_ratios():
    """Exp: E[T_sync]/E[T_async] = P H_P;  E[T_Kasync]/E[T_Kbatchasync] = P (H_P - H_{P-K})/K."""
    P, K = 8, 3
    sync = iteration_times(bulk("ksync", P, P, seed=11, R=64, J=600)).mean()
    asyn = iteration_times(bulk("kasync", P, 1, seed=12, R=64, J=600)).mean()
    assert abs(sync / asyn / (P * H(P)) - 1) < 0.03
    ka = iteration_times(bulk("kasync", P, K, seed=13, R=64, J=600)).mean()
    kba = iteration_times(bulk("kbatchasync", P, K, seed=14, R=64, J=600)).mean()
    assert abs(ka / kba / (P * (H(P) - H(P - K)) / K) - 1) < 0.03


def test_lemma6_p0_is_one_over_P_for_exponential():
    """Fully asynchronous SGD (K=1): a push has staleness 0 with probability 1/P; since every
    worker sends 1/P of the pushes the mean staleness is P-1 (derived, not in the paper)."""
    P = 8
    tr = bulk("kasync", P, 1, seed=15, R=64, J=1500)
    st = tr["stale"][:, 100:, 0]
    assert abs((st == 0).mean() - 1 / P) < 0.006
    assert abs(st.mean() - (P - 1)) < 0.15


# ---- identities (bit-exact because a task's draws are keyed by its own sequence number)
def same(a, b, keys=("t", "K", "worker", "stale", "seq")):
    return all(np.array_equal(a[k], b[k]) for k in keys)


def test_identity_K1_async_equals_batch_async_and_K1_sync_equals_batch_sync():
    assert same(bulk("kasync", 8, 1, seed=20, R=8, J=300), bulk("kbatchasync", 8, 1, seed=20, R=8, J=300))
    for kind, D in (("exp", 0.0), ("shifted_exp", 0.5)):
        assert same(bulk("ksync", 8, 1, kind, 1.0, D, seed=21, R=8, J=300),
                    bulk("kbatchsync", 8, 1, kind, 1.0, D, seed=21, R=8, J=300))


def test_identity_K_equals_P_sync_equals_async():
    a = bulk("ksync", 8, 8, seed=22, R=8, J=300)
    b = bulk("kasync", 8, 8, seed=22, R=8, J=300)
    assert same(a, b)


def test_identity_single_worker_all_variants_are_serial_sgd():
    ref = bulk("ksync", 1, 1, "shifted_exp", 2.0, 0.25, seed=23, R=4, J=200)
    x = [core.delay("shifted_exp", 2.0, 0.25, 23, 2, 0, s) for s in range(200)]
    assert np.array_equal(np.diff(np.concatenate([[0.0], ref["t"][2]])) > 0, np.ones(200, bool))
    acc, tt = 0.0, []
    for v in x:
        acc += v
        tt.append(acc)
    assert ref["t"][2].tolist() == tt
    for v in ("kbatchsync", "kasync", "kbatchasync"):
        assert same(ref, bulk(v, 1, 1, "shifted_exp", 2.0, 0.25, seed=23, R=4, J=200))


def test_ties_go_to_the_lower_worker_id():
    """mu = inf makes every delay equal to the shift, so every comparison is a tie."""
    P, K, D = 5, 3, 0.5
    inf = float("inf")
    a = bulk("ksync", P, K, "shifted_exp", inf, D, R=1, J=3)
    assert a["worker"][0].tolist() == [[0, 1, 2]] * 3 and a["t"][0].tolist() == [0.5, 1.0, 1.5]
    b = bulk("kbatchsync", P, K, "shifted_exp", inf, D, R=1, J=2)
    assert b["worker"][0].tolist() == [[0, 1, 2]] * 2 and b["seq"][0].tolist() == [[0, 0, 0], [2, 2, 1]]
    assert b["t"][0].tolist() == [0.5, 1.0]     # workers 0 and 1 relaunched inside update 0, worker 2 did not
    c = bulk("kasync", P, K, "shifted_exp", inf, D, R=1, J=3)
    # update 0: workers 0,1,2 at t=.5, restart, end at 1.0; 3,4 ended at .5 and wait (stale 1);
    # update 1: 3,4 then 0, at t=1.0, restart, end at 1.5; update 2: 1,2 (ended 1.0) then 0 (1.5)
    assert c["worker"][0].tolist() == [[0, 1, 2], [3, 4, 0], [1, 2, 0]]
    assert c["t"][0].tolist() == [0.5, 1.0, 1.5]
    assert c["stale"][0].tolist() == [[0, 0, 0], [1, 1, 0], [1, 1, 0]]
    d = bulk("kbatchasync", P, 2, "shifted_exp", inf, D, R=1, J=3)
    assert d["worker"][0].tolist() == [[0, 1], [2, 3], [4, 0]]
    # worker 0 pushed first in update 0 and fetched w_0 again before that update happened
    assert d["stale"][0].tolist() == [[0, 0], [1, 1], [2, 2]]
    assert d["t"][0].tolist() == [0.5, 0.5, 1.0]


def test_brute_force_small_ksync():
    """P <= 4: sort the P delays of each iteration by hand."""
    P, K, seed, r = 4, 3, 31, 5
    tr = core.BulkSchedule("ksync", P, K, "exp", 1.5, 0.0, seed, 1, replica_base=r).run(50)
    t = 0.0
    for j in range(50):
        x = [core.delay("exp", 1.5, 0.0, seed, r, i, j) for i in range(P)]
        order = sorted(range(P), key=lambda i: (x[i], i))[:K]
        t += x[order[-1]]
        assert tr["worker"][0, j].tolist() == order and tr["t"][0, j] == t


# ---- the growing-K schedule (Algorithm 1's interval structure, doubling rule)
def test_adasync_doubling_switches_at_interval_boundaries():
    P, K0, ti = 8, 1, 25.0
    tr = bulk("ksync", P, 0, "shifted_exp", 2.0, 1.0, seed=40, R=16, J=200, K0=K0, t_interval=ti)
    K, t = tr["K"].astype(int), tr["t"]
    t_start = np.concatenate([np.zeros((16, 1)), t[:, :-1]], axis=1)
    want = np.minimum(P, K0 * 2 ** np.minimum(np.floor(t_start / ti), 10)).astype(int)
    assert np.array_equal(K, want)
    assert np.all(np.diff(K, axis=1) >= 0) and set(np.unique(K)) == {1, 2, 4, 8}
    used = (tr["worker"] != 0xFFFF).sum(axis=2)
    assert np.array_equal(used, K)
    # an infinite interval is the fixed-K run
    a = bulk("kasync", P, 2, seed=41, R=4, J=100)
    b = bulk("kasync", P, 0, seed=41, R=4, J=100, K0=2, t_interval=1e300)
    assert np.array_equal(a["t"], b["t"]) and np.array_equal(a["worker"], b["worker"][:, :, :2])


def test_resume_is_bit_exact():
    for v in core.VARIANTS:
        one = core.BulkSchedule(v, 6, 3, "shifted_exp", 1.0, 0.3, 50, 4, K0=1, t_interval=20.0)
        a = one.run(120)
        two = core.BulkSchedule(v, 6, 3, "shifted_exp", 1.0, 0.3, 50, 4, K0=1, t_interval=20.0)
        b1, b2 = two.run(47), two.run(73)
        for k in a:
            assert np.array_equal(a[k], np.concatenate([b1[k], b2[k]], axis=1))


def test_replica_base_shards_the_same_global_stream():
    full = bulk("kbatchasync", 4, 2, seed=60, R=8, J=50)
    part = core.BulkSchedule("kbatchasync", 4, 2, "exp", 1.0, 0.0, 60, 3, replica_base=5).run(50)
    assert all(np.array_equal(full[k][5:8], part[k]) for k in full)


# ---- the bulk C routine and the event-driven Python simulator are two separate writings
@pytest.mark.parametrize("variant", list(core.VARIANTS))
@pytest.mark.parametrize("P,K,K0,ti", [(4, 2, 0, 0.0), (7, 7, 0, 0.0), (8, 1, 0, 0.0), (8, 0, 1, 6.0), (5, 0, 2, 3.0)])
def test_bulk_schedule_equals_event_simulator(variant, P, K, K0, ti):
    kind, mu, D, seed, J = "shifted_exp", 1.3, 0.2, 70, 60
    tr = core.BulkSchedule(variant, P, K, kind, mu, D, seed, 3, replica_base=2, K0=K0, t_interval=ti).run(J)
    for r in range(3):
        sim = OracleReplica(model=None, X=None, y=None, w0=None, P=P, K=K, variant=variant,
                            delay_kind=kind, mu=mu, shift=D, eta=0.0, m=1, seed=seed, replica=2 + r,
                            K0=K0, t_interval=ti).run(J)
        ev = sim.trace_arrays(K_stride=tr["worker"].shape[2])
        for k in ("t", "K", "worker", "stale", "seq"):
            assert np.array_equal(tr[k][r], ev[k]), (variant, k)


def test_ksync_order_statistics_under_pareto():
    """Lemma 1 holds for any law: T = X_{K:P}.  Pareto(2,1): the minimum of P is Pareto(2P,1), the
    maximum has CDF (1 - x^-2)^P (the heavy-tailed case of the paper's runtime simulations)."""
    from scipy import stats
    P = 8
    Tmin = iteration_times(bulk("ksync", P, 1, "pareto2", 2.0, 1.0, seed=80, R=64, J=300)).ravel()
    assert stats.kstest(Tmin, "pareto", args=(2.0 * P,)).pvalue > 1e-4
    Tmax = iteration_times(bulk("ksync", P, P, "pareto2", 2.0, 1.0, seed=81, R=64, J=300)).ravel()
    assert stats.kstest(Tmax, lambda x: (1.0 - np.minimum(1.0, x ** -2.0)) ** P).pvalue > 1e-4
    # K-batch-async: long-run K E[X] / P with E[X] = 2 (Lemma 5; infinite variance, so a loose check)
    tr = bulk("kbatchasync", 16, 4, "pareto2", 2.0, 1.0, seed=82, R=64, J=4000)
    rate = (tr["t"][:, -1] - tr["t"][:, 499]) / 3500
    assert abs(np.median(rate) - 4 * 2.0 / 16) < 0.05


def test_error_curve_by_hand():
    """Two replicas: at each grid time take the error of the last completed update, average those that have one."""
    from oracle.curves import error_curve
    t = np.array([[1.0, 2.0, 4.0], [0.5, 3.0, 3.5]])
    e = np.array([[10.0, 8.0, 6.0], [20.0, 12.0, 4.0]])
    mean, cnt = error_curve(t, e, [0.25, 0.5, 1.0, 2.5, 3.0, 10.0])
    assert cnt.tolist() == [0, 1, 2, 2, 2, 2]
    assert mean.tolist() == [0.0, 20.0, 15.0, 14.0, 10.0, 5.0]


def test_envelope_by_hand():
    """Three curves on a grid of five points: the smallest value among the curves with data, lowest index on ties."""
    from oracle.curves import envelope
    curves = np.array([[9.0, 5.0, 4.0, 4.0, 1.0], [7.0, 6.0, 3.0, 4.0, 2.0], [1.0, 1.0, 8.0, 4.5, 0.5]])
    counts = np.array([[0, 2, 2, 2, 2], [0, 1, 1, 1, 1], [0, 0, 3, 3, 3]])
    env, best = envelope(curves, counts)
    assert env.tolist() == [0.0, 5.0, 3.0, 4.0, 0.5]
    assert best.tolist() == [-1, 0, 1, 0, 2]
