"""GPU parity at the full sizes of the five workloads, in the launch configuration the benchmark
uses: the arrival process is compared on every replica and every update; parameters and losses
on sampled replicas that the oracle can follow one by one (replicas {0, 1, R/2, R-1}) and on all
replicas for the first updates."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

from oracle import core
from paper_2003_10579_b200 import inputs
from parity import (assert_loss_close, assert_params_close, assert_schedule_equal, oracle_replica, rel_norm, to_device)

pytestmark = pytest.mark.gpu
THREADS = min(8, os.cpu_count() or 1)


@pytest.fixture(scope="module")
def B():
    from paper_2003_10579_b200 import binding
    return binding


def oracle_schedule_parallel(wl, variant, K, R, J, K0=0, ti=0.0):
    """The oracle's bulk arrival process, replica ranges spread over host threads."""
    bounds = np.linspace(0, R, THREADS + 1).astype(int)

    def part(i):
        a, b = bounds[i], bounds[i + 1]
        if a == b:
            return None
        return core.BulkSchedule(variant, wl.P, K, wl.delay_kind, wl.mu, wl.shift, wl.seed, b - a, replica_base=a,
                                 K0=K0, t_interval=ti).run(J)

    with ThreadPoolExecutor(THREADS) as ex:
        parts = [p for p in ex.map(part, range(THREADS)) if p is not None]
    return {k: np.concatenate([p[k] for p in parts], axis=0) for k in parts[0]}


def check_run(B, wl, data, dev, variant, K, *, J, replicas, w0=None, w_ref=None, first_all=0, K0=0, ti=0.0,
              param_rtol=1e-5, loss_rtol=1e-5):
    """One (variant, K) run of workload wl for J updates; returns the library's trace."""
    R = wl.replicas
    w_ref_dev = torch.from_numpy(w_ref).cuda() if w_ref is not None else None
    sim = B.Simulation(dev, P=wl.P, K=K, variant=variant, delay_kind=wl.delay_kind, mu=wl.mu, shift=wl.shift, eta=wl.eta,
                       m=wl.m, seed=wl.seed, n_replicas=R, w_ref=w_ref_dev)
    if ti > 0:
        sim.set_adasync(K0, ti)
    w0 = wl.w0() if w0 is None else w0
    if np.any(w0):
        sim.set_params(torch.from_numpy(w0).cuda())
    sim.reserve(J)
    kw = dict(P=wl.P, K=K, variant=variant, delay_kind=wl.delay_kind, mu=wl.mu, shift=wl.shift, eta=wl.eta, m=wl.m,
              seed=wl.seed, w_ref=w_ref, K0=K0, t_interval=ti)
    w_first = None
    if first_all:
        sim.run(first_all)
        w_first = sim.params()
    sim.run(J - first_all)
    tr, w_end = sim.trace(), sim.params()
    sim.close()
    assert_schedule_equal(tr, oracle_schedule_parallel(wl, variant, K, R, J, K0, ti))

    def follow(r):
        o = oracle_replica(data, w0, r, **kw).run(J)
        return r, o

    with ThreadPoolExecutor(THREADS) as ex:
        for r, o in ex.map(follow, replicas):
            ot = o.trace_arrays(K_stride=tr["worker"].shape[2])
            what = "%s %s K=%d replica %d" % (wl.name, variant, K, r)
            ew = assert_params_close(w_end[r], o.w, what + " final", rtol=param_rtol)
            dw = float(np.linalg.norm(w_end[r].astype(np.float64) - o.w))
            strict = np.abs(tr["loss"][r].astype(np.float64) - ot["loss"]) / np.maximum(np.abs(ot["loss"]), 1e-6 * abs(float(ot["loss"][0])))
            el = assert_loss_close(tr["loss"][r], ot["loss"], what, rtol=loss_rtol, gnorm=ot["gnorm"], dw=dw)
            print("%s: param err %.2e; loss err max %.2e, %.1f%% of updates within %.0e" % (
                what, ew, el, 100.0 * (strict <= loss_rtol).mean(), loss_rtol))
            if w_ref is not None:
                # d|w - w_ref|^2 = 2 (w - w_ref) . dw
                dist = np.sqrt(np.maximum(ot["dist2"].astype(np.float64), 0.0))
                assert_loss_close(tr["dist2"][r], ot["dist2"], what + " dist2", rtol=loss_rtol, gnorm=dist, dw=dw)
    if first_all:
        def head(r):
            return r, oracle_replica(data, w0, r, **kw).run(first_all)
        with ThreadPoolExecutor(THREADS) as ex:
            for r, o in ex.map(head, range(R)):
                assert_params_close(w_first[r], o.w, "%s K=%d replica %d after %d" % (variant, K, r, first_all), rtol=param_rtol)
    return tr


def sampled(R):
    return sorted({0, 1, R // 2, R - 1})


def test_second_workload_sweep(B):
    """K-sync and K-batch-sync, K = 1..16, least squares 65536 x 1024, 1024 replicas x 1000 updates."""
    wl = inputs.WORKLOADS[2]
    data = wl.make_data()
    dev = to_device(data)
    numeric = {("ksync", 1), ("ksync", 16), ("kbatchsync", 7)}
    for variant, K in wl.runs:
        if (variant, K) in numeric:
            check_run(B, wl, data, dev, variant, K, J=wl.updates, replicas=sampled(wl.replicas), w_ref=data["w_star"],
                      first_all=10 if K == 7 else 0)
        else:   # arrival process only, every replica and update (clock-only handle: same streams)
            sim = B.Simulation(None, P=wl.P, K=K, variant=variant, delay_kind=wl.delay_kind, mu=wl.mu, shift=wl.shift,
                               eta=0.0, m=1, seed=wl.seed, n_replicas=wl.replicas)
            sim.run(wl.updates)
            tr = sim.trace()
            sim.close()
            assert_schedule_equal(tr, oracle_schedule_parallel(wl, variant, K, wl.replicas, wl.updates))


def test_third_workload_async_logistic(B):
    """K-async and K-batch-async, K in {1,4,8}, logistic regression 262144 x 4096, 256 replicas x 2000 updates."""
    wl = inputs.WORKLOADS[3]
    data = wl.make_data()
    dev = to_device(data)
    for variant, K in wl.runs:
        check_run(B, wl, data, dev, variant, K, J=wl.updates, replicas=sampled(wl.replicas) if K == 4 else [0],
                  first_all=10 if (variant, K) == ("kasync", 4) else 0)


def test_fourth_workload_adasync_softmax(B):
    """K-sync with K doubling 1 -> 8 every 800 time units, softmax 65536 x 3072 x 10, 128 replicas x 3000 updates."""
    wl = inputs.WORKLOADS[4]
    data = wl.make_data()
    dev = to_device(data)
    tr = check_run(B, wl, data, dev, "ksync", 1, J=wl.updates, replicas=sampled(wl.replicas), first_all=10, K0=wl.K0,
                   ti=wl.t_interval)
    assert set(np.unique(tr["K"])) == {1, 2, 4, 8}


def test_fifth_workload_mlp(B):
    """K-batch-async MLP 3072-512-10 on 262144 samples, P=16, K=4, m=128, 64 replicas: the arrival process for
    all 2000 updates; losses and parameters of replica 0 for the first 150 updates (all 2000 with
    SSIM_FULL_MLP=1: the oracle needs several minutes for that), all replicas for 3 updates."""
    wl = inputs.WORKLOADS[5]
    J = wl.updates if os.environ.get("SSIM_FULL_MLP") == "1" else 150
    data = wl.make_data()
    dev = to_device(data)
    tr = check_run(B, wl, data, dev, "kbatchasync", 4, J=J, replicas=[0], first_all=3, param_rtol=1e-3, loss_rtol=1e-3)
    assert np.all(np.isfinite(tr["loss"]))
    sim = B.Simulation(None, P=wl.P, K=4, variant="kbatchasync", delay_kind=wl.delay_kind, mu=wl.mu, shift=wl.shift,
                       eta=0.0, m=1, seed=wl.seed, n_replicas=wl.replicas)
    sim.run(wl.updates)
    full = sim.trace()
    sim.close()
    assert_schedule_equal(full, oracle_schedule_parallel(wl, "kbatchasync", 4, wl.replicas, wl.updates))
