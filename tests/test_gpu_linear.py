"""GPU parity, fp32 side: least squares and logistic regression under every variant, against the
oracle: schedule bit-exact, parameters to 1e-5 (relative 2-norm) at every compared step, losses
to 1e-5 relative at every update."""
import numpy as np
import pytest
import torch

from paper_2003_10579_b200 import inputs
from parity import (assert_loss_close, assert_params_close, assert_schedule_equal, oracle_replica, to_device)
from oracle import core

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2003_10579_b200 import binding
    return binding


def run_case(B, data, *, variant, P, K, m, eta, R, J, kind="exp", mu=1.0, shift=0.0, seed=3, base=0, K0=0, ti=0.0,
             replicas=None, w0=None, chunks=None, step_checks=6, use_ref=True, stages=0):
    dev = to_device(data)
    npar = data["X"].shape[1] * (data["n_classes"] if data["model"] == "softmax" else 1)
    w_ref_np = data.get("w_star") if use_ref else None
    w_ref = torch.from_numpy(np.ascontiguousarray(w_ref_np)).cuda() if w_ref_np is not None else None
    sim = B.Simulation(dev, P=P, K=K, variant=variant, delay_kind=kind, mu=mu, shift=shift, eta=eta, m=m,
                       seed=seed, n_replicas=R, replica_base=base, w_ref=w_ref)
    if ti > 0:
        sim.set_adasync(K0, ti)
    if stages:
        sim.set_tuning(stages)
    if w0 is None:
        w0 = np.zeros(npar, np.float32)
    else:
        sim.set_params(torch.from_numpy(w0).cuda())
    kw = dict(P=P, K=K, variant=variant, delay_kind=kind, mu=mu, shift=shift, eta=eta, m=m, seed=seed,
              w_ref=w_ref_np, K0=K0, t_interval=ti)
    replicas = list(range(R)) if replicas is None else replicas
    oras = {r: oracle_replica(data, w0, base + r, **kw) for r in replicas}
    # parameters after each of the first few updates, then at the end of each chunk
    plan = [1] * min(step_checks, J) + (chunks or [])
    plan = plan + ([J - sum(plan)] if J > sum(plan) else [])
    worst_w = 0.0
    for c in plan:
        sim.run(c)
        w = sim.params()
        for r, o in oras.items():
            o.run(c)
            worst_w = max(worst_w, assert_params_close(w[r], o.w, "%s replica %d update %d" % (variant, r, o.j)))
    tr = sim.trace()
    sim.close()
    sched = core.BulkSchedule(variant, P, K, kind, mu, shift, seed, R, replica_base=base, K0=K0, t_interval=ti).run(J)
    assert_schedule_equal(tr, sched)
    worst_l = 0.0
    for r, o in oras.items():
        ot = o.trace_arrays(K_stride=tr["worker"].shape[2])
        assert np.array_equal(ot["worker"], tr["worker"][r]) and np.array_equal(ot["t"], tr["t"][r])
        worst_l = max(worst_l, assert_loss_close(tr["loss"][r], ot["loss"], "%s replica %d" % (variant, r)))
        if w_ref is not None:
            assert_loss_close(tr["dist2"][r], ot["dist2"], "%s replica %d dist2" % (variant, r))
    print("%s %s K=%d d=%d: worst param err %.2e, worst loss err %.2e" % (data["model"], variant, K, data["X"].shape[1], worst_w, worst_l))
    return tr


def test_first_workload_whole(B):
    """K-sync least squares, n=4096 x d=64, P=4, K=2, m=16, eta=0.01, Exp(1), 64 replicas x 200 iterations."""
    wl = inputs.WORKLOADS[1]
    data = wl.make_data()
    run_case(B, data, variant="ksync", P=wl.P, K=2, m=wl.m, eta=wl.eta, R=wl.replicas, J=wl.updates,
             seed=wl.seed, replicas=[0, 1, 32, 63], chunks=[50, 100])


@pytest.mark.parametrize("variant", list(core.VARIANTS))
@pytest.mark.parametrize("d,m,K,P", [(64, 16, 2, 4), (72, 5, 3, 5), (1024, 32, 5, 16), (1000, 9, 16, 16), (4096, 11, 2, 6), (2052, 4, 1, 3)])
def test_lsq_variants_and_shapes(B, variant, d, m, K, P):
    """Several column-ownership shapes (d not a multiple of the thread count), ragged tiles (m not a
    multiple of the tile height) and contributor counts."""
    data = inputs.make_lsq(3000, d, 0.1, 77)
    run_case(B, data, variant=variant, P=P, K=K, m=m, eta=0.02 if d < 2000 else 0.002, R=5, J=40, kind="shifted_exp",
             mu=1.0, shift=0.5, base=7, chunks=[10])


@pytest.mark.parametrize("variant", list(core.VARIANTS))
@pytest.mark.parametrize("model,d,m", [("lsq", 1024, 32), ("lsq", 1000, 9), ("logistic", 516, 6), ("lsq", 64, 16),
                                       ("logistic", 4096, 6), ("lsq", 2052, 5), ("lsq", 2048, 7), ("logistic", 300, 19), ("lsq", 256, 12)])
def test_many_replicas_take_the_narrow_blocks(B, variant, model, d, m):
    """With more than two replicas per SM the rows go to narrower blocks with more column chunks a thread (one warp for up
    to 1024 features, two for up to 2048; rows of up to 128 features lose the extra producer warp); with more than one
    per SM rows of 2049 to 4096 features go to four warps x eight chunks: same results, followed on four of 300 replicas."""
    data = inputs.make_lsq(3000, d, 0.1, 83) if model == "lsq" else inputs.make_logistic(3000, d, 0.05, 84)
    run_case(B, data, variant=variant, P=6, K=3, m=m, eta=0.02 if model == "lsq" else 0.01, R=300, J=30, kind="shifted_exp",
             mu=1.0, shift=0.5, base=2, replicas=[0, 1, 150, 299], chunks=[10], use_ref=model == "lsq")


@pytest.mark.parametrize("variant", list(core.VARIANTS))
@pytest.mark.parametrize("d,m,K,P", [(64, 8, 2, 4), (4096, 64, 4, 32), (520, 13, 8, 8)])
def test_logistic_variants_and_shapes(B, variant, d, m, K, P):
    data = inputs.make_logistic(4000, d, 0.05, 78)
    run_case(B, data, variant=variant, P=P, K=K, m=m, eta=0.01, R=4, J=40, chunks=[10], use_ref=False)


@pytest.mark.parametrize("variant", ["ksync", "kbatchasync"])
def test_resume_is_bit_exact(B, variant):
    data = inputs.make_lsq(2000, 256, 0.1, 79)
    dev = to_device(data)
    kw = dict(P=6, K=3, variant=variant, delay_kind="exp", mu=1.0, eta=0.02, m=10, seed=1, n_replicas=7)
    a = B.Simulation(dev, **kw)
    a.run(60)
    b = B.Simulation(dev, **kw)
    for c in (1, 17, 42):
        b.run(c)
    ta, tb = a.trace(), b.trace()
    for k in ta:
        assert np.array_equal(ta[k], tb[k]), k
    assert np.array_equal(a.params(), b.params())
    a.close(); b.close()


def test_results_do_not_depend_on_ring_depth_or_sharding(B):
    data = inputs.make_lsq(2000, 512, 0.1, 80)
    dev = to_device(data)
    kw = dict(P=4, K=2, variant="kasync", delay_kind="exp", mu=1.0, eta=0.02, m=12, seed=2)
    full = B.Simulation(dev, n_replicas=6, **kw)
    full.run(30)
    part = B.Simulation(dev, n_replicas=2, replica_base=3, **kw)
    part.set_tuning(5)
    part.run(30)
    tf, tp = full.trace(), part.trace()
    for k in tf:
        assert np.array_equal(tf[k][3:5], tp[k]), k
    assert np.array_equal(full.params()[3:5], part.params())
    full.close(); part.close()


def test_growing_K_least_squares(B):
    data = inputs.make_lsq(3000, 128, 0.1, 81)
    run_case(B, data, variant="ksync", P=8, K=1, m=8, eta=0.02, R=6, J=120, kind="shifted_exp", mu=2.0, shift=1.0,
             K0=1, ti=25.0, replicas=[0, 5], chunks=[50])
    run_case(B, data, variant="kbatchasync", P=8, K=1, m=8, eta=0.02, R=3, J=80, K0=2, ti=3.0, replicas=[1], chunks=[30])


def test_noiseless_least_squares_converges_on_the_gpu(B):
    data = inputs.make_lsq(4096, 64, 0.0, 1001)
    dev = to_device(data)
    w_ref = torch.from_numpy(data["w_star"]).cuda()
    sim = B.Simulation(dev, P=4, K=2, variant="ksync", delay_kind="exp", mu=1.0, eta=0.05, m=16, seed=0,
                       n_replicas=8, w_ref=w_ref)
    sim.run(2000)
    d2 = sim.trace()["dist2"]
    sim.close()
    assert np.all(d2[:, -1] / float((data["w_star"].astype(np.float64) ** 2).sum()) < 1e-9)


def test_host_buffer_call_matches_device_call(B):
    data = inputs.make_lsq(1000, 64, 0.1, 82)
    kw = dict(P=4, K=2, variant="kbatchsync", delay_kind="exp", mu=1.0, eta=0.02, m=8, seed=4, n_replicas=5)
    out = B.simulate_host(data, iters=25, w_ref=data["w_star"], want=("t", "loss", "dist2", "K", "worker", "stale", "seq", "w"), **kw)
    sim = B.Simulation(to_device(data), w_ref=torch.from_numpy(data["w_star"]).cuda(), **kw)
    sim.run(25)
    tr = sim.trace()
    for k in ("t", "loss", "dist2", "K", "worker", "stale", "seq"):
        assert np.array_equal(out[k], tr[k]), k
    assert np.array_equal(out["w"], sim.params())
    sim.close()


def test_sweep_on_host_buffers_matches_single_runs(B):
    data = inputs.make_lsq(1500, 128, 0.1, 83)
    runs = [("ksync", 1), ("ksync", 3), ("kbatchsync", 2), ("kbatchasync", 2)]
    kw = dict(P=4, delay_kind="shifted_exp", mu=1.0, shift=0.5, eta=0.02, m=8, seed=5, n_replicas=6)
    out = B.sweep_host(data, runs, iters=30, w_ref=data["w_star"], want=("t", "loss", "dist2"), **kw)
    dev = to_device(data)
    for i, (variant, K) in enumerate(runs):
        sim = B.Simulation(dev, variant=variant, K=K, w_ref=torch.from_numpy(data["w_star"]).cuda(), **kw)
        sim.run(30)
        tr = sim.trace()
        sim.close()
        for k in ("t", "loss", "dist2"):
            assert np.array_equal(out[k][i], tr[k]), (variant, K, k)
    # the same call writing into arrays of the caller (pinned memory here), and a wrong one refused before any work
    mine = {"loss": torch.empty((len(runs), 6, 30), dtype=torch.float32).pin_memory().numpy()}
    again = B.sweep_host(data, runs, iters=30, w_ref=data["w_star"], want=("t", "loss"), out=mine, **kw)
    assert again["loss"] is mine["loss"] and np.array_equal(mine["loss"], out["loss"]) and np.array_equal(again["t"], out["t"])
    with pytest.raises(ValueError):
        B.sweep_host(data, runs, iters=30, want=("loss",), out={"loss": np.empty((len(runs), 6, 29), np.float32)}, **kw)
