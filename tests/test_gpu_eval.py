"""GPU parity of the full-data risk F(w) (Eq. 1) against the oracle, for the three linear models,
synchronous (parameters in place) and asynchronous (version pool) handles, ragged n and d."""
import numpy as np
import pytest
import torch

from oracle import models
from paper_2003_10579_b200 import inputs
from parity import to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("model,n,d,C,variant", [("lsq", 1000, 64, 1, "ksync"), ("lsq", 4099, 1000, 1, "kbatchasync"),
                                                 ("logistic", 2500, 520, 1, "kasync"), ("softmax", 1500, 200, 10, "ksync"),
                                                 ("softmax", 777, 64, 3, "kbatchasync"), ("softmax", 900, 128, 16, "kasync")])
def test_full_data_loss_matches_the_oracle(model, n, d, C, variant):
    from paper_2003_10579_b200 import binding as B
    if model == "lsq":
        data = inputs.make_lsq(n, d, 0.1, 31)
    elif model == "logistic":
        data = inputs.make_logistic(n, d, 0.05, 32)
    else:
        data = inputs.make_mixture(n, d, C, 0.5, 33)
    R = 70
    sim = B.Simulation(to_device(data), P=4, K=2, variant=variant, delay_kind="exp", mu=1.0, eta=0.02, m=8, seed=1, n_replicas=R)
    for steps in (0, 25):
        if steps:
            sim.run(steps)
        got = sim.eval_loss()
        w = sim.params()
        for r in (0, 1, 37, R - 1):
            want = models.full_loss(model, w[r], data["X"], data["y"], data["n_classes"])
            assert abs(got[r] - want) <= 1e-5 * abs(want), (model, steps, r, got[r], want)
    sim.close()


@pytest.mark.parametrize("variant,n,d,H,C", [("ksync", 1000, 128, 64, 3), ("kbatchasync", 3333, 256, 192, 10), ("kasync", 640, 3072, 512, 10)])
def test_full_data_loss_of_the_mlp_matches_the_oracle(variant, n, d, H, C):
    """The forward-only form of the tensor-core kernel over all rows (ragged last block of 128) against the oracle's
    full_loss with the same bf16 operand rounding: before any update, after an odd and after an even number."""
    from paper_2003_10579_b200 import binding as B
    data = inputs.make_mixture(n, d, C, 0.5 if d < 1000 else 0.1, 36, "mlp2", H)
    w0 = inputs.mlp_init(d, H, C, 37)
    R = 5
    sim = B.Simulation(to_device(data), P=4, K=2, variant=variant, delay_kind="exp", mu=1.0, eta=0.05, m=128, seed=1, n_replicas=R)
    sim.set_params(torch.from_numpy(w0).cuda())
    for steps in (0, 3, 4):
        if steps:
            sim.run(steps)
        got = sim.eval_loss()
        w = sim.params()
        for r in (0, 2, R - 1):
            want = models.full_loss("mlp2", w[r], data["X"], data["y"], C, H)
            assert abs(got[r] - want) <= 1e-3 * abs(want), (variant, steps, r, got[r], want)
    sim.close()


def test_full_data_loss_is_refused_without_a_model():
    from paper_2003_10579_b200 import binding as B
    sim = B.Simulation(None, P=2, K=1, variant="ksync", delay_kind="exp", mu=1.0, eta=0.1, m=1, seed=0, n_replicas=1)
    with pytest.raises(B.SimError) as e:
        sim.eval_loss()
    assert e.value.status == 1
    with pytest.raises(B.SimError) as e:
        sim.set_eval_every(5)
    assert e.value.status == 1
    sim.close()


def test_error_curve_matches_the_oracle():
    from oracle.curves import error_curve
    from paper_2003_10579_b200 import binding as B
    data = inputs.make_lsq(1000, 64, 0.1, 35)
    sim = B.Simulation(to_device(data), P=8, K=3, variant="kasync", delay_kind="exp", mu=1.0, eta=0.02, m=8, seed=2, n_replicas=300)
    with pytest.raises(B.SimError):
        sim.error_curve([1.0])
    sim.reserve(500)          # capacity larger than the updates done: the row pitch differs from J
    sim.run(120)
    tr = sim.trace()
    grid = np.concatenate([[0.0, 1e-6], np.linspace(0.05, tr["t"].max() * 1.1, 40)])
    mean, cnt = sim.error_curve(grid)
    want_mean, want_cnt = error_curve(tr["t"], tr["loss"], grid)
    assert np.array_equal(cnt, want_cnt)
    assert np.allclose(mean, want_mean, rtol=1e-6, atol=0)
    assert cnt[0] == 0 and cnt[-1] == 300 and mean[-1] < mean[5]
    sim.close()


def lsq_floor(data):
    """F* of least squares from the normal equations (fp64, on the host): the harness's part of F(w) - F*."""
    X, y = data["X"].astype(np.float64), data["y"].astype(np.float64)
    w = np.linalg.solve(X.T @ X, X.T @ y)
    r = X @ w - y
    return 0.5 * float(r @ r) / X.shape[0]


@pytest.mark.parametrize("variant,chunks", [("ksync", (37, 63)), ("kbatchasync", (5, 5, 90)), ("kasync", (100,))])
def test_risk_trace_inside_run_matches_the_oracle(variant, chunks):
    """sim_set_eval_every: F(w_j) before the first and after every 10th update, however sim_run is cut into calls,
    against the oracle's full_loss of the parameters the oracle holds at those updates; its clock is the trace's."""
    from paper_2003_10579_b200 import binding as B
    from parity import oracle_replica
    data = inputs.make_lsq(1500, 64, 0.1, 38)
    kw = dict(P=6, K=2, variant=variant, delay_kind="shifted_exp", mu=1.0, shift=0.3, eta=0.02, m=8, seed=4)
    R, every = 9, 10
    sim = B.Simulation(to_device(data), n_replicas=R, **kw)
    sim.set_eval_every(every)
    for c in chunks:
        sim.run(c)
    risk, t = sim.risk_trace()
    tr = sim.trace()
    E = 1 + sum(chunks) // every
    assert risk.shape == (R, E) and t.shape == (R, E)
    assert not t[:, 0].any() and np.array_equal(t[:, 1:], tr["t"][:, every - 1::every][:, :E - 1])
    for r in (0, 4, R - 1):
        o = oracle_replica(data, np.zeros(64, np.float32), r, **kw)
        for i in range(E):
            want = models.full_loss("lsq", o.w, data["X"], data["y"])
            assert abs(risk[r, i] - want) <= 1e-5 * abs(want), (variant, r, i, risk[r, i], want)
            o.run(every)
    # the resumed run is the same run: one call of the whole length gives the same bits
    whole = B.Simulation(to_device(data), n_replicas=R, **kw)
    whole.set_eval_every(every)
    whole.run(sum(chunks))
    assert np.array_equal(whole.risk_trace()[0], risk)
    whole.close(); sim.close()


def test_risk_curve_and_envelope_over_K_match_the_oracle():
    """The picture of Sections 1 and 5 on a noisy least-squares problem: F(w) - F* against wall clock for K = 1, 4
    and 16 of 16 workers (F* from the normal equations), each curve and the lower envelope over K against the oracle's
    curve routines fed with the library's own risk trace; and the trade-off itself - a small K is ahead early,
    a large K ends lower."""
    from oracle.curves import envelope, error_curve
    from paper_2003_10579_b200 import binding as B
    data = inputs.make_lsq(4000, 32, 0.5, 39)
    f_star = lsq_floor(data)
    dev = to_device(data)
    # updates per simulation chosen so that all three cover about the same span of simulated time (an update takes
    # 0.26, 0.48 and 3.6 time units on average for K = 1, 4, 16)
    Ks, plan, sims = (1, 4, 16), {1: (1700, 20), 4: (920, 10), 16: (120, 2)}, []
    for K in Ks:
        s = B.Simulation(dev, P=16, K=K, variant="ksync", delay_kind="shifted_exp", mu=1.0, shift=0.2, eta=0.05, m=4, seed=6,
                         n_replicas=200)
        s.set_eval_every(plan[K][1])
        s.run(plan[K][0])
        sims.append(s)
    t_end = min(s.risk_trace()[1][:, -1].min() for s in sims)
    grid = np.linspace(0.0, t_end, 60)
    curves, counts = [], []
    for s in sims:
        risk, t = s.risk_trace()
        mean, cnt = s.risk_curve(grid, f_star)
        want_mean, want_cnt = error_curve(t, risk.astype(np.float64) - np.float64(np.float32(f_star)), grid)
        assert np.array_equal(cnt, want_cnt) and cnt.min() == 200
        assert np.allclose(mean, want_mean, rtol=1e-5, atol=1e-7)
        curves.append(mean); counts.append(cnt)
    env, best = B.risk_envelope(sims, grid, f_star)
    want_env, want_best = envelope(np.array(curves), np.array(counts))
    assert np.array_equal(best, want_best) and np.array_equal(env, want_env.astype(np.float32))
    # early on the small K leads (more updates per unit time), at the end the large K sits at a lower error floor
    assert Ks[best[3]] == 1 and Ks[best[-1]] == 16 and 1 in best.tolist()
    assert curves[2][-1] < curves[1][-1] < curves[0][-1]
    for s in sims:
        s.close()


def test_risk_trace_of_the_mlp_and_refusals():
    from paper_2003_10579_b200 import binding as B
    data = inputs.make_mixture(700, 128, 3, 0.5, 40, "mlp2", 64)
    w0 = inputs.mlp_init(128, 64, 3, 41)
    sim = B.Simulation(to_device(data), P=4, K=2, variant="kbatchasync", delay_kind="exp", mu=1.0, eta=0.05, m=128, seed=1, n_replicas=3)
    sim.set_params(torch.from_numpy(w0).cuda())
    sim.set_eval_every(4)
    sim.run(9)
    risk, t = sim.risk_trace()
    assert risk.shape == (3, 3)
    want0 = models.full_loss("mlp2", w0, data["X"], data["y"], 3, 64)
    assert abs(risk[1, 0] - want0) <= 1e-3 * want0
    assert (risk[:, 2] < risk[:, 0]).all()                   # the risk falls while training
    with pytest.raises(B.SimError) as e:                      # only before the first update
        sim.set_eval_every(2)
    assert e.value.status == 5
    sim.close()
    lin = B.Simulation(to_device(inputs.make_lsq(300, 16, 0.1, 42)), P=4, K=1, variant="ksync", delay_kind="exp", mu=1.0, eta=0.05, m=4,
                       seed=1, n_replicas=2)
    lin.set_eval_every(3)
    with pytest.raises(B.SimError) as e:                      # the loss-driven K rule pauses replicas one by one
        lin.set_adasync_loss(1, 2.0)
    assert e.value.status == 5
    with pytest.raises(B.SimError) as e:
        lin.risk_curve([1.0])
    assert e.value.status == 5                                # nothing recorded yet
    lin.close()
