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


def test_full_data_loss_is_refused_for_the_mlp():
    from paper_2003_10579_b200 import binding as B
    data = inputs.make_mixture(256, 128, 4, 0.5, 34, "mlp2", 64)
    sim = B.Simulation(to_device(data), P=2, K=1, variant="ksync", delay_kind="exp", mu=1.0, eta=0.1, m=128, seed=0, n_replicas=1)
    with pytest.raises(B.SimError) as e:
        sim.eval_loss()
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
