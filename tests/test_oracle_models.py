"""Pins for the oracle's gradients and for the update rule of Eq. 2 / Eq. 3.  CPU only."""
import math

import numpy as np
import pytest
import torch

from oracle import core, models
from oracle.sim import OracleReplica
from paper_2003_10579_b200 import inputs


def _case(model, m=6, d=8, C=3, H=5, seed=0):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((m, d)).astype(np.float32)
    if model == "lsq":
        return X, rng.standard_normal(m).astype(np.float32), rng.standard_normal(d).astype(np.float32), 1, 0
    if model == "logistic":
        return X, rng.integers(0, 2, m).astype(np.int32), rng.standard_normal(d).astype(np.float32), 1, 0
    npar = models.n_params(model, d, C, H)
    return X, rng.integers(0, C, m).astype(np.int32), (0.5 * rng.standard_normal(npar)).astype(np.float32), C, H


@pytest.mark.parametrize("model", ["lsq", "logistic", "softmax", "mlp2"])
def test_gradient_matches_finite_differences(model):
    X, y, w, C, H = _case(model)
    loss, g = models.loss_and_grad(model, w, X, y, C, H, bf16=False)
    w64 = w.astype(np.float64)
    h = 1e-6
    for p in range(w.size):
        e = np.zeros_like(w64)
        e[p] = h
        lp, _ = models.loss_and_grad(model, w64 + e, X, y, C, H, bf16=False)
        lm, _ = models.loss_and_grad(model, w64 - e, X, y, C, H, bf16=False)
        assert abs((lp - lm) / (2 * h) / X.shape[0] - g[p]) < 1e-7, (model, p)


def _torch_loss(model, w, X, y, C, H):
    Xt = torch.tensor(X, dtype=torch.float64)
    if model == "lsq":
        return 0.5 * ((Xt @ w - torch.tensor(y, dtype=torch.float64)) ** 2).sum()
    if model == "logistic":
        return torch.nn.functional.binary_cross_entropy_with_logits(
            Xt @ w, torch.tensor(y, dtype=torch.float64), reduction="sum")
    lab = torch.tensor(y, dtype=torch.int64)
    d = X.shape[1]
    if model == "softmax":
        return torch.nn.functional.cross_entropy(Xt @ w.view(C, d).T, lab, reduction="sum")
    o1, o2, o3 = d * H, d * H + H, d * H + H + H * C
    hid = torch.relu(Xt @ w[:o1].view(d, H) + w[o1:o2])
    return torch.nn.functional.cross_entropy(hid @ w[o2:o3].view(H, C) + w[o3:], lab, reduction="sum")


@pytest.mark.parametrize("model", ["lsq", "logistic", "softmax", "mlp2"])
def test_loss_and_gradient_match_torch_autograd(model):
    """The same losses written with torch's library routines, differentiated by autograd."""
    X, y, w, C, H = _case(model, m=9, d=12, C=4, H=7, seed=1)
    wt = torch.tensor(w, dtype=torch.float64, requires_grad=True)
    L = _torch_loss(model, wt, X, y, C, H)
    L.backward()
    loss, g = models.loss_and_grad(model, w, X, y, C, H, bf16=False)
    assert abs(loss - L.item()) < 1e-12 * max(1.0, abs(L.item()))
    assert np.allclose(g, wt.grad.numpy() / X.shape[0], rtol=1e-12, atol=1e-13)


def test_bf16_rounding_is_torch_bfloat16():
    rng = np.random.default_rng(2)
    a = (rng.standard_normal(20000) * 10.0 ** rng.integers(-6, 6, 20000)).astype(np.float32)
    a[:4] = [1.00390625, 1.01171875, -1.00390625, 0.0]          # exact ties: to even
    want = torch.tensor(a).bfloat16().double().numpy()
    assert np.array_equal(models.bf16_round(a), want)


def test_mlp_bf16_operands_only_touch_the_d_sized_products():
    X, y, w, C, H = _case("mlp2", m=16, d=32, C=4, H=8, seed=3)
    d = X.shape[1]
    # inputs already representable in bf16 for x and W1 -> forward identical, only delta1 rounding remains
    Xq = models.bf16_round(X).astype(np.float32)
    wq = w.copy()
    wq[: d * H] = models.bf16_round(w[: d * H]).astype(np.float32)
    l1, g1 = models.loss_and_grad("mlp2", wq, Xq, y, C, H, bf16=True)
    l0, g0 = models.loss_and_grad("mlp2", wq, Xq, y, C, H, bf16=False)
    assert l1 == l0
    assert np.array_equal(g1[d * H:], g0[d * H:])                # b1, W2, b2 gradients untouched
    rel = np.linalg.norm(g1[: d * H] - g0[: d * H]) / np.linalg.norm(g0[: d * H])
    assert 0 < rel < 2.0 ** -8


def test_lsq_one_step_by_hand():
    """2 samples, d = 2, m = 2 rows (0 and 1): g = (1/2) X^T (X w - y)."""
    X = np.array([[1.0, 2.0], [3.0, -1.0]], np.float32)
    y = np.array([1.0, 0.5], np.float32)
    w = np.array([0.5, -0.25], np.float32)
    loss, g = models.loss_and_grad("lsq", w, X, y)
    r0, r1 = 0.5 - 0.5 - 1.0, 1.5 + 0.25 - 0.5
    assert loss == 0.5 * (r0 * r0 + r1 * r1)
    assert g.tolist() == [(1 * r0 + 3 * r1) / 2, (2 * r0 - 1 * r1) / 2]
    # a row drawn twice counts twice
    loss2, g2 = models.loss_and_grad("lsq", w, X[[0, 0]], y[[0, 0]])
    assert loss2 == r0 * r0 and g2.tolist() == [r0 * 1.0, r0 * 2.0]


def _serial_sgd(data, w0, eta, m, seed, replica, J, C=1, H=0):
    """Plain minibatch SGD, written separately: what every variant is at P = K = 1."""
    w = np.array(w0, np.float32)
    eta = float(np.float32(eta))
    losses = []
    for j in range(J):
        idx = core.minibatch_indices(seed, replica, 0, j, data["X"].shape[0], m)
        f, g = models.loss_and_grad(data["model"], w, data["X"][idx], data["y"][idx], C, H)
        w = (w.astype(np.float64) - eta * g).astype(np.float32)
        losses.append(np.float32(f / m))
    return w, np.array(losses)


@pytest.mark.parametrize("variant", list(core.VARIANTS))
@pytest.mark.parametrize("model", ["lsq", "logistic", "softmax", "mlp2"])
def test_single_worker_is_serial_sgd(variant, model):
    if model == "lsq":
        data = inputs.make_lsq(256, 16, 0.1, 5)
    elif model == "logistic":
        data = inputs.make_logistic(256, 16, 0.05, 5)
    else:
        data = inputs.make_mixture(256, 16, 4, 0.5, 5, model, 8 if model == "mlp2" else 0)
    C, H = data["n_classes"], data["hidden"]
    w0 = inputs.mlp_init(16, 8, 4, 1) if model == "mlp2" else np.zeros(models.n_params(model, 16, C, H), np.float32)
    sim = OracleReplica(model=model, X=data["X"], y=data["y"], w0=w0, P=1, K=1, variant=variant,
                        delay_kind="exp", mu=1.0, eta=0.05, m=8, seed=3, replica=4, n_classes=C,
                        hidden=H).run(30)
    w, losses = _serial_sgd(data, w0, 0.05, 8, 3, 4, 30, C, H)
    assert np.array_equal(sim.w, w)
    assert np.array_equal(sim.trace_arrays()["loss"], losses)


def test_ksync_update_rule_by_hand_one_iteration():
    """Eq. 2 for one iteration, P=3, K=2: average of the two earliest workers' gradients at w_0."""
    data = inputs.make_lsq(64, 4, 0.0, 6)
    w0 = np.array([0.1, -0.2, 0.3, 0.0], np.float32)
    sim = OracleReplica(model="lsq", X=data["X"], y=data["y"], w0=w0, P=3, K=2, variant="ksync",
                        delay_kind="exp", mu=1.0, eta=0.1, m=4, seed=8, replica=0,
                        w_ref=data["w_star"]).run(1)
    x = [core.delay("exp", 1.0, 0.0, 8, 0, i, 0) for i in range(3)]
    first = sorted(range(3), key=lambda i: x[i])[:2]
    g = np.zeros(4)
    loss = 0.0
    for i in first:
        idx = core.minibatch_indices(8, 0, i, 0, 64, 4)
        r = data["X"][idx].astype(np.float64) @ w0.astype(np.float64) - data["y"][idx]
        g += data["X"][idx].astype(np.float64).T @ r / 4
        loss += 0.5 * r @ r
    w1 = (w0.astype(np.float64) - float(np.float32(0.1)) / 2 * g).astype(np.float32)
    tr = sim.trace_arrays()
    assert np.array_equal(sim.w, w1)
    assert tr["loss"][0] == np.float32(loss / 8) and tr["t"][0] == sorted(x)[1]
    assert tr["dist2"][0] == np.float32(((w1.astype(np.float64) - data["w_star"]) ** 2).sum())


def test_kasync_uses_stale_parameters():
    """Eq. 3: with P=2, K=1 the second push is taken at w_0 whenever its staleness is 1."""
    data = inputs.make_lsq(64, 4, 0.0, 7)
    w0 = np.zeros(4, np.float32)
    sim = OracleReplica(model="lsq", X=data["X"], y=data["y"], w0=w0, P=2, K=1, variant="kasync",
                        delay_kind="exp", mu=1.0, eta=0.2, m=4, seed=2, replica=0)
    sim.run(1)
    w1 = sim.w.copy()
    sim.run(1)
    tr = sim.trace_arrays()
    i, s, st = int(tr["worker"][1, 0]), int(tr["seq"][1, 0]), int(tr["stale"][1, 0])
    at = w0 if st == 1 else w1
    idx = core.minibatch_indices(2, 0, i, s, 64, 4)
    _, g = models.loss_and_grad("lsq", at, data["X"][idx], data["y"][idx])
    assert np.array_equal(sim.w, (w1.astype(np.float64) - float(np.float32(0.2)) * g).astype(np.float32))
    assert {int(tr["worker"][0, 0]), i} == {0, 1} or st == 0


@pytest.mark.parametrize("variant,K", [("ksync", 2), ("kbatchsync", 3), ("kasync", 2), ("kbatchasync", 2)])
def test_noiseless_least_squares_converges_to_w_star(variant, K):
    """With sigma^2 = 0 the error floor eta L sigma^2/(2 c K m) of Theorem 3 / Lemma 7 is zero."""
    data = inputs.make_lsq(4096, 64, 0.0, 1001)
    sim = OracleReplica(model="lsq", X=data["X"], y=data["y"], w0=np.zeros(64, np.float32), P=4, K=K,
                        variant=variant, delay_kind="exp", mu=1.0, eta=0.05,
                        m=16, seed=0, replica=0, w_ref=data["w_star"]).run(2000)
    d2 = sim.trace_arrays()["dist2"]
    n2 = float((data["w_star"].astype(np.float64) ** 2).sum())
    assert d2[-1] / n2 < 1e-10
    assert d2[200] < d2[20] < d2[0]


def test_error_floor_scales_as_one_over_K():
    """Lemma 7: K-sync has the floor of minibatch SGD with batch K m, so doubling K halves it."""
    data = inputs.make_lsq(8192, 32, 1.0, 9)
    Xd, yd = data["X"].astype(np.float64), data["y"].astype(np.float64)
    w_ls = np.linalg.lstsq(Xd, yd, rcond=None)[0]

    def floor(K):
        acc = []
        for r in range(6):
            sim = OracleReplica(model="lsq", X=data["X"], y=data["y"], w0=np.zeros(32, np.float32), P=8,
                                K=K, variant="ksync", delay_kind="exp", mu=1.0, eta=0.02, m=4, seed=1,
                                replica=r, w_ref=w_ls).run(1500)
            acc.append(sim.trace_arrays()["dist2"][500:].mean())
        return np.mean(acc)

    ratio = floor(2) / floor(4)
    assert 1.4 < ratio < 2.8


def test_full_loss_is_the_mean_of_the_per_sample_losses_and_blocks_do_not_matter():
    """Eq. 1: F(w) = (1/N) sum_n f(w, xi_n)."""
    data = inputs.make_lsq(1000, 16, 0.3, 11)
    w = np.linspace(-1, 1, 16).astype(np.float32)
    r = data["X"].astype(np.float64) @ w.astype(np.float64) - data["y"]
    want = float(np.mean(0.5 * r * r))
    assert abs(models.full_loss("lsq", w, data["X"], data["y"]) - want) < 1e-14 * want
    assert abs(models.full_loss("lsq", w, data["X"], data["y"], rows=77) - want) < 1e-13 * want
    mix = inputs.make_mixture(500, 16, 4, 0.5, 12)
    W = (0.1 * np.arange(64) % 0.7).astype(np.float32)
    per = [models.loss_and_grad("softmax", W, mix["X"][i:i + 1], mix["y"][i:i + 1], 4)[0] for i in range(500)]
    assert abs(models.full_loss("softmax", W, mix["X"], mix["y"], 4, rows=64) - np.mean(per)) < 1e-13
    # at the least-squares solution of noiseless data the risk vanishes
    clean = inputs.make_lsq(400, 8, 0.0, 13)
    assert models.full_loss("lsq", clean["w_star"], clean["X"], clean["y"]) < 1e-12


def test_adasync_rule_closed_forms():
    """Section 6: K = K0 sqrt(F0/F) (three variants); K-sync: K^2/(P-K) = K0^2/(P-K0) F0/F."""
    from oracle.sim import adasync_next_K
    import math
    for v in ("kbatchsync", "kasync", "kbatchasync"):
        assert adasync_next_K(v, 1, 16, 1, 4.0, 1.0) == 2          # ratio 4 doubles K
        assert adasync_next_K(v, 2, 16, 2, 9.0, 1.0) == 6
        assert adasync_next_K(v, 1, 8, 1, 1.0, 1.0) == 1            # no progress, no change
        assert adasync_next_K(v, 1, 8, 3, 1.0, 1.0) == 3            # never decreases
        assert adasync_next_K(v, 1, 8, 1, 1.0, 1e-6) == 8           # capped at P
        assert adasync_next_K(v, 1, 8, 1, 1.0, 0.0) == 8            # F = F* = 0: fully synchronous
    rng = np.random.default_rng(5)
    for _ in range(200):
        P = int(rng.integers(2, 33)); K0 = int(rng.integers(1, P)); ratio = float(np.float32(10 ** rng.uniform(0, 3)))
        c = K0 * K0 / (P - K0) * ratio
        k_real = (math.sqrt(c * c + 4 * c * P) - c) / 2               # root of K^2 + cK - cP
        assert abs(k_real ** 2 / (P - k_real) - c) < 1e-9 * c and K0 - 1e-9 <= k_real < P
        got = adasync_next_K("ksync", K0, P, K0, ratio, 1.0)
        if abs(k_real + 0.5 - round(k_real + 0.5)) > 1e-6:
            assert got == min(P, max(K0, math.floor(k_real + 0.5)))
    assert adasync_next_K("ksync", 4, 4, 4, 5.0, 1.0) == 4
    assert adasync_next_K("ksync", 1, 8, 1, 1.0, 1.0) == 1


@pytest.mark.parametrize("variant", list(core.VARIANTS))
def test_loss_driven_adasync_in_the_simulator(variant):
    data = inputs.make_lsq(512, 16, 0.05, 14)
    kw = dict(model="lsq", X=data["X"], y=data["y"], w0=np.zeros(16, np.float32), P=8, K=1, variant=variant,
              delay_kind="shifted_exp", mu=2.0, shift=0.5, eta=0.05, m=4, seed=6, replica=3)
    sim = OracleReplica(K0=1, t_interval=4.0, k_rule="loss", **kw).run(250)
    tr = sim.trace_arrays()
    K = tr["K"].astype(int)
    assert K[0] == 1 and np.all(np.diff(K) >= 0) and K.max() <= 8 and K.max() > 1
    # K changes only at an update that starts in a new interval, and to the rule's value
    t_start = np.concatenate([[0.0], tr["t"][:-1]])
    for j in np.nonzero(np.diff(K))[0] + 1:
        assert math.floor(t_start[j] / 4.0) > math.floor(t_start[j - 1] / 4.0)
    from oracle.sim import adasync_next_K
    F0 = np.float32(models.full_loss("lsq", np.zeros(16, np.float32), data["X"], data["y"]))
    k_prev = 1
    for (j, F, k_new) in sim.k_events:
        assert k_new == adasync_next_K(variant, 1, 8, k_prev, F0, F) and K[j] == k_new
        k_prev = k_new
    # an interval that never ends leaves K at K0: the fixed-K run, bit for bit
    a = OracleReplica(K0=2, t_interval=1e300, k_rule="loss", **{**kw, "K": 0}).run(60).trace_arrays(K_stride=8)
    b = OracleReplica(**{**kw, "K": 2}).run(60).trace_arrays(K_stride=8)
    for k in ("t", "K", "worker", "stale", "seq", "loss"):
        assert np.array_equal(a[k], b[k]), k
