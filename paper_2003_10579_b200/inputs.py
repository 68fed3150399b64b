"""Seeded synthetic inputs for the five simulation workloads.

This module only makes data (torch CPU generator, fixed seeds): it contains none of the
simulation's arithmetic and is the one module that both the CUDA tests/benchmark and the CPU
oracle's tests may use, so that both sides receive the same bytes.

Recipes (every array is fp32 on the host; seed_data = 1000 + workload index):
  lsq       X ~ N(0,1)^{n x d}, w* ~ N(0,1)^d, y = X w* (+ N(0, noise^2)); the product is taken in
            fp64 and rounded once
  logistic  X ~ N(0,1)^{n x d}, label = [X w* > 0], flipped with probability `flip`
  mixture   n_classes means ~ N(0, mean_std^2)^d, class uniform, x = mean[class] + N(0,1)^d
            (a stand-in with the 32x32x3 = 3072-feature, 10-class shape of the paper's
            CIFAR-10 experiments of Section 5.1; no CIFAR data is used)
  mlp_init  uniform(+-1/sqrt(fan_in)) for both layers, biases included
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def _randn(shape, g) -> torch.Tensor:
    return torch.randn(shape, generator=g, dtype=torch.float32)


def _xw(X: torch.Tensor, w: torch.Tensor, rows: int = 8192) -> torch.Tensor:
    """X @ w in fp64, chunked over rows so that a 4 GiB X needs no 8 GiB copy."""
    out = torch.empty(X.shape[0], dtype=torch.float64)
    w64 = w.double()
    for a in range(0, X.shape[0], rows):
        out[a:a + rows] = X[a:a + rows].double() @ w64
    return out


def make_lsq(n: int, d: int, noise_std: float, seed: int):
    g = _gen(seed)
    X = _randn((n, d), g)
    w_star = _randn((d,), g)
    y = _xw(X, w_star)
    if noise_std > 0:
        y = y + noise_std * _randn((n,), g).double()
    return {"model": "lsq", "X": X.numpy(), "y": y.float().numpy(), "w_star": w_star.numpy(),
            "n_classes": 1, "hidden": 0}


def make_logistic(n: int, d: int, flip: float, seed: int):
    g = _gen(seed)
    X = _randn((n, d), g)
    w_star = _randn((d,), g)
    lab = (_xw(X, w_star) > 0)
    flips = torch.rand((n,), generator=g) < flip
    lab = (lab ^ flips).to(torch.int32)
    return {"model": "logistic", "X": X.numpy(), "y": lab.numpy(), "w_star": w_star.numpy(),
            "n_classes": 1, "hidden": 0}


def make_mixture(n: int, d: int, n_classes: int, mean_std: float, seed: int, model: str = "softmax",
                 hidden: int = 0):
    g = _gen(seed)
    means = mean_std * _randn((n_classes, d), g)
    lab = torch.randint(0, n_classes, (n,), generator=g, dtype=torch.int64)
    X = _randn((n, d), g)
    rows = 8192
    for a in range(0, n, rows):
        X[a:a + rows] += means[lab[a:a + rows]]
    return {"model": model, "X": X.numpy(), "y": lab.to(torch.int32).numpy(), "w_star": None,
            "n_classes": n_classes, "hidden": hidden}


def mlp_init(d: int, hidden: int, n_classes: int, seed: int) -> np.ndarray:
    """[W1 (d x hidden), b1, W2 (hidden x n_classes), b2], each uniform(+-1/sqrt(fan_in))."""
    g = _gen(seed)

    def u(shape, fan_in):
        return (torch.rand(shape, generator=g, dtype=torch.float32) * 2 - 1) / math.sqrt(fan_in)

    return torch.cat([u((d * hidden,), d), u((hidden,), d), u((hidden * n_classes,), hidden),
                      u((n_classes,), hidden)]).numpy()


@dataclass
class Workload:
    """One simulation workload: the data recipe plus the simulation's parameters."""
    name: str
    model: str
    n: int
    d: int
    P: int
    m: int
    eta: float
    delay_kind: str
    mu: float
    shift: float
    replicas: int
    updates: int
    runs: list = field(default_factory=list)      # [(variant, K), ...]
    n_classes: int = 1
    hidden: int = 0
    noise_std: float = 0.0
    flip: float = 0.0
    mean_std: float = 0.5
    seed_data: int = 0
    seed: int = 0
    K0: int = 0
    t_interval: float = 0.0

    def scaled(self, **kw) -> "Workload":
        """A copy with some sizes replaced (smaller n, d, replicas, updates for tests)."""
        w = Workload(**{**self.__dict__, **kw})
        w.runs = [(v, min(K, w.P)) for v, K in w.runs]
        return w

    def make_data(self):
        if self.model == "lsq":
            return make_lsq(self.n, self.d, self.noise_std, self.seed_data)
        if self.model == "logistic":
            return make_logistic(self.n, self.d, self.flip, self.seed_data)
        return make_mixture(self.n, self.d, self.n_classes, self.mean_std, self.seed_data,
                            self.model, self.hidden)

    def w0(self) -> np.ndarray:
        if self.model == "mlp2":
            return mlp_init(self.d, self.hidden, self.n_classes, self.seed_data + 500)
        npar = self.d * (self.n_classes if self.model == "softmax" else 1)
        return np.zeros(npar, np.float32)


WORKLOADS = {
    1: Workload("ksync_lsq_small", "lsq", 4096, 64, P=4, m=16, eta=0.01, delay_kind="exp", mu=1.0,
                shift=0.0, replicas=64, updates=200, runs=[("ksync", 2)], seed_data=1001),
    2: Workload("sync_sweep_lsq", "lsq", 65536, 1024, P=16, m=32, eta=0.005,
                delay_kind="shifted_exp", mu=1.0, shift=0.5, replicas=1024, updates=1000,
                runs=[(v, K) for v in ("ksync", "kbatchsync") for K in range(1, 17)],
                noise_std=0.1, seed_data=1002),
    3: Workload("async_logistic", "logistic", 262144, 4096, P=32, m=64, eta=0.01, delay_kind="exp",
                mu=1.0, shift=0.0, replicas=256, updates=2000,
                runs=[(v, K) for v in ("kasync", "kbatchasync") for K in (1, 4, 8)],
                flip=0.05, seed_data=1003),
    4: Workload("adasync_softmax", "softmax", 65536, 3072, P=8, m=128, eta=0.05,
                delay_kind="shifted_exp", mu=2.0, shift=1.0, replicas=128, updates=3000,
                runs=[("ksync", 1)], n_classes=10, mean_std=0.5, seed_data=1004, K0=1,
                t_interval=800.0),
    5: Workload("kbatchasync_mlp", "mlp2", 262144, 3072, P=16, m=128, eta=0.02, delay_kind="exp",
                mu=1.0, shift=0.0, replicas=64, updates=2000, runs=[("kbatchasync", 4)],
                n_classes=10, hidden=512, mean_std=0.5, seed_data=1005),
}
