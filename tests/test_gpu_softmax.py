"""GPU parity for softmax regression (multi-class linear model) under every variant and the
growing-K schedule, against the oracle."""
import numpy as np
import pytest

from oracle import core
from paper_2003_10579_b200 import inputs
from test_gpu_linear import run_case

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2003_10579_b200 import binding
    return binding


@pytest.mark.parametrize("variant", list(core.VARIANTS))
@pytest.mark.parametrize("d,C,m,K,P", [(64, 3, 8, 2, 4), (3072, 10, 21, 2, 8), (1536, 16, 6, 3, 5), (200, 10, 128, 1, 2), (1540, 7, 9, 4, 4)])
def test_softmax_variants_and_shapes(B, variant, d, C, m, K, P):
    data = inputs.make_mixture(2000, d, C, 0.5 if d < 1000 else 0.05, 90)
    run_case(B, data, variant=variant, P=P, K=K, m=m, eta=0.05, R=3, J=30, kind="shifted_exp", mu=2.0, shift=1.0,
             base=2, chunks=[10], use_ref=False)


@pytest.mark.parametrize("variant", ["ksync", "kbatchasync"])
@pytest.mark.parametrize("d,C,m", [(3072, 10, 21), (1540, 7, 9), (1536, 16, 6), (64, 3, 8)])
def test_softmax_distance_to_a_reference(B, variant, d, C, m):
    """`dist2` = |W_{j+1} - W_ref|^2 of every update, for both softmax kernels (tensor-memory parameters up to
    10 classes, shared-memory parameters beyond), ragged tiles included."""
    data = inputs.make_mixture(1500, d, C, 0.5 if d < 1000 else 0.05, 92)
    data["w_star"] = (0.01 * np.random.default_rng(93).standard_normal(C * d)).astype(np.float32)
    run_case(B, data, variant=variant, P=4, K=2, m=m, eta=0.05, R=2, J=20, kind="exp", mu=1.0, shift=0.0,
             base=0, chunks=[7], use_ref=True)


def test_softmax_growing_K_scaled_fourth_workload(B):
    """Shape of the AdaSync workload (P=8, m=128, eta=0.05, Delta=1, mu=2, K doubling 1 -> 8) on a
    smaller data set, with an interval short enough to cross every K within the run."""
    wl = inputs.WORKLOADS[4].scaled(n=4096, replicas=6, updates=90, t_interval=25.0)
    data = wl.make_data()
    tr = run_case(B, data, variant="ksync", P=wl.P, K=1, m=wl.m, eta=wl.eta, R=wl.replicas, J=wl.updates,
                  kind=wl.delay_kind, mu=wl.mu, shift=wl.shift, seed=wl.seed, K0=wl.K0, ti=wl.t_interval,
                  replicas=[0, 5], chunks=[30], use_ref=False)
    assert set(np.unique(tr["K"])) == {1, 2, 4, 8}


@pytest.mark.parametrize("variant,C", [("ksync", 10), ("kasync", 10), ("kbatchasync", 13)])
def test_softmax_results_do_not_depend_on_sharding(B, variant, C):
    """Replicas 3 and 4 of a six-replica handle and the same global replicas in a two-replica handle, bit for bit
    (both softmax kernels: up to 10 classes and 11 to 16)."""
    import torch
    from parity import to_device
    data = inputs.make_mixture(1500, 3072 if C <= 10 else 1536, C, 0.05, 93)      # the 11..16-class kernel takes d <= 1536
    dev = to_device(data)
    kw = dict(P=4, K=2, variant=variant, delay_kind="exp", mu=1.0, eta=0.05, m=20, seed=6)
    full = B.Simulation(dev, n_replicas=6, **kw)
    part = B.Simulation(dev, n_replicas=2, replica_base=3, **kw)
    for s in (full, part):
        s.run(15)
    tf, tp = full.trace(), part.trace()
    for k in tf:
        assert np.array_equal(tf[k][3:5], tp[k]), k
    assert np.array_equal(full.params()[3:5], part.params())
    full.close(); part.close()


def test_softmax_unsupported_shapes_are_refused(B):
    data = inputs.make_mixture(64, 4096, 10, 0.5, 91)
    from parity import to_device
    with pytest.raises(B.SimError) as e:
        B.Simulation(to_device(data), P=2, K=1, variant="ksync", delay_kind="exp", mu=1.0, eta=0.1, m=4, seed=0, n_replicas=1)
    assert e.value.status == 1
