"""GPU parity for the two-layer MLP (bf16 tensor-core products over d, fp32 elsewhere) against the
oracle, which rounds the same three operand tensors to bf16 and accumulates in fp64.  Schedule
bit-exact; every update's loss and the final loss within 1e-3 relative; parameters within 1e-3
in relative 2-norm (a flipped bf16 rounding of one delta1 element moves one gradient entry by
2^-9 of itself, so the fp32 bound of the linear models does not apply here)."""
import numpy as np
import pytest
import torch

from oracle import core
from paper_2003_10579_b200 import inputs
from parity import assert_schedule_equal, oracle_replica, rel_norm, to_device

pytestmark = pytest.mark.gpu

MLP_LOSS_RTOL = 1e-3
MLP_PARAM_RTOL = 1e-3


@pytest.fixture(scope="module")
def B():
    from paper_2003_10579_b200 import binding
    return binding


def run_mlp_case(B, data, w0, *, variant, P, K, m, eta, R, J, kind="exp", mu=1.0, shift=0.0, seed=3, base=0, K0=0,
                 ti=0.0, replicas=None, chunks=(1, 1), w_ref=None):
    dev = to_device(data)
    sim = B.Simulation(dev, P=P, K=K, variant=variant, delay_kind=kind, mu=mu, shift=shift, eta=eta, m=m,
                       seed=seed, n_replicas=R, replica_base=base, w_ref=None if w_ref is None else torch.from_numpy(w_ref).cuda())
    if ti > 0:
        sim.set_adasync(K0, ti)
    sim.set_params(torch.from_numpy(w0).cuda())
    kw = dict(P=P, K=K, variant=variant, delay_kind=kind, mu=mu, shift=shift, eta=eta, m=m, seed=seed, K0=K0, t_interval=ti,
              w_ref=w_ref)
    replicas = list(range(R)) if replicas is None else replicas
    oras = {r: oracle_replica(data, w0, base + r, **kw) for r in replicas}
    plan = list(chunks) + ([J - sum(chunks)] if J > sum(chunks) else [])
    worst_w = 0.0
    for c in plan:
        sim.run(c)
        w = sim.params()
        for r, o in oras.items():
            o.run(c)
            e = rel_norm(w[r], o.w)
            assert e <= MLP_PARAM_RTOL, "%s replica %d update %d: param err %.3g" % (variant, r, o.j, e)
            worst_w = max(worst_w, e)
    tr = sim.trace()
    sim.close()
    sched = core.BulkSchedule(variant, P, K, kind, mu, shift, seed, R, replica_base=base, K0=K0, t_interval=ti).run(J)
    assert_schedule_equal(tr, sched)
    worst_l = 0.0
    for r, o in oras.items():
        ot = o.trace_arrays(K_stride=tr["worker"].shape[2])
        ol = ot["loss"].astype(np.float64)
        err = np.abs(tr["loss"][r] - ol) / np.abs(ol)
        assert err.max() <= MLP_LOSS_RTOL, "%s replica %d: loss err %.3g at update %d" % (variant, r, err.max(), err.argmax())
        worst_l = max(worst_l, err.max())
        if w_ref is None:
            assert not tr["dist2"][r].any()
        else:       # Section 2.3's distance to a reference point, |w_{j+1} - w_ref|^2, over all four parameter blocks
            od = ot["dist2"].astype(np.float64)
            derr = np.abs(tr["dist2"][r] - od) / od
            assert derr.max() <= MLP_LOSS_RTOL, "%s replica %d: dist2 err %.3g at update %d" % (variant, r, derr.max(), derr.argmax())
    print("mlp %s K=%d d=%d H=%d: worst param err %.2e, worst loss err %.2e, final loss %.4f" % (
        variant, K, data["X"].shape[1], data["hidden"], worst_w, worst_l, tr["loss"][replicas[0], -1]))
    return tr


@pytest.mark.parametrize("variant", list(core.VARIANTS))
@pytest.mark.parametrize("d,H,C,m,K,P", [(128, 64, 3, 128, 2, 4), (256, 192, 10, 256, 3, 5), (3072, 512, 10, 128, 4, 16),
                                         # a hidden width whose halves are no multiple of 64, all 16 classes; 5..8 classes
                                         (128, 320, 16, 128, 2, 4), (256, 128, 7, 128, 2, 3)])
def test_mlp_variants_and_shapes(B, variant, d, H, C, m, K, P):
    data = inputs.make_mixture(4096, d, C, 0.5 if d < 1000 else 0.1, 95, "mlp2", H)
    w0 = inputs.mlp_init(d, H, C, 96)
    # every other case carries a reference vector: another draw of the initial weights, shifted so that no block of the
    # parameter vector is close to it by accident
    w_ref = (inputs.mlp_init(d, H, C, 197) + np.float32(0.01)) if (d + K) % 2 == 0 or variant == "kbatchasync" else None
    run_mlp_case(B, data, w0, variant=variant, P=P, K=K, m=m, eta=0.02, R=3, J=12 if d > 1000 else 25, base=1, w_ref=w_ref)


@pytest.mark.parametrize("variant", ["kasync", "kbatchasync"])
def test_mlp_more_workers_than_warp_lanes(B, variant):
    """P = 40: 42 parameter versions (and W1 shadows) per replica, two workers per lane in the arrival kernel."""
    data = inputs.make_mixture(2048, 128, 3, 0.5, 99, "mlp2", 64)
    w0 = inputs.mlp_init(128, 64, 3, 100)
    run_mlp_case(B, data, w0, variant=variant, P=40, K=3, m=128, eta=0.02, R=2, J=20, base=2)


def test_mlp_growing_K_and_resume(B):
    data = inputs.make_mixture(2048, 128, 4, 0.5, 97, "mlp2", 64)
    w0 = inputs.mlp_init(128, 64, 4, 98)
    run_mlp_case(B, data, w0, variant="kbatchasync", P=8, K=1, m=128, eta=0.02, R=4, J=60, K0=1, ti=2.0, chunks=(1, 7, 20))
    dev = to_device(data)
    kw = dict(P=6, K=3, variant="kasync", delay_kind="exp", mu=1.0, eta=0.02, m=128, seed=1, n_replicas=3)
    a, b = B.Simulation(dev, **kw), B.Simulation(dev, **kw)
    for s in (a, b):
        s.set_params(torch.from_numpy(w0).cuda())
    a.run(20)
    for c in (1, 6, 13):
        b.run(c)
    ta, tb = a.trace(), b.trace()
    for k in ta:
        assert np.array_equal(ta[k], tb[k]), k
    assert np.array_equal(a.params(), b.params())
    a.close(); b.close()


def test_mlp_results_do_not_depend_on_sharding(B):
    """Replicas 3 and 4 of a six-replica handle and the same global replicas in a two-replica handle: every trace array
    and every parameter bit for bit (the tile order of the persistent kernels depends on the replica count, the sums
    must not)."""
    data = inputs.make_mixture(2048, 256, 10, 0.5, 101, "mlp2", 512)
    w0 = inputs.mlp_init(256, 512, 10, 102)
    dev = to_device(data)
    kw = dict(P=5, K=3, variant="kbatchasync", delay_kind="exp", mu=1.0, eta=0.02, m=128, seed=4)
    full = B.Simulation(dev, n_replicas=6, **kw)
    part = B.Simulation(dev, n_replicas=2, replica_base=3, **kw)
    for s in (full, part):
        s.set_params(torch.from_numpy(w0).cuda())
        s.run(9)
    tf, tp = full.trace(), part.trace()
    for k in tf:
        assert np.array_equal(tf[k][3:5], tp[k]), k
    assert np.array_equal(full.params()[3:5], part.params())
    assert np.array_equal(full.eval_loss()[3:5], part.eval_loss())
    full.close(); part.close()


def test_mlp_unsupported_shapes_are_refused(B):
    data = inputs.make_mixture(64, 128, 4, 0.5, 99, "mlp2", 100)
    with pytest.raises(B.SimError) as e:
        B.Simulation(to_device(data), P=2, K=1, variant="ksync", delay_kind="exp", mu=1.0, eta=0.1, m=128, seed=0, n_replicas=1)
    assert e.value.status == 1
