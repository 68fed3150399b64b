"""Helpers shared by the GPU parity tests: run the library and the CPU oracle on the same seeded
inputs and compare.  Integers and fp64 times must be bit-identical; fp32 parameters must agree
to 1e-5 in relative 2-norm at every compared step and per-update losses to 1e-5 relative."""
import numpy as np
import torch

from oracle import core
from oracle.sim import OracleReplica

PARAM_RTOL = 1e-5
LOSS_RTOL = 1e-5


def to_device(data):
    out = {"model": data["model"], "n_classes": data.get("n_classes", 1), "hidden": data.get("hidden", 0)}
    out["X"] = torch.from_numpy(data["X"]).cuda()
    out["y"] = torch.from_numpy(data["y"]).cuda()
    return out


def assert_schedule_equal(gpu, ora, rows=None):
    """gpu: trace dict from the library; ora: dict from oracle BulkSchedule.run (same shapes)."""
    for k in ("t", "K", "worker", "stale", "seq"):
        a, b = gpu[k], ora[k]
        if rows is not None:
            a = a[rows]
        if k == "t":
            a, b = a.view(np.int64), b.view(np.int64)     # bit-exact fp64
        assert a.shape == b.shape, (k, a.shape, b.shape)
        if not np.array_equal(a, b):
            bad = np.argwhere(a != b)[0]
            raise AssertionError("schedule mismatch in %s at %s: gpu %s oracle %s" % (k, bad, a[tuple(bad)], b[tuple(bad)]))


def oracle_schedule(wl_kw, variant, K, R, J, replica_base=0, K0=0, t_interval=0.0, chunks=None):
    b = core.BulkSchedule(variant, wl_kw["P"], K, wl_kw["delay_kind"], wl_kw["mu"], wl_kw["shift"], wl_kw["seed"], R,
                          replica_base=replica_base, K0=K0, t_interval=t_interval)
    return b.run(J)


def oracle_replica(data, w0, r, *, P, K, variant, delay_kind, mu, shift, eta, m, seed, w_ref=None, K0=0, t_interval=0.0):
    return OracleReplica(model=data["model"], X=data["X"], y=data["y"], w0=w0, P=P, K=K, variant=variant,
                         delay_kind=delay_kind, mu=mu, shift=shift, eta=eta, m=m, seed=seed, replica=r,
                         n_classes=data.get("n_classes", 1), hidden=data.get("hidden", 0), w_ref=w_ref,
                         K0=K0, t_interval=t_interval)


def rel_norm(a, b):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    nb = np.linalg.norm(b)
    return np.linalg.norm(a - b) / (nb if nb > 0 else 1.0)


def max_elem_err(w_gpu, w_ora):
    """Largest element-wise difference relative to the largest parameter: max_i |dw_i| / max_i |w_i|."""
    a, b = np.asarray(w_gpu, np.float64), np.asarray(w_ora, np.float64)
    top = np.abs(b).max()
    return np.abs(a - b).max() / (top if top > 0 else 1.0)


def assert_params_close(w_gpu, w_ora, what="", rtol=PARAM_RTOL):
    """Two bounds at the same tolerance: the relative 2-norm of the difference, and every single element against
    the largest parameter (a norm alone would let one element of thousands be off by much more).  Returns the
    larger of the two measures."""
    e = rel_norm(w_gpu, w_ora)
    assert e <= rtol, "%s: |w_gpu - w_oracle| / |w_oracle| = %.3g > %.1g" % (what, e, rtol)
    a, b = np.asarray(w_gpu, np.float64), np.asarray(w_ora, np.float64)
    m = max_elem_err(a, b)
    if m > rtol:
        i = int(np.argmax(np.abs(a - b)))
        raise AssertionError("%s: element %d differs by %.3g (gpu %.9g oracle %.9g), %.3g of the largest parameter > %.1g" % (
            what, i, abs(a.flat[i] - b.flat[i]), a.flat[i], b.flat[i], m, rtol))
    return max(e, m)


def strict_loss_stats(l_gpu, l_ora, rtol=LOSS_RTOL):
    """The plain relative bound, with no allowance for trajectory drift: (fraction of updates inside rtol, worst
    relative error), relative to max(|L_oracle|, 1e-6 L_0)."""
    l_gpu, l_ora = np.asarray(l_gpu, np.float64), np.asarray(l_ora, np.float64)
    rel = np.abs(l_gpu - l_ora) / np.maximum(np.abs(l_ora), 1e-6 * abs(l_ora.flat[0]))
    return float((rel <= rtol).mean()), float(rel.max())


def assert_loss_close(l_gpu, l_ora, what="", rtol=LOSS_RTOL, gnorm=None, dw=0.0):
    """Per update: |dL| <= rtol * max(|L_oracle|, 1e-6 * L_0) + 2 |g_j| dw.

    L_0 is the first update's loss.  The second term is the first-order effect on the minibatch
    loss of the parameter difference actually measured between the two trajectories (dw = the
    largest |w_gpu - w_oracle|_2 seen at the compared steps, itself held to 1e-5 |w|; g_j = the
    oracle's averaged gradient of update j, the gradient of that minibatch loss): two fp32-stored
    trajectories drift apart by a few ulp per parameter, and a loss that has decayed by orders of
    magnitude (or sits at its noise floor) magnifies that drift beyond any fixed relative bound.
    Without gnorm the plain relative bound applies."""
    l_gpu, l_ora = np.asarray(l_gpu, np.float64), np.asarray(l_ora, np.float64)
    floor = 1e-6 * abs(l_ora.flat[0])
    allow = rtol * np.maximum(np.abs(l_ora), floor)
    if gnorm is not None:
        allow = allow + 2.0 * np.asarray(gnorm, np.float64) * dw
    err = np.abs(l_gpu - l_ora)
    bad = err > allow
    if bad.any():
        j = int(np.argmax(err / allow))
        raise AssertionError("%s: loss differs by %.3g (allowed %.3g) at update %d (gpu %.9g oracle %.9g)" % (
            what, err.flat[j], allow.flat[j], j, l_gpu.flat[j], l_ora.flat[j]))
    rel = err / np.maximum(np.abs(l_ora), floor)
    return rel.max()
