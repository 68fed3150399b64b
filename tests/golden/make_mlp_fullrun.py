"""Writes tests/golden/mlp_fullrun_replica0.npz: the CPU oracle's trajectory of replica 0 of the
K-batch-async MLP workload (3072-512-10 on 262144 samples, P = 16, K = 4, m = 128, eta = 0.02,
Exp(1) delays) over all 2000 updates, which the oracle needs several minutes for and the GPU
tests therefore read from this file instead of recomputing.

Calls only the oracle and the seeded input generators:

    python tests/golden/make_mlp_fullrun.py

Stored: the 2000 per-update minibatch losses (fp32), and at updates 150, 1000 and 2000 a fixed
sample of the parameter vector (every 389th entry - 389 is prime, so the sample runs through all
columns of W1 - plus the whole of b1, W2, b2), with the 2-norm of the full vector at each checkpoint.
"""
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle.sim import OracleReplica  # noqa: E402
from paper_2003_10579_b200 import inputs  # noqa: E402

CHECKPOINTS = (150, 1000, 2000)
STRIDE = 389
OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "mlp_fullrun_replica0.npz")


def sample_index(wl):
    dH = wl.d * wl.hidden
    npar = dH + wl.hidden + wl.hidden * wl.n_classes + wl.n_classes
    return np.concatenate([np.arange(0, dH, STRIDE), np.arange(dH, npar)]).astype(np.int64)


def fingerprint(data, w0):
    """Digest of the generated inputs: the stored trajectory belongs to these exact bytes."""
    import hashlib
    h = hashlib.sha256()
    for a in (data["X"][:: max(1, data["X"].shape[0] // 512)], data["y"], w0):
        h.update(np.ascontiguousarray(a).tobytes())
    return h.hexdigest()


def trajectory(wl, data, progress=False):
    """Replica 0 of the workload followed by the oracle for all its updates; returns the arrays that are stored."""
    variant, K = wl.runs[0]
    o = OracleReplica(model="mlp2", X=data["X"], y=data["y"], w0=wl.w0(), P=wl.P, K=K, variant=variant,
                      delay_kind=wl.delay_kind, mu=wl.mu, shift=wl.shift, eta=wl.eta, m=wl.m, seed=wl.seed, replica=0,
                      n_classes=wl.n_classes, hidden=wl.hidden)
    idx = sample_index(wl)
    out = {"index": idx, "checkpoints": np.array(CHECKPOINTS, np.int64), "inputs_sha256": np.array(fingerprint(data, wl.w0()))}
    t0 = time.time()
    for c in CHECKPOINTS:
        o.run(c - o.j)
        out["w_sample_%d" % c] = o.w[idx].copy()
        out["w_norm_%d" % c] = np.float64(np.linalg.norm(o.w.astype(np.float64)))
        if progress:
            print("update %d after %.0f s, loss %.6f" % (c, time.time() - t0, o.trace["loss"][-1]), flush=True)
    tr = o.trace_arrays()
    out["loss"] = tr["loss"]
    out["t"] = tr["t"]
    return out


def main():
    wl = inputs.WORKLOADS[5]
    out = trajectory(wl, wl.make_data(), progress=True)
    np.savez_compressed(OUT, **out)
    print("wrote", OUT, os.path.getsize(OUT), "bytes")


if __name__ == "__main__":
    main()
