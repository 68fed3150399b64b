"""ORACLE (test infrastructure, CPU only): event-driven simulator of one parameter server with P
straggling workers, one replica at a time, written from the definitions of Section 2.2.

Each worker holds the parameter vector it last fetched (a reference to an immutable array), the
sequence number of the minibatch it is working on and the time that task ends.  The server holds
w_j and the simulated wall clock.  One call of ``step()`` performs one server update
    w_{j+1} = w_j - (eta/K) sum_{l<=K} g(w_{tau(l,j)}, xi_{l,j})          (Eq. 2 / Eq. 3)
and records the clock, the contributors in arrival order, their staleness j - tau(l,j), the
minibatch loss (1/(K m)) sum_l sum_q f(w_{tau(l,j)}; xi) and, given w_ref, |w_{j+1} - w_ref|^2.

Random quantities come from ``oracle.core`` (delay of task (replica, worker, seq); the m sample
indices of that task).  Gradients come from ``oracle.models`` in fp64; the stored parameters are
fp32, rounded once per update.

Readings taken where the text leaves a choice:
  * ties in arrival time go to the lower worker id;
  * K-async: the K contributors wait for the update and restart together at the update time
    (Section 2.2 notes the idle wait; the proof of Lemma 3 has K of the read times equal t_0);
  * K-batch-async: a pusher fetches after its push has been counted, so the K-th pusher of an
    update reads w_{j+1};
  * a cancelled task still consumes its sequence number;
  * with a K schedule, K for an update is K0 doubled once per whole interval elapsed at the
    previous update's time, capped at P (Algorithm 1's interval structure);
  * with k_rule="loss" (Algorithm 1 and Section 6 as printed): whenever an update starts in a later
    interval than the one K was last set in, and K < P, K is recomputed from the full-data risk
    F(w_start) of the parameters at that moment (F* taken as 0, F rounded to fp32 as a device
    computes it): K = K0 sqrt(F(w_0)/F(w_start)) for K-batch-sync, K-async, K-batch-async; for K-sync
    the root of K^2/(P-K) = K0^2/(P-K0) F(w_0)/F(w_start).  The real value is rounded half up and
    K never decreases nor exceeds P.
"""
from __future__ import annotations

import math

import numpy as np

from . import core, models


def adasync_k_real(variant, K0, P, F0, F):
    """The real-valued K of Section 6 / Algorithm 1 (fp64 on fp32 risks); inf once F reaches F* = 0."""
    F0, F = float(np.float32(F0)), float(np.float32(F))
    if not (F > 0.0 and math.isfinite(F) and math.isfinite(F0)):
        return math.inf
    ratio = F0 / F
    if variant == "ksync":
        if K0 >= P:
            return float(P)
        c = (float(K0 * K0) / float(P - K0)) * ratio        # K^2 = c (P - K)
        disc = c * c + (4.0 * c) * float(P)
        return (math.sqrt(disc) + (-c)) * 0.5
    return float(K0) * math.sqrt(ratio)


def adasync_next_K(variant, K0, P, K_prev, F0, F):
    """One interval boundary: the real value rounded half up, never decreasing, at most P."""
    k_real = adasync_k_real(variant, K0, P, F0, F)
    K = int(math.floor(k_real + 0.5)) if k_real < 1e9 else P
    return min(P, max(K_prev, K))


class OracleReplica:
    def __init__(self, *, model, X, y, w0, P, K, variant, delay_kind, mu, shift=0.0, eta, m, seed,
                 replica, n_classes=1, hidden=0, w_ref=None, K0=0, t_interval=0.0, bf16=True, k_rule="doubling"):
        assert variant in core.VARIANTS and 1 <= P and 1 <= m
        self.model, self.X, self.y = model, X, y
        self.n = 0 if X is None else X.shape[0]
        self.n_classes, self.hidden, self.bf16 = n_classes, hidden, bf16
        self.P, self.K_fixed, self.variant = P, K, variant
        self.delay_kind, self.mu, self.shift = delay_kind, mu, shift
        self.eta = float(np.float32(eta))
        self.m, self.seed, self.r = m, seed, replica
        self.K0, self.t_interval = K0, t_interval
        self.k_rule, self.K_cur, self.q_last, self.F0 = k_rule, K0, 0, None
        self.k_events = []               # (update index, F(w_start), new K) at every recomputation
        self.w_ref = None if w_ref is None else np.asarray(w_ref, np.float64)
        self.w = None if w0 is None else np.array(w0, dtype=np.float32)   # w_j
        self.j = 0
        self.t = 0.0
        self.s = [0] * P                 # tasks launched so far by worker i
        self.tau = [0] * P               # version worker i last fetched
        self.snap = [self.w] * P         # the parameters worker i last fetched
        self.f = [0.0] * P               # absolute end time of worker i's running task
        self.started = False
        self.trace = {k: [] for k in ("t", "K", "worker", "stale", "seq", "loss", "dist2", "gnorm")}

    # -- random quantities ----------------------------------------------------------------
    def _delay(self, i):
        """Draw the compute time of worker i's next task and consume its sequence number."""
        x = core.delay(self.delay_kind, self.mu, self.shift, self.seed, self.r, i, self.s[i])
        self.s[i] += 1
        return x

    def _K_now(self):
        if not self.t_interval > 0.0:
            return self.K_fixed
        if self.k_rule == "loss":
            if self.F0 is None:
                self.F0 = np.float32(self._risk())
            q = math.floor(self.t / self.t_interval)
            if q > self.q_last and self.K_cur < self.P:
                F = np.float32(self._risk())
                self.K_cur = adasync_next_K(self.variant, self.K0, self.P, self.K_cur, self.F0, F)
                self.q_last = q
                self.k_events.append((self.j, float(F), self.K_cur))
            return self.K_cur
        q = math.floor(self.t / self.t_interval)
        K = self.K0
        while q > 0 and K < self.P:
            K, q = 2 * K, q - 1
        return min(K, self.P)

    # -- numerics -------------------------------------------------------------------------
    def _risk(self):
        return models.full_loss(self.model, self.w, self.X, self.y, self.n_classes, self.hidden, self.bf16)

    def _gradient(self, w_at, i, seq):
        idx = core.minibatch_indices(self.seed, self.r, i, seq, self.n, self.m)
        return models.loss_and_grad(self.model, w_at, self.X[idx], self.y[idx], self.n_classes,
                                    self.hidden, self.bf16)

    def _apply(self, contributions, K):
        """contributions: list of (worker, seq, parameters the gradient is taken at, tau)."""
        tr = self.trace
        tr["t"].append(self.t)
        tr["K"].append(K)
        tr["worker"].append([c[0] for c in contributions])
        tr["seq"].append([c[1] for c in contributions])
        tr["stale"].append([self.j - c[3] for c in contributions])
        if self.w is not None:
            total = np.zeros(self.w.shape[0], np.float64)
            loss = 0.0
            for (i, seq, w_at, _tau) in contributions:
                f_sum, g = self._gradient(w_at, i, seq)
                total += g
                loss += f_sum
            self.w = (self.w.astype(np.float64) - (self.eta / K) * total).astype(np.float32)
            tr["loss"].append(np.float32(loss / (K * self.m)))
            tr["gnorm"].append(float(np.linalg.norm(total)) / K)     # |averaged gradient| of this update
            if self.w_ref is not None:
                dv = self.w.astype(np.float64) - self.w_ref
                tr["dist2"].append(np.float32(dv @ dv))
        self.j += 1

    # -- one update of each variant ----------------------------------------------------------
    def _step_ksync(self):
        K, P = self._K_now(), self.P
        x = [self._delay(i) for i in range(P)]           # all P start a minibatch at w_j
        first = sorted(range(P), key=lambda i: (x[i], i))[:K]
        self.t += x[first[-1]]                           # the iteration lasts X_{K:P}
        self._apply([(i, self.s[i] - 1, self.w, self.j) for i in first], K)

    def _step_kbatchsync(self):
        K, P = self._K_now(), self.P
        c = [self._delay(i) for i in range(P)]           # offsets from the iteration start
        got = []
        for l in range(K):
            i = min(range(P), key=lambda a: (c[a], a))
            got.append((i, self.s[i] - 1, self.w, self.j))
            T = c[i]
            if l + 1 < K:                                # starts another minibatch at the same w_j
                c[i] = c[i] + self._delay(i)
        self.t += T
        self._apply(got, K)

    def _launch_all(self):
        for i in range(self.P):
            self.tau[i], self.snap[i] = 0, self.w
            self.f[i] = 0.0 + self._delay(i)
        self.started = True

    def _step_kasync(self):
        if not self.started:
            self._launch_all()
        K, P = self._K_now(), self.P
        first = sorted(range(P), key=lambda i: (self.f[i], i))[:K]
        self.t = self.f[first[-1]]
        self._apply([(i, self.s[i] - 1, self.snap[i], self.tau[i]) for i in first], K)
        for i in first:                                  # fetch w_{j+1}, restart together
            self.tau[i], self.snap[i] = self.j, self.w
            self.f[i] = self.t + self._delay(i)

    def _step_kbatchasync(self):
        if not self.started:
            self._launch_all()
        K, P = self._K_now(), self.P
        got, restart = [], []
        for l in range(K):
            i = min(range(P), key=lambda a: (self.f[a], a))
            got.append((i, self.s[i] - 1, self.snap[i], self.tau[i]))
            if l + 1 < K:                                # fetches the unchanged w_j, restarts at once
                self.tau[i], self.snap[i] = self.j, self.w
                self.f[i] = self.f[i] + self._delay(i)
            else:
                last = i
        self.t = self.f[last]
        self._apply(got, K)
        self.tau[last], self.snap[last] = self.j, self.w     # the K-th pusher reads w_{j+1}
        self.f[last] = self.f[last] + self._delay(last)

    def step(self):
        {"ksync": self._step_ksync, "kbatchsync": self._step_kbatchsync,
         "kasync": self._step_kasync, "kbatchasync": self._step_kbatchasync}[self.variant]()

    def run(self, iters):
        for _ in range(iters):
            self.step()
        return self

    # -- results ----------------------------------------------------------------------------
    def trace_arrays(self, K_stride=None):
        tr = self.trace
        J = len(tr["t"])
        Ks = K_stride or (self.P if self.t_interval > 0 else self.K_fixed)
        out = {"t": np.array(tr["t"], np.float64), "K": np.array(tr["K"], np.uint16),
               "worker": np.full((J, Ks), 0xFFFF, np.uint16),
               "stale": np.full((J, Ks), 0xFFFFFFFF, np.uint32),
               "seq": np.full((J, Ks), 0xFFFFFFFF, np.uint32),
               "loss": np.array(tr["loss"], np.float32), "dist2": np.array(tr["dist2"], np.float32),
               "gnorm": np.array(tr["gnorm"], np.float64)}
        for j in range(J):
            k = tr["K"][j]
            out["worker"][j, :k] = tr["worker"][j]
            out["stale"][j, :k] = tr["stale"][j]
            out["seq"][j, :k] = tr["seq"][j]
        return out
