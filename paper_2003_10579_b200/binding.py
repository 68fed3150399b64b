"""Thin ctypes binding of the C-ABI library (``include/straggler_sim.h``): argument marshalling
only.  torch supplies device memory and streams; every step of the simulation runs in the
library's CUDA kernels.  Importing this module loads ``libstraggler_sim.so`` and raises if it
has not been built - there is no CPU path behind these calls."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libstraggler_sim.so")

VARIANTS = {"ksync": 0, "kbatchsync": 1, "kasync": 2, "kbatchasync": 3}
MODELS = {"none": 0, "lsq": 1, "logistic": 2, "softmax": 3, "mlp2": 4}
DELAYS = {"exp": 0, "shifted_exp": 1, "pareto2": 2}
STATUS = {0: "SIM_OK", 1: "SIM_ERR_ARG", 2: "SIM_ERR_ALLOC", 3: "SIM_ERR_CUDA", 4: "SIM_ERR_TIMEOUT",
          5: "SIM_ERR_STATE", 6: "SIM_ERR_INTERNAL"}

EXPORTS = ["sim_create", "sim_set_params", "sim_set_adasync", "sim_set_adasync_loss", "sim_set_tuning", "sim_reserve", "sim_run",
           "sim_trace_size", "sim_get_trace", "sim_get_params", "sim_eval_loss", "sim_error_curve", "sim_set_eval_every", "sim_risk_trace_size",
           "sim_get_risk_trace", "sim_risk_curve", "sim_risk_envelope", "sim_selftest_wait_timeout", "sim_n_params", "sim_last_error",
           "sim_destroy", "sim_draw_delays", "sim_draw_indices", "sim_simulate_host", "sim_sweep_host", "sim_schedule_noalloc",
           "sim_noalloc_last_error"]


class SimProblem(C.Structure):
    _fields_ = [("model", C.c_int), ("n", C.c_int64), ("d", C.c_int32), ("n_classes", C.c_int32),
                ("hidden", C.c_int32), ("X", C.c_void_p), ("y", C.c_void_p), ("label", C.c_void_p),
                ("w_ref", C.c_void_p)]


class SimDelay(C.Structure):
    _fields_ = [("kind", C.c_int), ("mu", C.c_double), ("shift", C.c_double)]


class SimError(RuntimeError):
    def __init__(self, status, message):
        super().__init__("%s: %s" % (STATUS.get(status, status), message))
        self.status = status


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError("%s is missing: build it with `python -m paper_2003_10579_b200.build` "
                          "(there is no CPU fallback)" % LIB_PATH)
    L = C.CDLL(LIB_PATH)
    vp, i32, i64, u64, dbl = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_double
    L.sim_create.argtypes = [C.POINTER(SimProblem), i32, i32, C.c_int, SimDelay, C.c_float, i32, u64, i32,
                             i64, vp, C.POINTER(vp)]
    L.sim_set_params.argtypes = [vp, vp]
    L.sim_set_adasync.argtypes = [vp, i32, dbl]
    L.sim_set_adasync_loss.argtypes = [vp, i32, dbl]
    L.sim_set_tuning.argtypes = [vp, i32, i32, i32]
    L.sim_reserve.argtypes = [vp, i64]
    L.sim_run.argtypes = [vp, i64]
    L.sim_trace_size.argtypes = [vp, C.POINTER(i64), C.POINTER(i32)]
    L.sim_get_trace.argtypes = [vp] * 8
    L.sim_get_params.argtypes = [vp, vp]
    L.sim_eval_loss.argtypes = [vp, vp]
    L.sim_error_curve.argtypes = [vp, vp, i32, vp, vp]
    L.sim_selftest_wait_timeout.argtypes = [vp]
    L.sim_set_eval_every.argtypes = [vp, i64]
    L.sim_risk_trace_size.argtypes = [vp, C.POINTER(i64)]
    L.sim_get_risk_trace.argtypes = [vp, vp, vp]
    L.sim_risk_curve.argtypes = [vp, vp, i32, C.c_float, vp, vp]
    L.sim_risk_envelope.argtypes = [C.POINTER(vp), i32, vp, i32, C.c_float, vp, vp]
    L.sim_n_params.argtypes = [vp]
    L.sim_n_params.restype = i64
    L.sim_last_error.argtypes = [vp]
    L.sim_last_error.restype = C.c_char_p
    L.sim_destroy.argtypes = [vp]
    L.sim_destroy.restype = None
    L.sim_draw_delays.argtypes = [SimDelay, u64, i64, i32, i32, i32, vp, vp]
    L.sim_draw_indices.argtypes = [u64, i64, i32, i32, i32, i64, i32, vp, vp]
    L.sim_simulate_host.argtypes = [C.POINTER(SimProblem), i32, i32, C.c_int, SimDelay, C.c_float, i32, u64,
                                    i32, i64, vp, i32, dbl, i64] + [vp] * 8
    L.sim_sweep_host.argtypes = [C.POINTER(SimProblem), i32, i32, vp, vp, SimDelay, C.c_float, i32, u64, i32, i64, vp, i64,
                                 vp, vp, vp]
    L.sim_schedule_noalloc.argtypes = [i32, i32, C.c_int, SimDelay, u64, i64, i32, i32, dbl, i64] + [vp] * 6
    L.sim_noalloc_last_error.argtypes = []
    L.sim_noalloc_last_error.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("sim_n_params", "sim_last_error", "sim_destroy", "sim_noalloc_last_error"):
            getattr(L, name).restype = C.c_int
    return L


lib = _load()


def _check(status, handle=None):
    if status != 0:
        msg = lib.sim_last_error(handle)
        raise SimError(status, msg.decode() if msg else "")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    return None if stream is None else C.c_void_p(stream.cuda_stream)


_U16 = getattr(torch, "uint16")
_U32 = getattr(torch, "uint32")


class Simulation:
    """One handle of the library: n_replicas independent parameter servers on the current device.

    data: dict with model, X [n,d] float32 cuda, y (float32 targets or int32 labels) cuda,
    n_classes, hidden; w_ref optional cuda float32.  The tensors are borrowed by the library and
    kept alive by this object."""

    def __init__(self, data, *, P, K, variant, delay_kind, mu, shift=0.0, eta, m, seed, n_replicas,
                 replica_base=0, w_ref=None, stream=None):
        self._h = C.c_void_p()
        model = data["model"] if data is not None else "none"
        prob = SimProblem(MODELS[model], 0, 0, 0, 0, None, None, None, None)
        self._keep = []
        if model != "none":
            X, y = data["X"], data["y"]
            assert X.is_cuda and X.dtype == torch.float32 and X.is_contiguous()
            prob.n, prob.d = X.shape
            prob.n_classes, prob.hidden = int(data.get("n_classes", 1)), int(data.get("hidden", 0))
            prob.X = X.data_ptr()
            if model == "lsq":
                assert y.dtype == torch.float32 and y.is_cuda
                prob.y = y.data_ptr()
            else:
                assert y.dtype == torch.int32 and y.is_cuda
                prob.label = y.data_ptr()
            if w_ref is not None:
                assert w_ref.is_cuda and w_ref.dtype == torch.float32
                prob.w_ref = w_ref.data_ptr()
            self._keep = [X, y, w_ref]
        self.R, self.stream = n_replicas, stream
        self.device = torch.device("cuda", torch.cuda.current_device())
        _check(lib.sim_create(C.byref(prob), P, K, VARIANTS[variant], SimDelay(DELAYS[delay_kind], mu, shift),
                              eta, m, seed, n_replicas, replica_base, _stream_ptr(stream), C.byref(self._h)))

    def set_params(self, w0):
        assert w0.is_cuda and w0.dtype == torch.float32 and w0.numel() == self.n_params
        _check(lib.sim_set_params(self._h, _ptr(w0)), self._h)

    def set_adasync(self, K0, t_interval):
        _check(lib.sim_set_adasync(self._h, K0, t_interval), self._h)

    def set_adasync_loss(self, K0, t_interval):
        """Algorithm 1 as printed: K follows the full-data risk at interval boundaries."""
        _check(lib.sim_set_adasync_loss(self._h, K0, t_interval), self._h)

    def set_tuning(self, stages=0, tile_rows=0, threads=0):
        _check(lib.sim_set_tuning(self._h, stages, tile_rows, threads), self._h)

    def reserve(self, total_updates):
        _check(lib.sim_reserve(self._h, total_updates), self._h)

    def run(self, iters):
        _check(lib.sim_run(self._h, iters), self._h)

    @property
    def n_params(self):
        return int(lib.sim_n_params(self._h))

    def trace_size(self):
        J, Km = C.c_int64(), C.c_int32()
        _check(lib.sim_trace_size(self._h, C.byref(J), C.byref(Km)), self._h)
        return J.value, Km.value

    def trace(self, to_numpy=True):
        J, Km = self.trace_size()
        R, dev = self.R, self.device
        out = {"t": torch.empty((R, J), dtype=torch.float64, device=dev),
               "loss": torch.empty((R, J), dtype=torch.float32, device=dev),
               "dist2": torch.empty((R, J), dtype=torch.float32, device=dev),
               "K": torch.empty((R, J), dtype=_U16, device=dev),
               "worker": torch.empty((R, J, Km), dtype=_U16, device=dev),
               "stale": torch.empty((R, J, Km), dtype=_U32, device=dev),
               "seq": torch.empty((R, J, Km), dtype=_U32, device=dev)}
        _check(lib.sim_get_trace(self._h, *[_ptr(out[k]) for k in ("t", "loss", "dist2", "K", "worker", "stale", "seq")]),
               self._h)
        return {k: v.cpu().numpy() for k, v in out.items()} if to_numpy else out

    def params(self, to_numpy=True):
        w = torch.empty((self.R, self.n_params), dtype=torch.float32, device=self.device)
        _check(lib.sim_get_params(self._h, _ptr(w)), self._h)
        return w.cpu().numpy() if to_numpy else w

    def eval_loss(self, to_numpy=True):
        """Full-data risk F(w_j) of every replica's current parameters."""
        out = torch.empty((self.R,), dtype=torch.float32, device=self.device)
        _check(lib.sim_eval_loss(self._h, _ptr(out)), self._h)
        if self.stream is not None:
            self.stream.synchronize()
        else:
            torch.cuda.synchronize()
        return out.cpu().numpy() if to_numpy else out

    def error_curve(self, grid):
        """Mean minibatch loss over replicas against simulated wall clock at the times in `grid`."""
        g = torch.as_tensor(np.asarray(grid, np.float64)).to(self.device)
        mean = torch.empty((g.numel(),), dtype=torch.float32, device=self.device)
        cnt = torch.empty((g.numel(),), dtype=torch.int32, device=self.device)
        _check(lib.sim_error_curve(self._h, _ptr(g), g.numel(), _ptr(mean), _ptr(cnt)), self._h)
        return mean.cpu().numpy(), cnt.cpu().numpy()

    def set_eval_every(self, every):
        """Record the full-data risk of every replica before the first and after every `every`-th update."""
        _check(lib.sim_set_eval_every(self._h, every), self._h)

    def risk_trace(self, to_numpy=True):
        """(risk [R, E], t [R, E]): entry 0 is F(w_0) at time 0, entry i the risk after i * every updates."""
        E = C.c_int64()
        _check(lib.sim_risk_trace_size(self._h, C.byref(E)), self._h)
        risk = torch.empty((self.R, E.value), dtype=torch.float32, device=self.device)
        t = torch.empty((self.R, E.value), dtype=torch.float64, device=self.device)
        _check(lib.sim_get_risk_trace(self._h, _ptr(risk), _ptr(t)), self._h)
        return (risk.cpu().numpy(), t.cpu().numpy()) if to_numpy else (risk, t)

    def risk_curve(self, grid, f_star=0.0):
        """Mean over replicas of F(w) - f_star against simulated wall clock at the times in `grid`."""
        g = torch.as_tensor(np.asarray(grid, np.float64)).to(self.device)
        mean = torch.empty((g.numel(),), dtype=torch.float32, device=self.device)
        cnt = torch.empty((g.numel(),), dtype=torch.int32, device=self.device)
        _check(lib.sim_risk_curve(self._h, _ptr(g), g.numel(), f_star, _ptr(mean), _ptr(cnt)), self._h)
        return mean.cpu().numpy(), cnt.cpu().numpy()

    def selftest_wait_timeout(self):
        """Diagnostic: makes a bounded device-side wait run out on this handle (it is unusable afterwards)."""
        _check(lib.sim_selftest_wait_timeout(self._h), self._h)

    def close(self):
        if self._h:
            lib.sim_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def risk_envelope(sims, grid, f_star=0.0):
    """Lower envelope over several simulations' risk curves on a common grid: (env [G], best [G])."""
    dev = sims[0].device
    g = torch.as_tensor(np.asarray(grid, np.float64)).to(dev)
    env = torch.empty((g.numel(),), dtype=torch.float32, device=dev)
    best = torch.empty((g.numel(),), dtype=torch.int32, device=dev)
    hs = (C.c_void_p * len(sims))(*[s._h for s in sims])
    st = lib.sim_risk_envelope(hs, len(sims), _ptr(g), g.numel(), f_star, _ptr(env), _ptr(best))
    _check(st)
    return env.cpu().numpy(), best.cpu().numpy()


def draw_delays(delay_kind, mu, shift, seed, replica_base, n_replicas, P, n_seq):
    out = torch.empty((n_replicas, P, n_seq), dtype=torch.float64, device="cuda")
    _check(lib.sim_draw_delays(SimDelay(DELAYS[delay_kind], mu, shift), seed, replica_base, n_replicas, P, n_seq,
                               _ptr(out), _stream_ptr(torch.cuda.current_stream())))
    return out.cpu().numpy()


def draw_indices(seed, replica_base, n_replicas, P, n_seq, n, m):
    out = torch.empty((n_replicas, P, n_seq, m), dtype=_U32, device="cuda")
    _check(lib.sim_draw_indices(seed, replica_base, n_replicas, P, n_seq, n, m, _ptr(out),
                                _stream_ptr(torch.cuda.current_stream())))
    return out.cpu().numpy()


def schedule_noalloc(out, *, P, K, variant, delay_kind, mu, shift=0.0, seed, n_replicas, iters, replica_base=0,
                     K0=0, t_interval=0.0, stream=None):
    """Clock-only simulation through the entry point that allocates nothing: the caller brings
    the five output tensors (`out`: t, K, worker, stale, seq on the device, shaped as in
    Simulation.trace) because the library may not create them.  For callers that cannot call
    cudaMalloc; the worker state sits in a fixed array inside the library, so sizes are capped and
    calls on one device must not overlap."""
    Ks = P if t_interval > 0 else K
    need = {"t": (torch.float64, n_replicas * iters), "K": (_U16, n_replicas * iters),
            "worker": (_U16, n_replicas * iters * Ks), "stale": (_U32, n_replicas * iters * Ks),
            "seq": (_U32, n_replicas * iters * Ks)}
    for k, (dt, count) in need.items():     # the library writes through raw pointers: a wrong buffer would be an out-of-bounds write
        t = out[k]
        if not (t.is_cuda and t.is_contiguous() and t.dtype == dt and t.numel() >= count):
            raise ValueError("schedule_noalloc: out[%r] must be a contiguous CUDA tensor of %s with at least %d elements" % (k, dt, count))
    st = lib.sim_schedule_noalloc(P, K, VARIANTS[variant], SimDelay(DELAYS[delay_kind], mu, shift), seed,
                                  replica_base, n_replicas, K0, t_interval, iters,
                                  *[_ptr(out[k]) for k in ("t", "K", "worker", "stale", "seq")],
                                  _stream_ptr(stream))
    if st != 0:
        raise SimError(st, lib.sim_noalloc_last_error().decode())


def simulate_host(data, *, P, K, variant, delay_kind, mu, shift=0.0, eta, m, seed, n_replicas, iters,
                  replica_base=0, w0=None, w_ref=None, K0=0, t_interval=0.0, want=("t", "loss")):
    """The one-shot call on HOST numpy arrays (copies in, runs, copies the trace back)."""
    model = data["model"] if data is not None else "none"
    prob = SimProblem(MODELS[model], 0, 0, 0, 0, None, None, None, None)
    keep = []

    def hp(a, dt):
        if a is None:
            return None
        a = np.ascontiguousarray(a, dtype=dt)
        keep.append(a)
        return a.ctypes.data

    npar = 0
    if model != "none":
        prob.n, prob.d = data["X"].shape
        prob.n_classes, prob.hidden = int(data.get("n_classes", 1)), int(data.get("hidden", 0))
        prob.X = hp(data["X"], np.float32)
        if model == "lsq":
            prob.y = hp(data["y"], np.float32)
        else:
            prob.label = hp(data["y"], np.int32)
        prob.w_ref = hp(w_ref, np.float32)
        d, Cc, H = prob.d, prob.n_classes, prob.hidden
        npar = {"lsq": d, "logistic": d, "softmax": Cc * d, "mlp2": d * H + H + H * Cc + Cc}[model]
    Ks = P if t_interval > 0 else K
    R, J = n_replicas, iters
    shapes = {"t": ((R, J), np.float64), "loss": ((R, J), np.float32), "dist2": ((R, J), np.float32),
              "K": ((R, J), np.uint16), "worker": ((R, J, Ks), np.uint16), "stale": ((R, J, Ks), np.uint32),
              "seq": ((R, J, Ks), np.uint32), "w": ((R, npar), np.float32)}
    out = {k: np.empty(*shapes[k]) for k in want}
    ptrs = [C.c_void_p(out[k].ctypes.data) if k in out else None
            for k in ("t", "loss", "dist2", "K", "worker", "stale", "seq", "w")]
    w0p = hp(w0, np.float32)
    _check(lib.sim_simulate_host(C.byref(prob), P, K, VARIANTS[variant], SimDelay(DELAYS[delay_kind], mu, shift),
                                 eta, m, seed, n_replicas, replica_base, w0p, K0, t_interval, iters, *ptrs))
    return out


def sweep_host(data, runs, *, P, delay_kind, mu, shift=0.0, eta, m, seed, n_replicas, iters, replica_base=0, w0=None,
               w_ref=None, want=("t", "loss"), out=None):
    """All (variant, K) pairs of `runs` on one HOST data set in one call: the data is copied in once,
    the runs overlap on the device, the traces come back as [n_runs, R, iters] numpy arrays.  `out` may hold
    arrays to write into (for instance views of pinned memory): C-contiguous, of that shape, float64 for "t" and
    float32 for "loss" and "dist2"; missing ones are made here."""
    model = data["model"]
    prob = SimProblem(MODELS[model], 0, 0, 0, 0, None, None, None, None)
    keep = []

    def hp(a, dt):
        if a is None:
            return None
        a = np.ascontiguousarray(a, dtype=dt)
        keep.append(a)
        return a.ctypes.data

    prob.n, prob.d = data["X"].shape
    prob.n_classes, prob.hidden = int(data.get("n_classes", 1)), int(data.get("hidden", 0))
    prob.X = hp(data["X"], np.float32)
    if model == "lsq":
        prob.y = hp(data["y"], np.float32)
    else:
        prob.label = hp(data["y"], np.int32)
    prob.w_ref = hp(w_ref, np.float32)
    variants = np.array([VARIANTS[v] for v, _ in runs], np.int32)
    Ks = np.array([k for _, k in runs], np.int32)
    shape = (len(runs), n_replicas, iters)
    dtypes = {"t": np.float64, "loss": np.float32, "dist2": np.float32}
    given, out = out or {}, {}
    for k in want:
        a = given.get(k)
        if a is None:
            a = np.empty(shape, dtypes[k])
        elif a.shape != shape or a.dtype != dtypes[k] or not a.flags["C_CONTIGUOUS"] or not a.flags["WRITEABLE"]:
            raise ValueError("out[%r] must be a writeable C-contiguous %s array of shape %r" % (k, np.dtype(dtypes[k]).name, shape))
        out[k] = a
    ptrs = [C.c_void_p(out[k].ctypes.data) if k in out else None for k in ("t", "loss", "dist2")]
    _check(lib.sim_sweep_host(C.byref(prob), P, len(runs), C.c_void_p(variants.ctypes.data), C.c_void_p(Ks.ctypes.data),
                              SimDelay(DELAYS[delay_kind], mu, shift), eta, m, seed, n_replicas, replica_base,
                              hp(w0, np.float32), iters, *ptrs))
    return out
