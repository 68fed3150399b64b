"""ORACLE (test infrastructure, CPU only): ctypes access to ``sched_core.c``.

The C file holds the integer / fp64 side of the simulation (Philox4x32-10, the deterministic
``-ln(u)``, delays, minibatch indices and a bulk arrival-process routine).  It is compiled here
with gcc on first use.  Nothing in this package is imported by the CUDA library or its binding.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sched_core.c")
_LIB = os.path.join(_HERE, "liboracle_core.so")

VARIANTS = {"ksync": 0, "kbatchsync": 1, "kasync": 2, "kbatchasync": 3}
DELAYS = {"exp": 0, "shifted_exp": 1, "pareto2": 2}


def build(force: bool = False) -> str:
    """Compile the C core (contraction off: each fp64 operation is the IEEE one written)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fvisibility=hidden", "-shared",
             "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [("variant", C.c_int32), ("P", C.c_int32), ("K", C.c_int32), ("K0", C.c_int32),
                ("t_interval", C.c_double), ("delay_kind", C.c_int32), ("mu", C.c_double),
                ("shift", C.c_double), ("seed", C.c_uint64)]


class _State(C.Structure):
    _fields_ = [("t", C.c_double), ("j", C.c_int64), ("started", C.c_int32),
                ("s", C.POINTER(C.c_uint32)), ("tau", C.POINTER(C.c_uint32)),
                ("f", C.POINTER(C.c_double))]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.ora_philox4x32_10.argtypes = [C.POINTER(C.c_uint32)] * 3
        L.ora_philox4x32_10.restype = None
        L.ora_neg_log_uniform.argtypes = [C.c_uint32, C.c_uint32]
        L.ora_neg_log_uniform.restype = C.c_double
        L.ora_delay.argtypes = [C.c_int, C.c_double, C.c_double, C.c_uint64, C.c_uint32,
                                C.c_uint32, C.c_uint32]
        L.ora_delay.restype = C.c_double
        L.ora_minibatch_indices.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32,
                                            C.c_uint64, C.c_int32, C.POINTER(C.c_uint32)]
        L.ora_minibatch_indices.restype = None
        L.ora_schedule_run.argtypes = [C.POINTER(_Cfg), C.c_uint32, C.POINTER(_State), C.c_int64,
                                       C.c_int32, C.POINTER(C.c_double), C.POINTER(C.c_uint16),
                                       C.POINTER(C.c_uint16), C.POINTER(C.c_uint32),
                                       C.POINTER(C.c_uint32)]
        L.ora_schedule_run.restype = C.c_int
        _lib = L
    return _lib


def philox4x32_10(key, ctr):
    """Four 32-bit words of Philox4x32-10 for key (2 words) and counter (4 words)."""
    k = (C.c_uint32 * 2)(*[int(v) & 0xFFFFFFFF for v in key])
    c = (C.c_uint32 * 4)(*[int(v) & 0xFFFFFFFF for v in ctr])
    o = (C.c_uint32 * 4)()
    lib().ora_philox4x32_10(k, c, o)
    return [int(v) for v in o]


def neg_log_uniform(x0: int, x1: int) -> float:
    return float(lib().ora_neg_log_uniform(int(x0) & 0xFFFFFFFF, int(x1) & 0xFFFFFFFF))


def delay(kind: str, mu: float, shift: float, seed: int, replica: int, worker: int, seq: int) -> float:
    """Compute time of task `seq` of `worker` in `replica`: shift + Exp(rate mu), or for "pareto2"
    a Pareto law of shape 2 (mu must be 2) and scale `shift`."""
    return float(lib().ora_delay(DELAYS[kind], float(mu), float(shift), int(seed), int(replica),
                                 int(worker), int(seq)))


def minibatch_indices(seed: int, replica: int, worker: int, seq: int, n: int, m: int) -> np.ndarray:
    out = np.empty(m, dtype=np.uint32)
    lib().ora_minibatch_indices(int(seed), int(replica), int(worker), int(seq), int(n), int(m),
                                out.ctypes.data_as(C.POINTER(C.c_uint32)))
    return out


class BulkSchedule:
    """Arrival process of many replicas, schedule only (no parameters), resumable.

    run(iters) returns dict(t[R,iters] f64, K[R,iters] u16, worker/stale/seq[R,iters,K_stride]).
    """

    def __init__(self, variant: str, P: int, K: int, delay_kind: str, mu: float, shift: float,
                 seed: int, n_replicas: int, replica_base: int = 0, K0: int = 0,
                 t_interval: float = 0.0):
        self.cfg = _Cfg(VARIANTS[variant], P, K, K0, float(t_interval), DELAYS[delay_kind],
                        float(mu), float(shift), int(seed))
        self.P, self.R, self.base = P, n_replicas, replica_base
        self.K_stride = P if t_interval > 0 else K
        self.s = np.zeros((n_replicas, P), np.uint32)
        self.tau = np.zeros((n_replicas, P), np.uint32)
        self.f = np.zeros((n_replicas, P), np.float64)
        self.t = np.zeros(n_replicas, np.float64)
        self.j = np.zeros(n_replicas, np.int64)
        self.started = np.zeros(n_replicas, np.int32)

    def run(self, iters: int):
        R, Ks = self.R, self.K_stride
        t = np.empty((R, iters), np.float64)
        K = np.empty((R, iters), np.uint16)
        worker = np.empty((R, iters, Ks), np.uint16)
        stale = np.empty((R, iters, Ks), np.uint32)
        seq = np.empty((R, iters, Ks), np.uint32)
        L = lib()
        pu32, pf64, pu16 = C.POINTER(C.c_uint32), C.POINTER(C.c_double), C.POINTER(C.c_uint16)
        for r in range(R):
            st = _State(self.t[r], self.j[r], self.started[r],
                        self.s[r].ctypes.data_as(pu32), self.tau[r].ctypes.data_as(pu32),
                        self.f[r].ctypes.data_as(pf64))
            rc = L.ora_schedule_run(C.byref(self.cfg), self.base + r, C.byref(st), iters, Ks,
                                    t[r].ctypes.data_as(pf64), K[r].ctypes.data_as(pu16),
                                    worker[r].ctypes.data_as(pu16), stale[r].ctypes.data_as(pu32),
                                    seq[r].ctypes.data_as(pu32))
            if rc != 0:
                raise ValueError("ora_schedule_run: bad argument")
            self.t[r], self.j[r], self.started[r] = st.t, st.j, st.started
        return {"t": t, "K": K, "worker": worker, "stale": stale, "seq": seq}
