#!/usr/bin/env python
"""Benchmark: simulated SGD updates per second.

Headline workload (per GPU): the K-sweep - least squares, n = 65536 x d = 1024 fp32,
y = X w* + N(0, 0.1^2), P = 16 workers, m = 32, eta = 0.005, shifted-exponential delays
(Delta = 0.5, mu = 1); K-sync and K-batch-sync for every K = 1..16 (32 simulations), 1024 replicas
each.  One step advances all 32 simulations by `--updates-per-step` server updates (default 50, so
the default 3 warm-up + 17 timed steps are exactly the workload's 1000 updates).  The 32
simulations are independent and are enqueued on 32 streams; the step time is taken with CUDA
events on a stream that forks to and joins all of them.

At one GPU the same JSON line also carries a `workloads` list: the other four workloads (small
K-sync least squares, asynchronous logistic regression, growing-K softmax regression,
K-batch-async MLP) and the clock-only arrival process, each timed on the device at its full size
with its own algorithmic-bytes roofline, and the CPU oracle timed on one core and on all cores.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (under torchrun) every rank simulates its own 1024 replicas (global replica ids
rank*1024 ...): weak scaling, no data-path collective.  `--impl reference` times the CPU oracle
on a bounded sample of the headline workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import re
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "simulated SGD updates/sec across replicas"
UNIT = "updates/s"
KSWEEP_PROFILE = "profiles/linear1_kernel_ksweep_launch_shape_counters.txt"


def n_params_of(wl):
    if wl.model == "softmax":
        return wl.n_classes * wl.d
    if wl.model == "mlp2":
        return wl.d * wl.hidden + wl.hidden + wl.hidden * wl.n_classes + wl.n_classes
    return wl.d


def algorithmic_bytes_per_update(K, m, d, n_params, async_variant=False):
    """Bytes the method must move per server update: each of the K gradients reads its m rows
    and m targets once (plus its stale snapshot for the asynchronous variants); the update reads
    w_j and writes w_{j+1} once.  Gradients and accumulators stay on chip."""
    per_grad = m * (4 * d + 4) + (4 * n_params if async_variant else 0)
    return K * per_grad + 8 * n_params


def measured_traffic_ratio():
    """DRAM bytes / algorithmic bytes of one linear1_kernel launch in the benchmark's launch shape, as the
    committed ncu summary states it (a line `dram_over_algorithmic = X`); None if the file does not say."""
    try:
        text = open(os.path.join(ROOT, KSWEEP_PROFILE)).read()
        return float(re.search(r"dram_over_algorithmic\s*=\s*([0-9.]+)", text).group(1))
    except Exception:
        return None


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index, period=0.1):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz, self.period = index, [], set(), None, period
        self._stop_evt = threading.Event()

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40,
                     "sw_thermal_slowdown": 0x20, "hw_power_brake": 0x80, "sync_boost": 0x10,
                     "applications_clocks": 0x2}
            while not self._stop_evt.is_set():
                self.samples.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
                self.reasons |= {k for k, b in names.items() if mask & b}
                time.sleep(self.period)
        except Exception as e:  # clocks are evidence, not a dependency of the measurement
            self.reasons.add("nvml_unavailable:%s" % type(e).__name__)

    def finish(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ---- the CPU oracle as a timed baseline -------------------------------------------------------------
def oracle_sample(wl, data, replica_ids, updates):
    """The CPU oracle, as it stands, on the given replicas x `updates` updates of each of the
    workload's runs, on one thread; returns (updates done, seconds)."""
    from threadpoolctl import threadpool_limits
    from oracle.sim import OracleReplica
    w0 = wl.w0()
    done = 0
    with threadpool_limits(limits=1):
        t0 = time.perf_counter()
        for variant, K in wl.runs:
            for r in replica_ids:
                OracleReplica(model=data["model"], X=data["X"], y=data["y"], w0=w0, P=wl.P, K=K,
                              variant=variant, delay_kind=wl.delay_kind, mu=wl.mu, shift=wl.shift, eta=wl.eta,
                              m=wl.m, seed=wl.seed, replica=r, n_classes=wl.n_classes, hidden=wl.hidden,
                              w_ref=data["w_star"]).run(updates)
                done += updates
        dt = time.perf_counter() - t0
    return done, dt


def oracle_workload(wl, data, variant, K, replica_ids, updates, t_interval=None):
    """The CPU oracle on one thread on one (variant, K) run of a workload: `updates` updates of each given replica.
    Returns the `cpu_oracle` object of a `workloads` entry."""
    from threadpoolctl import threadpool_limits
    from oracle.sim import OracleReplica
    ti = wl.t_interval if t_interval is None else t_interval
    w0 = wl.w0()
    with threadpool_limits(limits=1):
        t0 = time.perf_counter()
        for r in replica_ids:
            OracleReplica(model=data["model"], X=data["X"], y=data["y"], w0=w0, P=wl.P, K=K, variant=variant,
                          delay_kind=wl.delay_kind, mu=wl.mu, shift=wl.shift, eta=wl.eta, m=wl.m, seed=wl.seed, replica=r,
                          n_classes=wl.n_classes, hidden=wl.hidden, K0=wl.K0 if ti > 0 else 0, t_interval=ti).run(updates)
        dt = time.perf_counter() - t0
    n = len(replica_ids) * updates
    return {"value": n / dt, "unit": "updates/s", "cores": 1, "kind": "oracle",
            "sample": "%d replica(s) x %d updates of this run%s (%.1f s)" % (
                len(replica_ids), updates, "" if ti == wl.t_interval else ", K doubling every %g time units" % ti, dt)}


def _oracle_worker(index, reps, updates, ready, go, out):
    """One process of the all-cores baseline: makes its own copy of the data, waits for the common start,
    follows replicas [index*reps, (index+1)*reps) of every run."""
    from paper_2003_10579_b200 import inputs
    wl = inputs.WORKLOADS[2]
    data = wl.make_data()
    oracle_sample(wl, data, [index * reps], 1)      # imports, the C core, numpy's first call
    ready.put(index)
    go.wait()
    done, dt = oracle_sample(wl, data, range(index * reps, (index + 1) * reps), updates)
    out.put((index, done, dt))


def oracle_all_cores(reps, updates, max_procs=32):
    """N processes over disjoint replica ranges (the replicas are independent); N = the host's cores, at most
    max_procs.  Returns (updates done, wall seconds of the common region, N).  The processes are spawned, not
    forked: a child forked after the first CUDA call cannot be trusted."""
    import multiprocessing as mp
    ctx = mp.get_context("spawn")
    n = max(1, min(os.cpu_count() or 1, max_procs))
    ready, out, go = ctx.Queue(), ctx.Queue(), ctx.Event()
    procs = [ctx.Process(target=_oracle_worker, args=(i, reps, updates, ready, go, out), daemon=True) for i in range(n)]
    for p in procs:
        p.start()
    for _ in procs:
        ready.get(timeout=600)
    t0 = time.perf_counter()
    go.set()
    done = 0
    for _ in procs:
        done += out.get(timeout=900)[1]
    dt = time.perf_counter() - t0
    for p in procs:
        p.join(timeout=30)
    return done, dt, n


def headline_config(wl, R, U):
    """The `config` object of the headline workload: the same for both arms."""
    return {"workload": wl.name, "n": wl.n, "d": wl.d, "P": wl.P, "m": wl.m, "runs": len(wl.runs),
            "replicas_per_run_per_gpu": R, "updates_per_step": U,
            "l2": "input X is 256 MiB, larger than L2; rows are gathered at random"}


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    data = wl.make_data()
    reps, ups = 4, 25
    for _ in range(args.warmup):
        oracle_sample(wl, data, [0], 1)
    t0 = time.perf_counter()
    done = 0
    for _ in range(args.steps):
        done += oracle_sample(wl, data, range(reps), ups)[0]
    dt = time.perf_counter() - t0
    value = done / dt
    sample = "%d replica x %d updates of each of the %d (variant, K) runs per step" % (reps, ups, len(wl.runs))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": headline_config(wl, args.replicas or wl.replicas, args.updates_per_step),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ---- one simulation of another workload, timed on the device ---------------------------------------
def device_data(data):
    import torch
    return {"model": data["model"], "X": torch.from_numpy(data["X"]).cuda(), "y": torch.from_numpy(data["y"]).cuda(),
            "n_classes": data["n_classes"], "hidden": data["hidden"]}


def make_sim(wl, dev, variant, K, R, interval=None, w_ref=None):
    import torch
    from paper_2003_10579_b200.binding import Simulation
    sim = Simulation(dev, P=wl.P, K=K, variant=variant, delay_kind=wl.delay_kind, mu=wl.mu, shift=wl.shift, eta=wl.eta,
                     m=wl.m, seed=wl.seed, n_replicas=R, w_ref=w_ref)
    ti = wl.t_interval if interval is None else interval
    if ti > 0:
        sim.set_adasync(wl.K0, ti)
    if dev is not None:
        w0 = wl.w0()
        if np.any(w0):
            sim.set_params(torch.from_numpy(w0).cuda())
    return sim


def timed_run(sim, warm_steps, warm_updates, updates, local):
    """`warm_steps` untimed runs of `warm_updates` updates, then `updates` updates between two CUDA events on
    the current stream (the stream the handle enqueues on); returns (ms, clocks)."""
    import torch
    sim.reserve(warm_steps * warm_updates + updates)
    for _ in range(warm_steps):
        sim.run(warm_updates)
    torch.cuda.synchronize()
    sampler = ClockSampler(local, period=0.02)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    sim.run(updates)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1), sampler.finish()


def entry(name, wl, variant, K_label, R, updates, ms, clocks, trace_K, peak, note=None, bound="hbm"):
    """One line of the `workloads` list.  Algorithmic bytes are summed over the K actually used by every
    (replica, update) of the timed range (the growing-K schedule changes K during the run)."""
    asyn = variant in ("kasync", "kbatchasync")
    npar = n_params_of(wl)
    k_sum = float(np.asarray(trace_K, np.float64).sum())
    n_upd = R * updates
    total = k_sum * (wl.m * (4 * wl.d + 4) + (4 * npar if asyn else 0)) + n_upd * 8 * npar
    gbs = total / (ms * 1e-3) / 1e9
    e = {"workload": name, "model": wl.model, "variant": variant, "K": K_label, "replicas": R, "updates": updates,
         "device_ms": ms, "value": n_upd / (ms * 1e-3), "unit": UNIT, "us_per_update_step": 1e3 * ms / updates,
         "roofline": {"bound": bound, "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                      "algorithmic_bytes": total},
         "clocks": clocks}
    if note:
        e["note"] = note
    return e


def timed_eval(sim, local, reps=3):
    """sim_eval_loss on the handle's current parameters: one warm-up call, then `reps` calls between two CUDA events."""
    import torch
    sim.eval_loss()
    torch.cuda.synchronize()
    sampler = ClockSampler(local, period=0.02)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        out = sim.eval_loss(to_numpy=False)
    e1.record()
    torch.cuda.synchronize()
    assert bool(torch.isfinite(out).all())
    return e0.elapsed_time(e1) / reps, sampler.finish()


def run_other_workloads(inputs, peak, peaks, local, data2, with_oracle=True):
    import torch
    out = []
    fp32_peak = 148 * 128 * 2 * 1.965e9 / 1e12       # TFLOP/s: 148 SMs x 128 FMA lanes x 2 flop at the 1965 MHz maximum clock

    # -- full-data risk of all replicas (Eq. 1), K-sweep shape: one fp32 product X W^T over 1024 replicas
    wl = inputs.WORKLOADS[2]
    dev = device_data(data2)
    sim = make_sim(wl, dev, "ksync", 8, wl.replicas)
    sim.run(5)
    ms, clocks = timed_eval(sim, local)
    tf = 2.0 * wl.n * wl.d * wl.replicas / (ms * 1e-3) / 1e12
    out.append({"workload": "full_data_risk_" + wl.name, "model": wl.model, "replicas": wl.replicas, "device_ms": ms,
                "value": wl.replicas / (ms * 1e-3), "unit": "replica-evaluations/s", "clocks": clocks,
                "roofline": {"bound": "alu", "achieved": tf, "peak": fp32_peak, "unit": "TFLOP/s", "frac": tf / fp32_peak,
                             "note": "fp32 FMA product on the CUDA cores (the integer K of the loss-driven rule needs fp32 logits); "
                                     "peak = 148 SMs x 128 lanes x 2 flop x 1965 MHz"}})
    sim.close()
    del dev

    def last_K(sim, updates):
        tr = sim.trace(to_numpy=False)
        assert bool(torch.isfinite(tr["loss"][:, -1]).all())
        return tr["K"][:, -updates:].to(torch.int32).cpu().numpy()

    # -- workload 1: small K-sync least squares; latency-bound by construction (1 MiB data set, 200 serial updates)
    wl = inputs.WORKLOADS[1]
    data = wl.make_data()
    dev = device_data(data)
    for R in (65536, wl.replicas):       # the large launch first: the 64-replica run lasts 1.5 ms and would otherwise meet idle clocks
        sim = make_sim(wl, dev, "ksync", 2, R)
        ms, clocks = timed_run(sim, 3, wl.updates, wl.updates, local)
        out.append(entry("%s%s" % (wl.name, "" if R == wl.replicas else "_65536_replicas"), wl, "ksync", 2, R, wl.updates, ms, clocks,
                         last_K(sim, wl.updates), peak,
                         note="data set of 1 MiB lives in L2 and each replica's 200 updates are serial: no HBM roofline applies; "
                              "read updates/s and us_per_update_step" if R == wl.replicas else
                              "same workload with 65536 replicas: the launch fills the GPU"))
        sim.close()
    if with_oracle:      # the whole workload: all 64 replicas x 200 updates
        out[-1]["cpu_oracle"] = oracle_workload(wl, data, "ksync", 2, range(wl.replicas), wl.updates)
    del dev, data

    # -- workload 3: asynchronous variants with stale snapshots, logistic regression, K = 4
    wl = inputs.WORKLOADS[3]
    data = wl.make_data()
    dev = device_data(data)
    for variant in ("kasync", "kbatchasync"):
        sim = make_sim(wl, dev, variant, 4, wl.replicas)
        ms, clocks = timed_run(sim, 3, 20, 200, local)
        out.append(entry(wl.name, wl, variant, 4, wl.replicas, 200, ms, clocks, last_K(sim, 200), peak))
        sim.close()
        if with_oracle:
            out[-1]["cpu_oracle"] = oracle_workload(wl, data, variant, 4, range(2), 100)
    del dev, data
    torch.cuda.empty_cache()

    # -- workload 4: K-sync with K doubling 1 -> 8, softmax regression, the whole run (K depends on the clock)
    wl = inputs.WORKLOADS[4]
    data = wl.make_data()
    dev = device_data(data)
    warm = make_sim(wl, dev, "ksync", 1, wl.replicas, interval=10.0)     # a short interval: the warm-up meets every K
    warm.run(20); warm.run(20); warm.run(20)
    warm.close()
    sim = make_sim(wl, dev, "ksync", 1, wl.replicas)
    ms, clocks = timed_run(sim, 0, 0, wl.updates, local)
    Ks = last_K(sim, wl.updates)
    e = entry(wl.name, wl, "ksync", "1,2,4,8 (doubling every %g time units)" % wl.t_interval, wl.replicas, wl.updates, ms,
              clocks, Ks, peak,
              note="bound by fp32 FMA issue, not by HBM: 2 passes x 10 classes = 20 FMA per 4-byte feature (10 flop/B), and 128 "
                   "replicas occupy 128 of 148 SMs; `alu` gives the same run against the fp32 FMA peak of the whole GPU")
    tf = 2.0 * 20 * wl.d * wl.m * float(Ks.astype(np.float64).sum()) / (ms * 1e-3) / 1e12
    e["alu"] = {"bound": "alu", "achieved": tf, "peak": fp32_peak, "unit": "TFLOP/s", "frac": tf / fp32_peak}
    out.append(e)
    sim.close()
    if with_oracle:      # a shorter interval for the timing run only, so that 300 updates meet K = 1, 2, 4 and 8
        e["cpu_oracle"] = oracle_workload(wl, data, "ksync", 1, range(2), 300, t_interval=80.0)
    del dev, data
    torch.cuda.empty_cache()

    # -- workload 5: K-batch-async MLP 3072-512-10 (bf16 tensor-core products over d)
    wl = inputs.WORKLOADS[5]
    data = wl.make_data()
    dev = device_data(data)
    sim = make_sim(wl, dev, "kbatchasync", 4, wl.replicas)
    ms, clocks = timed_run(sim, 3, 10, 180, local)
    e = entry(wl.name, wl, "kbatchasync", 4, wl.replicas, 180, ms, clocks, last_K(sim, 180), peak,
              note="bytes counted for fp32 operands; the kernels read bf16 copies of X and W1, so DRAM traffic is lower")
    flops = 180 * wl.replicas * 4 * wl.m * (4 * wl.d * wl.hidden)      # forward and dW1 products, 2 flop per multiply-add
    e["tensor_tflops"] = flops / (ms * 1e-3) / 1e12
    if with_oracle:
        e["cpu_oracle"] = oracle_workload(wl, data, "kbatchasync", 4, range(1), 20)
    out.append(e)
    ms, clocks = timed_eval(sim, local, reps=2)
    tf = 2.0 * wl.n * wl.d * wl.hidden * wl.replicas / (ms * 1e-3) / 1e12
    tpeak = float(peaks.get("bf16_tflops", 1590.0))
    out.append({"workload": "full_data_risk_" + wl.name, "model": wl.model, "replicas": wl.replicas, "device_ms": ms,
                "value": wl.replicas / (ms * 1e-3), "unit": "replica-evaluations/s", "clocks": clocks,
                "roofline": {"bound": "tensor", "achieved": tf, "peak": tpeak, "unit": "TFLOP/s", "frac": tf / tpeak,
                             "note": "forward-only pass of the tcgen05 kernel over all 262144 rows for each of the 64 replicas"}})
    sim.close()
    del dev, data
    torch.cuda.empty_cache()

    # -- the arrival process alone (clock-only mode, the runtime results of Section 3): replicas x updates per second
    wl = inputs.WORKLOADS[2]
    for variant, K in (("ksync", 8), ("kbatchasync", 8)):
        R, J = 262144, 100
        sim = make_sim(wl, None, variant, K, R)
        ms, clocks = timed_run(sim, 3, 10, J, local)
        out.append({"workload": "clock_only", "model": "none", "variant": variant, "K": K, "P": wl.P, "replicas": R, "updates": J,
                    "device_ms": ms, "value": R * J / (ms * 1e-3), "unit": "replica-updates/s", "clocks": clocks,
                    "roofline": {"bound": "alu", "note": "fp64 latency chains of one warp per replica; no memory roofline applies"}})
        sim.close()
    return out


def run_profile_case(args, wl):
    """One small run of a workload (run number --profile-run of its (variant, K) list), for profiler captures."""
    import torch
    wl = wl.scaled(n=args.profile_n) if args.profile_n else wl
    data = wl.make_data()
    dev = device_data(data)
    variant, K = wl.runs[args.profile_run]
    if args.profile_variant:
        variant, K = args.profile_variant, args.profile_K
    R = args.profile_replicas or wl.replicas
    interval = args.profile_interval or None
    if args.profile_variant and wl.t_interval > 0:
        interval = 0.0                   # a given (variant, K) is run as it is, without the AdaSync rule
    sim = make_sim(wl, dev, variant, K, R, interval=interval)
    J = args.profile_updates
    sim.reserve(J)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    sim.run(J)
    e1.record()
    torch.cuda.synchronize()
    tr = sim.trace()
    asyn = variant in ("kasync", "kbatchasync")
    total = float(tr["K"].astype(np.float64).sum()) * (wl.m * (4 * wl.d + 4) + (4 * n_params_of(wl) if asyn else 0)) + R * J * 8 * n_params_of(wl)
    print(json.dumps({"profile_case": args.profile_case, "workload": wl.name, "variant": variant, "K": K, "n": wl.n,
                      "replicas": R, "updates": J, "device_ms": e0.elapsed_time(e1), "algorithmic_bytes": total,
                      "last_loss": float(tr["loss"][0, -1])}))
    sim.close()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=17)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--updates-per-step", type=int, default=50)
    ap.add_argument("--replicas", type=int, default=0, help="replicas per simulation (default: the workload's 1024)")
    ap.add_argument("--serial", action="store_true", help="one stream for all simulations (for profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-workloads", action="store_true", help="skip the `workloads` list (the other four workloads)")
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--profile-case", type=int, default=0, choices=[0, 1, 2, 3, 4, 5],
                    help="instead of the benchmark, run one simulation of that workload at --profile-n samples for "
                         "--profile-updates updates (a capture-sized case for ncu) and print its device time")
    ap.add_argument("--profile-n", type=int, default=65536, help="samples of the profile case (0: the workload's)")
    ap.add_argument("--profile-run", type=int, default=0, help="which of the workload's (variant, K) runs")
    ap.add_argument("--profile-variant", default="", choices=["", "ksync", "kbatchsync", "kasync", "kbatchasync"],
                    help="run the profile case with this variant and --profile-K instead of one of the workload's runs")
    ap.add_argument("--profile-K", type=int, default=4)
    ap.add_argument("--profile-updates", type=int, default=3)
    ap.add_argument("--profile-replicas", type=int, default=0)
    ap.add_argument("--profile-interval", type=float, default=0.0, help="AdaSync interval of the profile case (default: the workload's)")
    args = ap.parse_args()

    from paper_2003_10579_b200 import inputs
    if args.profile_case:
        return run_profile_case(args, inputs.WORKLOADS[args.profile_case])
    wl = inputs.WORKLOADS[2]
    if args.impl == "reference":
        return run_reference(args, wl)

    import torch
    import torch.distributed as dist
    from paper_2003_10579_b200.binding import Simulation, sweep_host
    from paper_2003_10579_b200.sharding import replica_block

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    R = args.replicas or wl.replicas
    U = args.updates_per_step
    total_steps = args.steps + args.warmup
    data = wl.make_data()
    dev = {"model": "lsq", "X": torch.from_numpy(data["X"]).cuda(), "y": torch.from_numpy(data["y"]).cuda()}
    w_ref = torch.from_numpy(data["w_star"]).cuda()

    main_stream = torch.cuda.current_stream()
    sims, streams = [], []
    for variant, K in wl.runs:
        st = main_stream if args.serial else torch.cuda.Stream()
        sim = Simulation(dev, P=wl.P, K=K, variant=variant, delay_kind=wl.delay_kind, mu=wl.mu, shift=wl.shift,
                         eta=wl.eta, m=wl.m, seed=wl.seed, n_replicas=R, replica_base=replica_block(rank, world, R)[0], w_ref=w_ref,
                         stream=None if args.serial else st)
        sim.reserve(total_steps * U)
        if args.stages:
            sim.set_tuning(args.stages)
        sims.append(sim)
        streams.append(st)
    torch.cuda.synchronize()

    def step():
        if args.serial:
            for sim in sims:
                sim.run(U)
            return
        fork = torch.cuda.Event()
        fork.record(main_stream)
        for sim, st in zip(sims, streams):
            st.wait_event(fork)
            sim.run(U)
            done = torch.cuda.Event()
            done.record(st)
            main_stream.wait_event(done)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(main_stream)
    for _ in range(args.steps):
        step()
    e1.record(main_stream)
    barrier()
    clocks = sampler.finish()
    ms = e0.elapsed_time(e1)
    if world > 1:
        t = torch.tensor([ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())

    updates_per_step_rank = len(wl.runs) * R * U
    value = world * updates_per_step_rank * args.steps / (ms * 1e-3)
    step_bytes = sum(algorithmic_bytes_per_update(K, wl.m, wl.d, wl.d) for _, K in wl.runs) * R * U
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    peak = float(peaks.get("hbm_gbs", 6650.0))
    achieved = step_bytes * args.steps / (ms * 1e-3) / 1e9
    ratio = measured_traffic_ratio()
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                # DRAM bytes of one step: dram read + write of an ncu capture of this kernel in the benchmark's launch
                # shape (1024 replicas, six one-warp CTAs per SM) over its algorithmic bytes, times the step's algorithmic
                # bytes (traffic grows with the rows gathered); null if the committed summary does not state the ratio
                "traffic": None if ratio is None else ratio * step_bytes,
                "traffic_scaled_from": KSWEEP_PROFILE if ratio is not None else None,
                # the same traffic as a rate: algorithmic bytes count every gathered row, but part of the sectors hit
                # in L2, so `frac` can pass 1 while the DRAM itself runs at this fraction of the measured copy peak
                "dram_frac": None if ratio is None else ratio * achieved / peak,
                "peak_source": "measured" if peaks else "fallback",
                "kernel": "linear1_kernel (32 concurrent launches per step; summed algorithmic bytes over the step's device time)"}

    # a simulation that ran must have produced a finite trace (also surfaces device-side errors)
    J, _ = sims[0].trace_size()
    assert J == total_steps * U
    last = sims[-1].trace(to_numpy=False)["loss"][:, -1]
    assert bool(torch.isfinite(last).all())

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": headline_config(wl, R, U),
            "roofline": roofline, "clocks": clocks,
            "gpu_launches": 2 * len(sims) * args.steps}
    for sim in sims:
        sim.close()
    sims = []
    del dev
    torch.cuda.empty_cache()

    if world == 1 and not args.no_workloads:
        line["workloads"] = run_other_workloads(inputs, peak, peaks, local, data, with_oracle=not args.no_cpu_baseline)

    if not args.no_e2e:
        # the public one-shot call on pinned host buffers: one step's work (all 32 runs, U updates from
        # w_0) including the copy of the data set to the device and of the traces back, every step
        Xp = torch.from_numpy(data["X"]).pin_memory()
        yp = torch.from_numpy(data["y"]).pin_memory()
        host = {"model": "lsq", "X": Xp.numpy(), "y": yp.numpy()}
        kw = dict(P=wl.P, delay_kind=wl.delay_kind, mu=wl.mu, shift=wl.shift, eta=wl.eta, m=wl.m, seed=wl.seed,
                  n_replicas=R, replica_base=rank * R, iters=U, want=("t", "loss"))
        e2e_steps = max(1, min(args.steps, 10))
        shape = (len(wl.runs), R, U)         # the traces land in pinned memory too
        kw["out"] = {"t": torch.empty(shape, dtype=torch.float64).pin_memory().numpy(),
                     "loss": torch.empty(shape, dtype=torch.float32).pin_memory().numpy()}
        sweep_host(host, wl.runs, **kw)
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            out = sweep_host(host, wl.runs, **kw)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        if world > 1:
            tt = torch.tensor([dt], device="cuda")
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            dt = float(tt.item())
        assert np.isfinite(out["loss"]).all()
        line["e2e"] = {"value": world * e2e_steps * len(wl.runs) * R * U / dt, "unit": UNIT,
                       "h2d_bytes_per_step": Xp.numel() * 4 + yp.numel() * 4,
                       "d2h_bytes_per_step": len(wl.runs) * R * U * 12, "steps": e2e_steps,
                       "note": "sim_sweep_host per step: data set host->device, 32 runs x %d updates, "
                               "clocks and losses device->host; host wall clock, max over ranks" % U}

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        reps, ups = 4, 100
        done1, dt1 = oracle_sample(wl, data, range(reps), ups)
        doneN, dtN, cores = oracle_all_cores(2, ups)
        line["cpu_baseline"] = {"value": doneN / dtN, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": "%d processes x 2 replicas x %d updates of each of the %d (variant, K) runs "
                                          "(%.1f s wall)" % (cores, ups, len(wl.runs), dtN),
                                "one_core": {"value": done1 / dt1, "unit": UNIT, "cores": 1,
                                             "sample": "%d replicas x %d updates of each of the %d (variant, K) runs (%.1f s)"
                                                       % (reps, ups, len(wl.runs), dt1)}}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
