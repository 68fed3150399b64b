#!/usr/bin/env python
"""Benchmark: simulated SGD updates per second on the K-sweep workload.

Workload (per GPU): least squares, n = 65536 x d = 1024 fp32, y = X w* + N(0, 0.1^2), P = 16
workers, m = 32, eta = 0.005, shifted-exponential delays (Delta = 0.5, mu = 1); K-sync and
K-batch-sync for every K = 1..16 (32 simulations), 1024 replicas each.  One step advances all
32 simulations by `--updates-per-step` server updates (default 50, so the default 3 warm-up + 17
timed steps are exactly the workload's 1000 updates).  The 32 simulations are independent and
are enqueued on 32 streams; the step time is taken with CUDA events on a stream that forks to
and joins all of them.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (under torchrun) every rank simulates its own 1024 replicas (global replica ids
rank*1024 ...): weak scaling, no data-path collective.  `--impl reference` times the CPU oracle
on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "simulated SGD updates/sec across replicas"
UNIT = "updates/s"


def algorithmic_bytes_per_update(K, m, d, n_params, async_variant=False):
    """Bytes the method must move per server update: each of the K gradients reads its m rows
    and m targets once (plus its stale snapshot for the asynchronous variants); the update reads
    w_j and writes w_{j+1} once.  Gradients and accumulators stay on chip."""
    per_grad = m * (4 * d + 4) + (4 * n_params if async_variant else 0)
    return K * per_grad + 8 * n_params


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
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
                time.sleep(0.1)
        except Exception as e:  # clocks are evidence, not a dependency of the measurement
            self.reasons.add("nvml_unavailable:%s" % type(e).__name__)

    def finish(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def oracle_sample(wl, data, replicas, updates):
    """The CPU oracle, as it stands, on `replicas` replicas x `updates` updates of each of the
    workload's runs; returns (updates done, seconds, threads used)."""
    from threadpoolctl import threadpool_limits
    from oracle.sim import OracleReplica
    w0 = wl.w0()
    done = 0
    with threadpool_limits(limits=1):
        t0 = time.perf_counter()
        for variant, K in wl.runs:
            for r in range(replicas):
                OracleReplica(model=data["model"], X=data["X"], y=data["y"], w0=w0, P=wl.P, K=K,
                              variant=variant, delay_kind=wl.delay_kind, mu=wl.mu, shift=wl.shift, eta=wl.eta,
                              m=wl.m, seed=wl.seed, replica=r, n_classes=wl.n_classes, hidden=wl.hidden,
                              w_ref=data["w_star"]).run(updates)
                done += updates
        dt = time.perf_counter() - t0
    return done, dt, 1


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    data = wl.make_data()
    reps, ups = 4, 25
    for _ in range(args.warmup):
        oracle_sample(wl, data, 1, 1)
    t0 = time.perf_counter()
    done = 0
    for _ in range(args.steps):
        n, _, cores = oracle_sample(wl, data, reps, ups)
        done += n
    dt = time.perf_counter() - t0
    value = done / dt
    sample = "%d replica x %d updates of each of the %d (variant, K) runs per step" % (reps, ups, len(wl.runs))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "n": wl.n, "d": wl.d, "P": wl.P, "m": wl.m, "runs": len(wl.runs)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_profile_case(args, wl):
    """One small run of another workload (first of its (variant, K) runs), for profiler captures."""
    import torch
    from paper_2003_10579_b200.binding import Simulation
    wl = wl.scaled(n=args.profile_n)
    data = wl.make_data()
    dev = {"model": data["model"], "X": torch.from_numpy(data["X"]).cuda(), "y": torch.from_numpy(data["y"]).cuda(),
           "n_classes": data["n_classes"], "hidden": data["hidden"]}
    variant, K = wl.runs[0]
    R = args.profile_replicas or wl.replicas
    sim = Simulation(dev, P=wl.P, K=K, variant=variant, delay_kind=wl.delay_kind, mu=wl.mu, shift=wl.shift, eta=wl.eta,
                     m=wl.m, seed=wl.seed, n_replicas=R)
    if wl.t_interval > 0:
        sim.set_adasync(wl.K0, args.profile_interval or wl.t_interval)
    w0 = wl.w0()
    if np.any(w0):
        sim.set_params(torch.from_numpy(w0).cuda())
    J = args.profile_updates
    sim.reserve(J)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    sim.run(J)
    e1.record()
    torch.cuda.synchronize()
    tr = sim.trace()
    print(json.dumps({"profile_case": args.profile_case, "workload": wl.name, "variant": variant, "K": K, "n": args.profile_n,
                      "replicas": R, "updates": J, "device_ms": e0.elapsed_time(e1), "last_loss": float(tr["loss"][0, -1])}))
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
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--profile-case", type=int, default=0, choices=[0, 3, 4, 5],
                    help="instead of the benchmark, run workload 3, 4 or 5 once at --profile-n samples for "
                         "--profile-updates updates (a capture-sized case for ncu) and print its device time")
    ap.add_argument("--profile-n", type=int, default=65536)
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
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                # DRAM bytes of the step: ncu small-case capture of this kernel (profiles/), dram read+write =
                # 0.678 x algorithmic bytes, scaled by the rows gathered
                "traffic": 0.678 * step_bytes, "traffic_scaled_from": "profiles/linear1_kernel_small_case_counters.txt",
                # the same traffic as a rate: algorithmic bytes count every gathered row, but 23 % of the sectors hit
                # in L2, so `frac` can pass 1 while the DRAM itself runs at this fraction of the measured copy peak
                "dram_frac": 0.678 * achieved / peak,
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
            "config": {"workload": wl.name, "n": wl.n, "d": wl.d, "P": wl.P, "m": wl.m, "runs": len(wl.runs),
                       "replicas_per_run_per_gpu": R, "updates_per_step": U,
                       "l2": "input X is 256 MiB, larger than L2; rows are gathered at random"},
            "roofline": roofline, "clocks": clocks,
            "gpu_launches": 2 * len(sims) * args.steps}

    if not args.no_e2e:
        # the public one-shot call on pinned host buffers: one step's work (all 32 runs, U updates from
        # w_0) including the copy of the data set to the device and of the traces back, every step
        for sim in sims:
            sim.close()
        sims = []
        torch.cuda.empty_cache()
        Xp = torch.from_numpy(data["X"]).pin_memory()
        yp = torch.from_numpy(data["y"]).pin_memory()
        host = {"model": "lsq", "X": Xp.numpy(), "y": yp.numpy()}
        kw = dict(P=wl.P, delay_kind=wl.delay_kind, mu=wl.mu, shift=wl.shift, eta=wl.eta, m=wl.m, seed=wl.seed,
                  n_replicas=R, replica_base=rank * R, iters=U, want=("t", "loss"))
        e2e_steps = max(1, min(args.steps, 10))
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
        reps, ups = 8, 150
        done, dt, cores = oracle_sample(wl, data, reps, ups)
        line["cpu_baseline"] = {"value": done / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": "%d replicas x %d updates of each of the %d (variant, K) runs (%.1f s)"
                                          % (reps, ups, len(wl.runs), dt)}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
