#!/usr/bin/env python
"""Benchmark of the fused SGP step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload resnet50] [--impl ours|reference]

One "step" is one whole SGP iteration (local Nesterov update, PushSum mix, weight mix, de-bias) for
all n simulated nodes.  The default workload is the ResNet-50-sized run: n = 32 nodes, d = 25,557,032
parameters, one-peer exponential graph, Nesterov 0.9, weight decay 1e-4, Z written (24 algorithmic
bytes per node-parameter).  Prints ONE JSON line on rank 0.

With N > 1 every rank runs an independent replica of the same workload on its own GPU (the path has
no exchange step between GPUs); `value` is the sum over ranks divided by the slowest rank's time.
`--impl reference` times the float64 CPU oracle on a bounded column sample instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "node_param_updates_per_sec"
UNIT = "updates/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the fused step kernel, from one ncu capture of the
# same kernel on a column-scaled case (d = 2,000,000), scaled by the units a full launch processes.
NCU_TRAFFIC_BYTES = {
    # 1479.6 MB per launch at d = 2,000,000, x (25,557,032 / 2,000,000)
    "resnet50": 18.907e9,
    # 1990.5 MB per launch at d = 2,000,000, same scaling
    "resnet50_osgp1": 25.436e9,
}


def bytes_per_update(w, write_z=True) -> int:
    """Algorithmic HBM bytes per node-parameter per step (fp32, in place)."""
    b = 4 * (2 + 1)                       # read x, g; write x
    if getattr(w, "optimizer", "sgd") == "adam":
        b += 16                           # read and write both moment arrays
    elif w.momentum != 0.0:
        b += 8                            # read u, write u
    if write_z:
        b += 4
    if w.tau > 0:
        b += 8                            # read + write one ring slot
    return b


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Polls NVML for SM clock and throttle reasons while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._armed = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                if self._armed:
                    self.samples.append(mhz)
                    for k, bit in names.items():
                        if mask & bit:
                            self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def arm(self, on: bool):
        self._armed = on

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=1.0)

    def summary(self):
        s = sorted(self.samples)
        return {"sm_mhz": (s[len(s) // 2] if s else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


def oracle_sample_run(w, sample_cols: int, steps: int, warmup: int):
    """Times the float64 oracle, as it stands, on the first `sample_cols` columns of the workload.
    Returns (seconds per step, BLAS threads)."""
    import numpy as np
    import torch
    from oracle import schedule as osched
    from oracle import sgp as osgp
    from paper_1811_10792_b200 import inputs

    def oracle_P_of_k(w):
        if w.graph == "random":
            return lambda k: osched.mixing_matrix("random", w.n, k, seed=w.seed, max_outdeg=w.max_outdeg,
                                                  num_steps=w.num_steps)
        return lambda k: osched.mixing_matrix(w.graph, w.n, k, peers=w.peers)

    x0 = inputs.initial_x(w, device="cpu", d=sample_cols).numpy().astype(np.float64)
    G = torch.empty((w.n, sample_cols), dtype=torch.float32)
    grads = [inputs.gradient(w, k, G).numpy().astype(np.float64) for k in range(min(4, steps + warmup))]
    P_of_k = oracle_P_of_k(w)
    adam = (lambda k: (k + 1, w.beta1, w.beta2, w.adam_eps)) if w.optimizer == "adam" else (lambda k: None)
    st = osgp.init_state(x0, w.tau)
    for k in range(warmup):
        osgp.sgp_step(st, grads[k % len(grads)], P_of_k(k), w.lr, w.momentum, w.nesterov, w.weight_decay, adam=adam(k))
    t0 = time.perf_counter()
    for k in range(warmup, warmup + steps):
        osgp.sgp_step(st, grads[k % len(grads)], P_of_k(k), w.lr, w.momentum, w.nesterov, w.weight_decay, adam=adam(k))
    dt = (time.perf_counter() - t0) / steps
    threads = 1
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        pass
    return dt, threads


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample_cols = min(w.d, 1 << 18)
    dt, threads = oracle_sample_run(w, sample_cols, args.steps, args.warmup)
    value = w.n * sample_cols / dt
    sample = f"float64 numpy oracle, columns [0, {sample_cols}) of {w.d} ({100.0 * sample_cols / w.d:.2f}%), all {w.n} nodes"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, extra={"sample_cols": sample_cols}),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def max_over_ranks(value: float, device="cpu") -> float:
    """Slowest rank's figure (all-reduce MAX over the default process group; identity for one rank)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, units_per_rank_per_step: int, steps: int, max_ms: float) -> float:
    """Replicas only: every rank processes the same number of units; the job ends with the slowest rank."""
    return world * units_per_rank_per_step * steps / (max_ms * 1e-3)


def workload_config(w, extra=None):
    cfg = {"workload": f"{w.name}: n={w.n} nodes x d={w.d} fp32 parameters, {w.peers}-peer exponential digraph"
                       if w.graph == "exp" else f"{w.name}: n={w.n} x d={w.d}, {w.graph} digraph",
           "n": w.n, "d": w.d, "graph": w.graph, "peers": w.peers, "tau": w.tau, "lr": w.lr, "momentum": w.momentum,
           "nesterov": w.nesterov, "weight_decay": w.weight_decay, "writes_z": True, "optimizer": w.optimizer,
           "l2_policy": ("inputs larger than L2 (arrays of %.2f GB each, streamed once per step)" % (4e-9 * w.n * w.d))
                        if 4 * w.n * w.d > (512 << 20) else "working set comparable to L2: a launch-latency figure"}
    if extra:
        cfg.update(extra)
    return cfg


def run_sweep(args):
    """Scaling sweep (random digraphs, Nesterov, Z written): one JSON line per (n, d) point that fits 150 GB."""
    import torch
    from paper_1811_10792_b200 import binding, inputs
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, peak_kind = measured_peak()
    for n in inputs.SWEEP_N:
        for d in inputs.SWEEP_D:
            if 4 * 4 * n * d > 150e9:
                continue                                    # (256, 1e8): 410 GB for X, M, G, Z
            w = inputs.sweep_workload(n, d)
            X, ld = binding.empty_matrix(n, d, device=dev, pitch_multiple=args.ld_align)
            X.copy_(inputs.initial_x(w, device=dev))
            M, _ = binding.empty_matrix(n, d, device=dev, pitch_multiple=args.ld_align, fill=0.0)
            Z, _ = binding.empty_matrix(n, d, device=dev, pitch_multiple=args.ld_align)
            G, _ = binding.empty_matrix(n, d, device=dev, pitch_multiple=args.ld_align)
            inputs.gradient(w, 0, G)
            Wt = torch.ones(n, device=dev)
            K = w.K
            with binding.Sgp(n, d, binding.graph_desc(w), ld=ld) as h:
                for k in range(max(3, args.warmup)):
                    h.step(X, Wt, M, G, Z, k, w.lr, w.momentum, 0.0, True)
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for k in range(K):
                    h.step(X, Wt, M, G, Z, 3 + k, w.lr, w.momentum, 0.0, True)
                e1.record()
                torch.cuda.synchronize()
                ms = e0.elapsed_time(e1) / K
                launch = {k: h.get_option(k) for k in ("last_variant", "last_grid", "last_tile_cols")}
                graph_ms = None
                if 4 * 4 * n * d < (256 << 20):
                    # launch-bound point: the same K steps captured once in a CUDA graph and replayed
                    side = torch.cuda.Stream()
                    graph = torch.cuda.CUDAGraph()
                    with torch.cuda.stream(side):
                        with torch.cuda.graph(graph, stream=side):
                            for k in range(K):
                                h.step(X, Wt, M, G, Z, k, w.lr, w.momentum, 0.0, True, stream=side)
                    graph.replay()
                    torch.cuda.synchronize()
                    e0.record()
                    for _ in range(10):
                        graph.replay()
                    e1.record()
                    torch.cuda.synchronize()
                    graph_ms = e0.elapsed_time(e1) / (10 * K)
            achieved = 24.0 * n * d / (ms * 1e-3) / 1e9
            print(json.dumps({"metric": METRIC, "value": n * d / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K,
                              "ms_per_step": ms, "graph_replay_ms_per_step": graph_ms, "dtype": "f32",
                              "data": "synthetic",
                              "config": workload_config(w, extra={"row_pitch_floats": ld, **launch}),
                              "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                                           "frac": achieved / peak, "peak_kind": f"of {peak_kind}"}}), flush=True)
            del X, M, Z, G
            torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="resnet50",
                    help="resnet50 | transformer | resnet50_osgp1 | tiny | sweep:<n>:<d>")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--d", type=int, default=0, help="override the parameter count (profiling on a small case)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--option", action="append", default=[], help="key=value passed to sgp_set_option")
    ap.add_argument("--ld-align", type=int, default=256,
                    help="row pitch of every n x d array is rounded up to this many floats (256 = 1 KB rows)")
    ap.add_argument("--sweep", action="store_true", help="run every scaling-sweep point, one JSON line each")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.sweep:
        run_sweep(args)
        return

    from paper_1811_10792_b200 import inputs
    if args.workload.startswith("sweep:"):            # sweep:<n>:<d>  (scaling-sweep point, random digraphs)
        _, sn, sd = args.workload.split(":")
        w = inputs.sweep_workload(int(sn), int(sd))
    else:
        w = inputs.WORKLOADS[args.workload]
    if args.d > 0:
        w = w.scaled(args.d)
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_1811_10792_b200 import binding     # raises if the CUDA library is missing: no fallback

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU path)")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    n, d, K, Wm = w.n, w.d, args.steps, args.warmup
    free_b, _total_b = torch.cuda.mem_get_info()
    arr_bytes = 4 * n * d
    n_state = 3 + (1 if w.tau else 0) + (1 if w.optimizer == "adam" else 0)   # X, M, Z (+ ring, + second moment)
    pool = max(1, min(K, int((free_b * 0.6 - n_state * arr_bytes) // arr_bytes)))
    ld = (d + args.ld_align - 1) // args.ld_align * args.ld_align

    def matrix():
        # n x d view of an n x ld allocation: rows start on 1 KB boundaries when ld is a multiple of 256
        return torch.zeros((n, ld), dtype=torch.float32, device=dev)[:, :d]

    X = matrix()
    X.copy_(inputs.initial_x(w, device=dev))
    adam = w.optimizer == "adam"
    M = matrix() if (w.momentum != 0.0 or adam) else None
    V2 = matrix() if adam else None
    Z = matrix()
    Wt = torch.ones(n, device=dev)
    Gs = []
    for k in range(pool):
        G = matrix()
        inputs.gradient(w, k, G)
        Gs.append(G)
    h = binding.Sgp(n, d, binding.graph_desc(w), tau=w.tau, ld=ld)
    for kv in args.option:
        key, val = kv.split("=")
        h.set_option(key, int(val))

    def step(k):
        if adam:
            h.step_adam(X, Wt, M, V2, Gs[k % pool], Z, k, k + 1, w.lr, w.beta1, w.beta2, w.adam_eps, w.weight_decay)
        else:
            h.step(X, Wt, M, Gs[k % pool], Z, k, w.lr, w.momentum, w.weight_decay, w.nesterov)

    sampler = ClockSampler(local_rank)
    sampler.start()
    for k in range(Wm):
        step(k)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
    launches_before = h.get_option("launches")
    sampler.arm(True)
    for i in range(K):
        evs[i].record()
        step(Wm + i)
    evs[K].record()
    torch.cuda.synchronize()
    sampler.arm(False)
    if world > 1:
        dist.barrier()
    gpu_launches = h.get_option("launches") - launches_before      # step kernels launched inside the timed region
    total_ms = evs[0].elapsed_time(evs[K])
    per_step_ms = [evs[i].elapsed_time(evs[i + 1]) for i in range(K)]
    assert h.device_status() == 0
    max_ms = max_over_ranks(total_ms, dev)
    value = whole_job_value(world, n * d, K, max_ms)

    # ---- end to end through the host-buffer entry point (gradients in, de-biased parameters out)
    e2e = None
    if not args.no_e2e and not adam:
        hG = torch.empty((n, ld), dtype=torch.float32, pin_memory=True)[:, :d]
        hZ = torch.empty((n, ld), dtype=torch.float32, pin_memory=True)[:, :d]
        hG.copy_(Gs[0])
        dG = Gs[0]
        torch.cuda.synchronize()
        e2e_steps = K
        h.step_host(X, Wt, M, hG, hZ, dG, Z, Wm + K, w.lr, w.momentum, w.weight_decay, w.nesterov)   # warm
        if world > 1:
            dist.barrier()
        t0 = time.perf_counter()
        for i in range(e2e_steps):
            h.step_host(X, Wt, M, hG, hZ, dG, Z, Wm + K + 1 + i, w.lr, w.momentum, w.weight_decay, w.nesterov)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        dt_max = max_over_ranks(dt, dev)
        e2e = {"value": whole_job_value(world, n * d, e2e_steps, dt_max * 1e3), "unit": UNIT,
               "h2d_bytes_per_step": arr_bytes, "d2h_bytes_per_step": arr_bytes, "steps": e2e_steps,
               "ms_per_step": dt_max * 1e3 / e2e_steps}
        del hG, hZ
    sampler.stop()

    if rank == 0:
        peak, peak_kind = measured_peak()
        bpu = bytes_per_update(w)
        kern_ms = sum(per_step_ms) / len(per_step_ms)
        achieved = bpu * n * d / (kern_ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "traffic": NCU_TRAFFIC_BYTES.get(w.name), "peak_kind": f"of {peak_kind}",
                    "kernel": "sgp_step (fused update + mix + de-bias)", "algorithmic_bytes_per_launch": bpu * n * d,
                    "kernel_ms": kern_ms, "frac_of_nominal_8TBps": achieved / NOMINAL_HBM_GBS}
        cpu = None
        if not args.no_cpu_baseline and world == 1:          # the CPU oracle is timed in single-GPU runs only
            sample_cols = min(d, 1 << 20)
            dt, threads = oracle_sample_run(w, sample_cols, steps=8, warmup=1)
            cpu = {"value": n * sample_cols / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
                   "sample": f"8 steps of the float64 numpy oracle on columns [0, {sample_cols}) "
                             f"({100.0 * sample_cols / d:.2f}% of d), all {n} nodes; host has "
                             f"{len(os.sched_getaffinity(0))} usable cores"}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": max_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": workload_config(w, extra={"gradient_pool": pool, "parallelism": f"replicas x{world}",
                                                "row_pitch_floats": ld}),
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": gpu_launches,
            "clocks": sampler.summary(),
        }
        print(json.dumps(line), flush=True)
    h.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
