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

Other modes (one JSON line each, not the headline):
    --sweep                         every scaling-sweep point that fits, with a clock record per point
    --mode rowshard-loopback        one node per GPU emulated on ONE device (n ranks, separate buffers)
    --mode rowshard [--arm sgp|osgp|allreduce]   one node per GPU under torchrun (NVLink peer loads; the
                                    all-reduce arm is parallel SGD with NCCL for context, Sec. 6.1)
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

# DRAM traffic of the fused step kernel from ncu captures of a column-scaled case of the same kernel and launch
# plan (profiles/*_small_ncu.md): dram__bytes_read.sum / dram__bytes_write.sum per launch at `d` columns.  Traffic
# grows in proportion to the columns processed, except that the last lines written are still dirty in L2 when the
# kernel ends (written back afterwards, invisible to the capture): that tail is the gap between the algorithmic
# write bytes and the captured ones at the small size, a constant per launch.
NCU_CAPTURES = {
    "resnet50": {"d": 2_000_008, "read": 768_238_848, "write": 710_679_552},
    "resnet50_osgp1": {"d": 2_000_008, "read": 1_024_070_144, "write": 966_900_480},
    "transformer": {"d": 4_000_000, "read": 512_055_808, "write": 456_322_560},
    "transformer_adam": {"d": 4_000_000, "read": 1_024_104_704, "write": 965_950_720},
}


def read_write_bytes_per_update(w, write_z=True):
    """Algorithmic HBM (read, write) bytes per node-parameter per step (fp32, in place)."""
    rd, wr = 8, 4                         # read x, g; write x
    if getattr(w, "optimizer", "sgd") == "adam":
        rd, wr = rd + 8, wr + 8           # both moment arrays
    elif w.momentum != 0.0:
        rd, wr = rd + 4, wr + 4           # u
    if write_z:
        wr += 4
    if w.tau > 0:
        rd, wr = rd + 4, wr + 4           # one ring slot
    return rd, wr


def bytes_per_update(w, write_z=True) -> int:
    return sum(read_write_bytes_per_update(w, write_z))


def scaled_traffic(w):
    """(bytes, detail) of one full-size launch from the workload's small-case capture, or (None, None)."""
    cap = NCU_CAPTURES.get(w.name.split("[")[0])
    if cap is None:
        return None, None
    _rd, wr = read_write_bytes_per_update(w)
    tail = max(0.0, wr * w.n * cap["d"] - cap["write"])        # dirty in L2 at kernel end, written back later
    read = cap["read"] * (w.d / cap["d"])
    write_in_kernel = wr * w.n * w.d - tail
    detail = {"capture_d": cap["d"], "dram_read_bytes": read, "dram_write_bytes_in_kernel": write_in_kernel,
              "l2_dirty_tail_bytes": tail,
              "how": "ncu dram__bytes_read.sum / dram__bytes_write.sum of one launch at capture_d columns, scaled by "
                     "the columns of a full launch; the tail is written back after the kernel ends and is counted"}
    return read + write_in_kernel + tail, detail


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

    def reset(self):
        self.samples, self.reasons = [], set()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=1.0)

    def summary(self):
        s = sorted(self.samples)
        return {"sm_mhz": (s[len(s) // 2] if s else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


# ------------------------------------------------------------------------------------------ CPU oracle legs
def _oracle_P_of_k(w):
    from oracle import schedule as osched
    if w.graph == "random":
        return lambda k: osched.mixing_matrix("random", w.n, k, seed=w.seed, max_outdeg=w.max_outdeg,
                                              num_steps=w.num_steps)
    return lambda k: osched.mixing_matrix(w.graph, w.n, k, peers=w.peers)


def _oracle_chunk(job):
    """The oracle, as it stands, on columns [c0, c1) of the workload; returns the seconds its timed steps took."""
    w, c0, c1, steps, warmup, one_blas_thread = job
    if one_blas_thread:
        try:
            from threadpoolctl import threadpool_limits
            threadpool_limits(1)
        except Exception:
            pass
    import numpy as np
    import torch
    from oracle import sgp as osgp
    from paper_1811_10792_b200 import inputs
    if one_blas_thread:
        torch.set_num_threads(1)
    cols = c1 - c0
    x0 = inputs.initial_x(w, device="cpu", d=cols, col_offset=c0).numpy().astype(np.float64)
    G = torch.empty((w.n, cols), dtype=torch.float32)
    grads = [inputs.gradient(w, k, G, col_offset=c0).numpy().astype(np.float64) for k in range(min(4, steps + warmup))]
    P_of_k = _oracle_P_of_k(w)
    adam = (lambda k: (k + 1, w.beta1, w.beta2, w.adam_eps)) if w.optimizer == "adam" else (lambda k: None)
    st = osgp.init_state(x0, w.tau)
    for k in range(warmup):
        osgp.sgp_step(st, grads[k % len(grads)], P_of_k(k), w.lr, w.momentum, w.nesterov, w.weight_decay, adam=adam(k))
    t0 = time.perf_counter()
    for k in range(warmup, warmup + steps):
        osgp.sgp_step(st, grads[k % len(grads)], P_of_k(k), w.lr, w.momentum, w.nesterov, w.weight_decay, adam=adam(k))
    return time.perf_counter() - t0


def oracle_single_process(w, sample_cols: int, steps: int, warmup: int):
    """(seconds per step, BLAS threads numpy used for P @ h; its elementwise work runs on one core)."""
    dt = _oracle_chunk((w, 0, sample_cols, steps, warmup, False)) / steps
    threads = 1
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        pass
    return dt, threads


def oracle_all_cores(w, sample_cols: int, steps: int, warmup: int):
    """The same oracle function mapped over column chunks in a process pool on every usable core (columns are
    independent, so this changes nothing numerically).  Returns (seconds per step of the whole sample, workers)."""
    import multiprocessing as mp
    workers = max(1, len(os.sched_getaffinity(0)))
    chunk = (sample_cols + workers - 1) // workers
    jobs = [(w, c0, min(sample_cols, c0 + chunk), steps, warmup, True) for c0 in range(0, sample_cols, chunk)]
    ctx = mp.get_context("spawn")
    pool = ctx.Pool(len(jobs))
    try:
        # every wait is bounded: a pool whose workers cannot start must not hold the benchmark up
        pool.map_async(_oracle_chunk, [(w, 0, 64, 1, 0, True)] * len(jobs), chunksize=1).get(timeout=180)   # start-up, imports
        # one chunk per worker, all running at once: the sample is done when the slowest worker's timed steps are
        times = pool.map_async(_oracle_chunk, jobs, chunksize=1).get(timeout=300)
    finally:
        pool.terminate()
        pool.join()
    return max(times) / steps, len(jobs)


def cpu_baseline(w, sample_cols: int, steps: int):
    """Both legs: one process, and all cores; `value` is the faster leg's, `cores` the processes it used."""
    dt1, blas = oracle_single_process(w, sample_cols, steps=steps, warmup=1)
    v1 = w.n * sample_cols / dt1
    usable = len(os.sched_getaffinity(0))
    legs = {"single_process": {"value": v1, "cores": 1, "blas_threads_for_the_mix": blas,
                               "note": "numpy elementwise work runs on one core; only P @ h is threaded"}}
    best, cores = v1, 1
    try:
        dtn, workers = oracle_all_cores(w, sample_cols, steps=steps, warmup=1)
        vn = w.n * sample_cols / dtn
        legs["all_cores"] = {"value": vn, "cores": workers,
                             "note": "the same oracle function mapped over column chunks in a process pool, one chunk "
                                     "per core, all at once; time of the slowest worker's timed steps"}
        if vn > best:
            best, cores = vn, workers
    except Exception as e:                                                      # the pool is a convenience, not the product
        legs["all_cores"] = {"value": None, "error": repr(e)}
    return {"value": best, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{steps} steps of the float64 numpy oracle on columns [0, {sample_cols}) "
                      f"({100.0 * sample_cols / w.d:.2f}% of d), all {w.n} nodes; host has {usable} usable cores",
            **legs}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample_cols = min(w.d, 1 << 18)
    dt, threads = oracle_single_process(w, sample_cols, args.steps, args.warmup)
    value = w.n * sample_cols / dt
    sample = f"float64 numpy oracle, columns [0, {sample_cols}) of {w.d} ({100.0 * sample_cols / w.d:.2f}%), all {w.n} nodes"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, extra={"parallelism": f"replicas x{args.gpus}"}),
        "sample_cols": sample_cols,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                         "blas_threads_for_the_mix": threads},
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


def roofline_of(w, kern_ms, peak, peak_kind):
    bpu = bytes_per_update(w)
    achieved = bpu * w.n * w.d / (kern_ms * 1e-3) / 1e9
    traffic, detail = scaled_traffic(w)
    return {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": traffic, "traffic_detail": detail, "peak_kind": f"of {peak_kind}",
            "kernel": "sgp_step (fused update + mix + de-bias)", "algorithmic_bytes_per_launch": bpu * w.n * w.d,
            "kernel_ms": kern_ms, "frac_of_nominal_8TBps": achieved / NOMINAL_HBM_GBS}


def run_sweep(args):
    """Scaling sweep (random digraphs, Nesterov, Z written): one JSON line per (n, d) point that fits 150 GB,
    each with its own clock record."""
    import torch
    from paper_1811_10792_b200 import binding, inputs
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, peak_kind = measured_peak()
    sampler = ClockSampler(0)
    sampler.start()
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
            # points that finish in microseconds are repeated so that the clock sampler sees them under load
            reps = max(1, int(0.15 / max(1e-6, K * 24.0 * n * d / 6.5e12)))
            with binding.Sgp(n, d, binding.graph_desc(w), ld=ld) as h:
                for kv in args.option:
                    key, val = kv.split("=")
                    h.set_option(key, int(val))
                for k in range(max(3, args.warmup)):
                    h.step(X, Wt, M, G, Z, k, w.lr, w.momentum, 0.0, True)
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                sampler.reset()
                sampler.arm(True)
                e0.record()
                for _rep in range(reps):
                    for k in range(K):
                        h.step(X, Wt, M, G, Z, 3 + k, w.lr, w.momentum, 0.0, True)
                e1.record()
                torch.cuda.synchronize()
                sampler.arm(False)
                clocks = sampler.summary()
                ms = e0.elapsed_time(e1) / (K * reps)
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
            print(json.dumps({"metric": METRIC, "value": n * d / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K * reps,
                              "ms_per_step": ms, "graph_replay_ms_per_step": graph_ms, "dtype": "f32",
                              "data": "synthetic",
                              "config": workload_config(w, extra={"row_pitch_floats": ld, **launch}),
                              "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                                           "frac": achieved / peak, "peak_kind": f"of {peak_kind}"},
                              "clocks": clocks}), flush=True)
            del X, M, Z, G
            torch.cuda.empty_cache()
    sampler.stop()


def link_probe(dev, nbytes: int, reps: int = 3):
    """Plain pinned copies, host->device and device->host at the same time on two streams: what the link gives
    a step that moves `nbytes` each way.  Returns GB/s per direction."""
    import torch
    nbytes = min(nbytes, 1 << 30)
    h_in = torch.empty(nbytes // 4, dtype=torch.float32, pin_memory=True)
    h_out = torch.empty(nbytes // 4, dtype=torch.float32, pin_memory=True)
    d_in = torch.empty(nbytes // 4, dtype=torch.float32, device=dev)
    d_out = torch.empty(nbytes // 4, dtype=torch.float32, device=dev)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    best = 0.0
    for _ in range(reps):
        t0 = time.perf_counter()
        with torch.cuda.stream(s1):
            d_in.copy_(h_in, non_blocking=True)
        with torch.cuda.stream(s2):
            h_out.copy_(d_out, non_blocking=True)
        torch.cuda.synchronize()
        best = max(best, nbytes / (time.perf_counter() - t0) / 1e9)
    return best


# ------------------------------------------------------------------------------------------ one node per GPU
def run_rowshard_loopback(args, w):
    """w.n ranks of the one-node-per-GPU mode on ONE device: the split kernels' HBM efficiency without NVLink.
    Algorithmic bytes per node-parameter: tau = 0: update (read x, g, u; write u, message) + mix (read own message
    and one per in-neighbour; write x, z); tau >= 1: one kernel (read x, g, u and one message per delayed
    in-neighbour; write u, message, x, z)."""
    import torch
    from paper_1811_10792_b200 import binding, inputs, rowshard
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    n, d, K = w.n, w.d, args.steps
    X0 = inputs.initial_x(w, device=dev)
    xs = [X0[r].clone() for r in range(n)]
    del X0
    ms = [torch.zeros(d, device=dev) for _ in range(n)]
    zs = [torch.empty(d, device=dev) for _ in range(n)]
    gs = [torch.empty(d, device=dev) for _ in range(n)]
    G = torch.empty((1, d), device=dev)
    for r in range(n):
        inputs.fill_normal(G, seed=w.seed, stream=inputs.STREAM_GRAD, step=0, std=w.grad_std, row_offset=r)
        gs[r].copy_(G[0])
    ws = [torch.ones(1, device=dev) for _ in range(n)]
    sampler = ClockSampler(0)
    sampler.start()
    with rowshard.LoopbackGroup(n, d, binding.graph_desc(w), tau=w.tau) as grp:
        for k in range(max(3, args.warmup)):
            grp.step(xs, ws, ms, gs, zs, k, w.lr, w.momentum, w.weight_decay, w.nesterov)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler.arm(True)
        e0.record()
        for k in range(K):
            grp.step(xs, ws, ms, gs, zs, 3 + k, w.lr, w.momentum, w.weight_decay, w.nesterov)
        e1.record()
        torch.cuda.synchronize()
        sampler.arm(False)
        assert grp.device_status() == 0
    sampler.stop()
    ms_step = e0.elapsed_time(e1) / K
    indeg = {"exp": w.peers, "bipartite": 1}.get(w.graph, 2.5)
    mom = 8 if w.momentum != 0.0 else 0
    bpu = (8 + mom + 4) + (4 + 4 * indeg + 8) if w.tau == 0 else (8 + mom + 4 * indeg + 4 + 8)
    peak, peak_kind = measured_peak()
    achieved = bpu * n * d / (ms_step * 1e-3) / 1e9
    print(json.dumps({"metric": METRIC, "value": n * d / (ms_step * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K,
                      "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True, "dtype": "f32",
                      "data": "synthetic", "mode": "rowshard-loopback",
                      "config": workload_config(w, extra={"parallelism": f"{n} virtual ranks on one device",
                                                          "kernels_per_step": n * (2 if w.tau == 0 else 1)}),
                      "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                                   "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                                   "algorithmic_bytes_per_update": bpu},
                      "clocks": sampler.summary()}), flush=True)


def run_rowshard(args, w):
    """One node per GPU under torchrun: world = n nodes; `value` = n * d / slowest rank's step time.  Arms: sgp
    (tau = 0: update, barrier, pull+mix), osgp (tau = 1: one fused kernel per step), allreduce (parallel SGD: NCCL
    all-reduce of the gradients, then the local Nesterov step -- the baseline SGP is compared with in Sec. 6.1)."""
    import dataclasses
    import torch
    import torch.distributed as dist
    from paper_1811_10792_b200 import binding, inputs, rowshard
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist.init_process_group("nccl", device_id=dev)
    tau = {"sgp": 0, "osgp": 1, "allreduce": 0}[args.arm]
    w = dataclasses.replace(w, n=world, tau=tau)
    d, K = w.d, args.steps
    G = torch.empty((1, d), device=dev)
    inputs.fill_normal(G, seed=w.seed, stream=inputs.STREAM_X0, step=0, std=w.x0_std, row_offset=0 if w.x0_shared else rank)
    x = G[0].clone()
    m, z = torch.zeros(d, device=dev), torch.empty(d, device=dev)
    inputs.fill_normal(G, seed=w.seed, stream=inputs.STREAM_GRAD, step=0, std=w.grad_std, row_offset=rank)
    g = G[0].clone()
    wt = torch.ones(1, device=dev)
    if args.arm == "allreduce":
        h = binding.Sgp(1, d, binding.GraphDesc.complete())
        gsum = torch.empty_like(g)

        def step(k):
            gsum.copy_(g)
            dist.all_reduce(gsum)                                   # NCCL over NVLink / NVSwitch
            gsum.mul_(1.0 / world)
            h.step(x.view(1, d), wt, m.view(1, d), gsum.view(1, d), z.view(1, d), k, w.lr, w.momentum, w.weight_decay, True)
        closer = h.close
    else:
        node = rowshard.DistributedRank(d, binding.graph_desc(w), tau=tau)

        def step(k):
            node.step(x, wt, m, g, z, k, w.lr, w.momentum, w.weight_decay, True)
        closer = node.close
    for k in range(max(3, args.warmup)):
        step(k)
    torch.cuda.synchronize()
    dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.arm(True)
    e0.record()
    for k in range(K):
        step(3 + k)
    e1.record()
    torch.cuda.synchronize()
    clocks_note = None
    if e0.elapsed_time(e1) < 600.0:
        # the timed region is shorter than a few sampling intervals: the same steps go on, untimed, until the sampler
        # has seen the load (every rank runs the same count, so the barriers inside the steps still pair up)
        extra = int(600.0 / max(1e-3, e0.elapsed_time(e1) / K)) + 1
        extra = int(max_over_ranks(float(extra), dev))
        for k in range(extra):
            step(3 + K + k)
        torch.cuda.synchronize()
        clocks_note = "sampled while the same steps were repeated right after the timed region (the region is shorter than the sampling interval)"
    sampler.arm(False)
    dist.barrier()
    sampler.stop()
    max_ms = max_over_ranks(e0.elapsed_time(e1), dev)
    clocks = sampler.summary()
    if clocks_note:
        clocks["note"] = clocks_note
    # this library's kernels per step and rank: update + pull/mix (sgp), one fused kernel (osgp), the local step (allreduce)
    launches = {"sgp": 2, "osgp": 1, "allreduce": 1}[args.arm] * K
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": world * d * K / (max_ms * 1e-3), "unit": UNIT, "n_gpus": world,
                          "steps": K, "warmup": max(3, args.warmup), "ms_per_step": max_ms / K, "higher_is_better": True,
                          "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic", "mode": "rowshard",
                          "arm": args.arm,
                          "config": workload_config(w, extra={"parallelism": f"one node per GPU x{world}"}),
                          "gpu_launches": launches, "clocks": clocks}), flush=True)
    closer()
    dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="resnet50",
                    help="resnet50 | transformer | resnet50_osgp1 | transformer_adam | tiny | sweep:<n>:<d>")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--mode", default="replicas", choices=["replicas", "rowshard", "rowshard-loopback"])
    ap.add_argument("--arm", default="sgp", choices=["sgp", "osgp", "allreduce"], help="--mode rowshard only")
    ap.add_argument("--d", type=int, default=0, help="override the parameter count (profiling on a small case)")
    ap.add_argument("--n", type=int, default=0, help="override the node count (rowshard-loopback)")
    ap.add_argument("--tau", type=int, default=-1, help="override the delay")
    ap.add_argument("--peers", type=int, default=0, help="override the out-neighbours per node of the exponential graph")
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

    import dataclasses
    from paper_1811_10792_b200 import inputs
    if args.workload.startswith("sweep:"):            # sweep:<n>:<d>  (scaling-sweep point, random digraphs)
        _, sn, sd = args.workload.split(":")
        w = inputs.sweep_workload(int(sn), int(sd))
    else:
        w = inputs.WORKLOADS[args.workload]
    if args.d > 0:
        w = w.scaled(args.d)
    if args.n > 0:
        w = dataclasses.replace(w, n=args.n)
    if args.tau >= 0:
        w = dataclasses.replace(w, tau=args.tau)
    if args.peers > 0:
        w = dataclasses.replace(w, peers=args.peers)
    if args.impl == "reference":
        run_reference(args, w)
        return
    if args.mode == "rowshard-loopback":
        run_rowshard_loopback(args, w)
        return
    if args.mode == "rowshard":
        run_rowshard(args, w)
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
    launch = {k: h.get_option(k) for k in ("last_variant", "last_grid", "last_tile_cols", "last_smem")}
    total_ms = evs[0].elapsed_time(evs[K])
    per_step_ms = [evs[i].elapsed_time(evs[i + 1]) for i in range(K)]
    assert h.device_status() == 0
    max_ms = max_over_ranks(total_ms, dev)
    value = whole_job_value(world, n * d, K, max_ms)

    # ---- end to end through the host-buffer entry point (gradients in, de-biased parameters out)
    e2e = None
    if not args.no_e2e:
        hG = torch.empty((n, ld), dtype=torch.float32, pin_memory=True)[:, :d]
        hZ = torch.empty((n, ld), dtype=torch.float32, pin_memory=True)[:, :d]
        hG.copy_(Gs[0])
        dG = Gs[0]
        torch.cuda.synchronize()
        e2e_steps = K

        def host_step(k):
            if adam:
                h.step_adam_host(X, Wt, M, V2, hG, hZ, dG, Z, k, k + 1, w.lr, w.beta1, w.beta2, w.adam_eps, w.weight_decay)
            else:
                h.step_host(X, Wt, M, hG, hZ, dG, Z, k, w.lr, w.momentum, w.weight_decay, w.nesterov)
        host_step(Wm + K)                                                                            # warm
        if world > 1:
            dist.barrier()
        t0 = time.perf_counter()
        for i in range(e2e_steps):
            host_step(Wm + K + 1 + i)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        dt_max = max_over_ranks(dt, dev)
        e2e = {"value": whole_job_value(world, n * d, e2e_steps, dt_max * 1e3), "unit": UNIT,
               "h2d_bytes_per_step": arr_bytes, "d2h_bytes_per_step": arr_bytes, "steps": e2e_steps,
               "ms_per_step": dt_max * 1e3 / e2e_steps,
               "gbs_each_way": arr_bytes / (dt_max / e2e_steps) / 1e9}
        del hG, hZ
        if rank == 0:
            e2e["link_probe_gbs_each_way"] = link_probe(dev, arr_bytes)      # plain pinned copies, both directions at once
    sampler.stop()

    if rank == 0:
        peak, peak_kind = measured_peak()
        kern_ms = sum(per_step_ms) / len(per_step_ms)
        roofline = roofline_of(w, kern_ms, peak, peak_kind)
        cpu = None
        if not args.no_cpu_baseline and world == 1:          # the CPU oracle is timed in single-GPU runs only
            cpu = cpu_baseline(w, min(d, 1 << 20), steps=8)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": max_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            # the same keys and values as the reference arm's line; how this arm laid the workload out is in "launch"
            "config": workload_config(w, extra={"parallelism": f"replicas x{world}"}),
            "launch": {"gradient_pool": pool, "row_pitch_floats": ld, **launch},
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": gpu_launches,
            "clocks": sampler.summary(),
        }
        print(json.dumps(line), flush=True)
    h.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
