#!/usr/bin/env python
"""Throughput of the fused DeTAG step: worker-coordinate updates per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg5] [--impl ours|reference]

One "step" is one whole DeTAG iteration (tracker fold, K accelerated-gossip rounds on tracker and model,
model update, stochastic gradient) over all n workers of the chosen synthetic configuration.  With N > 1
(launched by torch.distributed.run, one rank per GPU) every rank steps its own coordinate shard of the same
size; the step has no exchange between coordinates, so there is no data-path collective (weak scaling).

With --gpus N > 1 and no launcher around it (WORLD_SIZE unset) the script starts its own N ranks through
torch.distributed.run on 127.0.0.1.  `--host-only` (used by the CPU test of that path) makes the ranks meet over
gloo, exchange the two scalars the real run reduces, and stop before the first CUDA call.

Prints ONE JSON line on rank 0.  `--impl reference` times the float64 CPU oracle on a bounded sample instead.
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
sys.path.insert(0, ROOT)

from paper_2006_08085_b200 import inputs  # noqa: E402

METRIC = "worker-coord updates/s per DeTAG step (n*d/s)"
UNIT = "wc/s"
BYTES_PER_WC = 32  # read x, y, g, a, c + write x, y, g, float32 each: the fused step's minimum HBM traffic

# DRAM traffic per worker-coordinate (dram__bytes_read.sum + dram__bytes_write.sum from one ncu capture on a
# small case of the same kernel; traffic grows in proportion to n*d).  Keyed by the sha256 prefix of the kernel
# sources the capture was taken on: a changed kernel reports null until it is captured again.
KERNEL_SOURCES = {
    "wide": ("step_wide.cu", "pipeline.cuh", "noise.cuh"),
    "mma": ("step_mma.cu", "mma_common.cuh", "pipeline.cuh", "noise.cuh"),
    "band": ("step_band.cu", "pipeline.cuh", "noise.cuh"),
    "ring": ("step_ring.cu", "pipeline.cuh", "noise.cuh"),
    "csr": ("step_csr.cu", "noise.cuh"),
    "torus": ("step_torus.cu", "torus_basis.h", "pipeline.cuh", "noise.cuh"),
}
MEASURED_TRAFFIC = {
    # (kernel, mode): (source digest, bytes per wc)
    ("mma", "dense"): ("22eae46feb506e80", 31.46),     # cfg5 shape at d = 2 M: 1.2949 GB read + 0.7183 GB written / 64 M wc
    ("torus", "torus8"): ("427a2bff49b63d9c", 31.27),  # cfg3 shape at d = 1 M: 1.2803 + 0.7208 GB / 64 M wc
    ("ring", "band"): ("60c16ee651aa8e4f", 31.12),     # cfg4 shape at d = 200 k: 1.0280 + 0.5652 GB / 51.2 M wc
    ("wide", "dense"): ("77d5b7be943b4c42", 30.83),    # 100-worker random graph at d = 400 k: 0.8011 + 0.4321 GB / 40 M wc
    ("csr", "rounds"): ("bcc2ab2f791da0eb", 31.17),    # the same graph through the rounds kernel: 0.8088 + 0.4381 GB / 40 M wc
}

# Float64 multiply-adds per worker-coordinate on the FP64 pipe (both contractions, padded shapes) and that
# pipe's peak: 64 multiply-adds per clock and SM (measured: 61 with m8n8k4 MMAs from 16 warps) x 148 SMs x max clock.
FP64_FMA_PER_WC = {("mma", "dense"): 64, ("ring", "band"): 80, ("band", "dense"): 128,
                   ("torus", "torus8"): 26, ("torus", "torus4"): 28}
VARIANT_NAMES = {1: "csr", 2: "dense", 3: "ring", 4: "torus"}
FP64_FMA_PER_CLK_SM = 64
SM_COUNT = 148


def kernel_key(variant: str, n: int):
    if variant == "dense":
        return ("mma", "dense") if n <= 32 else ("band", "dense") if n <= 64 else ("wide", "dense")
    if variant == "ring":
        return ("ring", "band")
    if variant == "csr":
        return ("csr", "rounds")
    if variant == "torus":
        return ("torus", "torus8" if n == 64 else "torus4")
    return None


def source_digest(kernel: str) -> str:
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES[kernel]:
        with open(os.path.join(ROOT, "paper_2006_08085_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def measured_traffic_bytes(variant: str, n: int, wc: int):
    key = kernel_key(variant, n)
    if key is None or key not in MEASURED_TRAFFIC:
        return None
    digest, per_wc = MEASURED_TRAFFIC[key]
    try:
        if source_digest(key[0]) != digest:
            return None
    except OSError:
        return None
    return per_wc * wc


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return 6650.0, "fallback (earlier measurement on this pool)"


# ------------------------------------------------------------------------------------ oracle timing
def _oracle_sample(cfg, j0: int, m: int):
    """The oracle's problem and initial state for coordinates [j0, j0 + m) of a configuration."""
    from oracle import detag_oracle as orc

    gm = inputs.gossip_matrix(cfg)
    eta = orc.spectrum(gm.to_dense()).eta
    a, c, x0 = inputs.objective_data(cfg, j0, j0 + m)
    p = orc.Problem(gm.row_ptr, gm.col_idx, gm.vals, cfg.K, eta, cfg.alpha, a, c, cfg.sigma, cfg.seed, j0)
    return orc, p, orc.init_state(p, x0)


def oracle_throughput(cfg, budget_s: float, sample_d: int, steps: int):
    """Times the float64 oracle (as it stands, one process) on `sample_d` coordinates; returns a dict."""
    m = min(sample_d, cfg.d)
    orc, p, s = _oracle_sample(cfg, 0, m)
    done, t0 = 0, time.perf_counter()
    while done < steps and (done == 0 or time.perf_counter() - t0 < budget_s):
        s = orc.step(p, s)
        done += 1
    dt = time.perf_counter() - t0
    return {"value": cfg.n * m * done / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{done} steps of {cfg.name} on the first {m} of {cfg.d} coordinates "
                      f"(all {cfg.n} workers), {dt:.1f} s, single process",
            "_ms_per_step": dt / done * 1e3, "_steps": done, "_sample_wc": cfg.n * m}


def _oracle_worker(job):
    """One process of the all-cores leg: its own coordinate range, stepped until the time budget is spent."""
    name, j0, m, budget_s = job
    cfg = inputs.CONFIGS[name]
    orc, p, s = _oracle_sample(cfg, j0, m)
    done, t0 = 0, time.perf_counter()
    while done == 0 or time.perf_counter() - t0 < budget_s:
        s = orc.step(p, s)
        done += 1
    return done, time.perf_counter() - t0


def oracle_throughput_all_cores(cfg, budget_s: float, sample_d: int):
    """One oracle process per host core on disjoint coordinate ranges (the step never mixes coordinates).
    The processes are started with `spawn`: a process forked after the first CUDA call would hang."""
    import multiprocessing as mp

    cores = min(os.cpu_count() or 1, 128)
    m = max(1, min(sample_d, cfg.d // cores))
    os.environ.setdefault("OMP_NUM_THREADS", "1")  # one core per process: no nested threading in the children
    jobs = [(cfg.name, k * m, m, budget_s) for k in range(cores)]
    with mp.get_context("spawn").Pool(cores) as pool:
        res = pool.map(_oracle_worker, jobs)
    value = sum(cfg.n * m * done / dt for done, dt in res)
    return {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{cores} processes, one per host core, each stepping its own {m} coordinates of {cfg.name} "
                      f"(all {cfg.n} workers) for {budget_s:.0f} s: {sum(d for d, _ in res)} steps in total"}


def cpu_baseline(cfg, budget_s: float):
    sample_d = max(1024, min(cfg.d, 400_000 // cfg.n))
    one = oracle_throughput(cfg, budget_s, sample_d, 10 ** 9)
    out = oracle_throughput_all_cores(cfg, budget_s, sample_d)
    out["one_core"] = {k: v for k, v in one.items() if not k.startswith("_")}
    return out


def run_reference(args, rank: int) -> None:
    if rank != 0:
        return
    cfg = inputs.CONFIGS[args.config]
    sample_d = max(1024, min(cfg.d, 400_000 // cfg.n))
    # each "step" is one oracle step on the bounded sample; warm-up steps are run and dropped
    oracle_throughput(cfg, 1e9, sample_d, max(args.warmup, 0) or 1) if args.warmup > 0 else None
    r = oracle_throughput(cfg, 150.0, sample_d, args.steps)
    line = {
        "impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": r["_steps"], "warmup": args.warmup, "ms_per_step": r["_ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "n": cfg.n, "d": cfg.d, "K": cfg.K, "graph": cfg.graph,
                   "sample_coordinates": sample_d},
        "cpu_baseline": {k: v for k, v in r.items() if not k.startswith("_")},
        "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------ clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ready = threading.Event()  # set once the first sample is in (NVML start-up can take a while)
        self.error = None

    def run(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            while not self._stop_evt.is_set():
                self.samples.append(int(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                mask = int(pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
                self.ready.set()
                time.sleep(self.period)
        except Exception as exc:  # NVML missing: report it, the timing itself is unaffected
            self.error = repr(exc)
            self.ready.set()

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2.0)
        out = {"sm_mhz": float(np.median(self.samples)) if self.samples else None, "sm_max_mhz": self.max_mhz,
               "reasons": sorted(self.reasons), "samples": len(self.samples)}
        if self.error:
            out["error"] = self.error
        return out


# ------------------------------------------------------------------------------------ our arm
def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def time_config(name: str, dev, args) -> dict:
    """Device-resident step time of one configuration at its full size (a short run: 3 warm-up steps, then 20
    or 200 timed ones), with both roofline fractions.  Inputs are the configuration's own seeded arrays."""
    import torch

    from paper_2006_08085_b200 import binding as B
    from paper_2006_08085_b200.session import Session

    cfg = inputs.CONFIGS[name]
    gm = inputs.gossip_matrix(cfg)
    ld = (cfg.d + 3) // 4 * 4
    s = Session(gm, cfg.d, cfg.K, float("nan"), cfg.alpha, None, None, None, cfg.sigma, cfg.seed, ld=ld, device=str(dev))
    chunk = 1 << 21
    for j0 in range(0, cfg.d, chunk):  # objective data chunk by chunk: bounded host memory
        j1 = min(cfg.d, j0 + chunk)
        a, c, x0 = inputs.objective_data(cfg, j0, j1, threads=min(32, os.cpu_count() or 1))
        for nm, arr in (("a", a), ("c", c), ("x", x0)):
            getattr(s, nm)[:, j0:j1].copy_(torch.from_numpy(arr))
    variant = VARIANT_NAMES.get(B.detag_get_variant(s.state), "other")
    stream = torch.cuda.current_stream(dev)
    s.init()
    steps = 200 if 20 * cfg.wc < 4 * 126e6 else 20
    for _ in range(3):
        B.detag_step(s.state, stream)
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        B.detag_step(s.state, stream)
    e1.record(stream)
    torch.cuda.synchronize(dev)
    s.status()
    ms = e0.elapsed_time(e1) / steps
    ce = s.consensus_error()
    s.close()
    del s
    torch.cuda.empty_cache()
    peak, _ = measured_peak_gbs()
    achieved = BYTES_PER_WC * cfg.wc / (ms * 1e-3) / 1e9
    key = kernel_key(variant, cfg.n)
    out = {"workload": cfg.name, "n": cfg.n, "d": cfg.d, "K": cfg.K, "graph": cfg.graph, "variant": variant,
           "steps": steps, "ms_per_step": ms, "value": cfg.wc / (ms * 1e-3), "unit": UNIT,
           "achieved_gbs": achieved, "frac_of_measured_peak": achieved / peak,
           "frac_of_8TBps_nominal": achieved / 8000.0, "consensus_error_after_run": ce,
           "l2": "exceeds L2" if 20 * cfg.wc > 4 * 126e6 else "working set fits the 126 MB L2: not an HBM measurement"}
    if key in FP64_FMA_PER_WC:
        out["fp64_fma_per_wc"] = FP64_FMA_PER_WC[key]
        out["fp64_pipe_frac"] = FP64_FMA_PER_WC[key] * out["value"] / (FP64_FMA_PER_CLK_SM * SM_COUNT * 1965e6)
    traffic = measured_traffic_bytes(variant, cfg.n, cfg.wc)  # ncu DRAM bytes of a small case, scaled; None if stale
    out["traffic_bytes_per_step"] = traffic
    return out


def theorem3_regime(dev, args) -> dict:
    """cfg4's 256-ring at the configuration's K = 16 and at Theorem 3's phase length (K = 196, where the gossip
    polynomial is a dense circulant), on a 200,000-coordinate cut: step time and the consensus error per
    worker-coordinate after every step (it grows at K = 16 and contracts at Theorem 3's K)."""
    import dataclasses

    import torch

    from paper_2006_08085_b200 import binding as B
    from paper_2006_08085_b200.session import Session

    base = inputs.CONFIGS["cfg4"].with_d(200_000)
    gm = inputs.gossip_matrix(base)
    lam = B.detag_spectral(gm.n, gm.row_ptr, gm.col_idx, gm.vals)[2]
    k_thm = B.detag_phase_length(gm.n, lam)
    a, c, x0 = inputs.objective_data(base, threads=min(32, os.cpu_count() or 1))
    out = {"workload": "cfg4 ring, d = 200,000", "lambda": lam, "runs": []}
    stream = torch.cuda.current_stream(dev)
    for K in (base.K, k_thm):
        cfg = dataclasses.replace(base, K=K)
        s = Session(gm, cfg.d, cfg.K, float("nan"), cfg.alpha, a, c, x0, cfg.sigma, cfg.seed, device=str(dev))
        s.init()
        ce = [s.consensus_error() / cfg.wc]
        steps = 10
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ms = 0.0
        for _ in range(steps):
            e0.record(stream)
            B.detag_step(s.state, stream)
            e1.record(stream)
            torch.cuda.synchronize(dev)
            ms += e0.elapsed_time(e1)
            ce.append(s.consensus_error() / cfg.wc)
        s.status()
        out["runs"].append({"K": K, "variant": VARIANT_NAMES.get(B.detag_get_variant(s.state), "other"),
                            "ms_per_step": ms / steps, "value": cfg.wc / (ms / steps * 1e-3), "unit": UNIT,
                            "fp64_fma_per_wc": 80 if K == base.K else 2 * cfg.n,
                            "consensus_error_per_wc_by_step": ce})
        s.close()
        del s
    torch.cuda.empty_cache()
    return out


def general_graph(dev, args) -> dict:
    """Graphs none of the structured kernels takes - seeded random 4-regular graphs with 100 and with 72 workers,
    K = 6, d = 2,000,000: step time and roofline fractions of the kernel the library picks (the dense polynomial
    held in registers, whose bound is the FP64 tensor pipe: 2 * n_padded multiply-adds per worker-coordinate) and,
    for the 100-worker graph, of the generic rounds kernel that takes every graph."""
    import torch

    from paper_2006_08085_b200 import binding as B
    from paper_2006_08085_b200.session import Session

    d, K = (args.d if args.leg == "general_graph" and args.d else 2_000_000), 6
    peak, _ = measured_peak_gbs()
    stream = torch.cuda.current_stream(dev)

    def one(n: int, forced: int) -> dict:
        gm = inputs.metropolis_weights(inputs.random_regular4_graph(n, 7))
        s = Session(gm, d, K, float("nan"), 0.001, None, None, None, 0.1, 7, device=str(dev), variant=forced)
        gen = torch.Generator(device=dev).manual_seed(7)
        s.a.uniform_(0.5, 2.0, generator=gen)  # objective data drawn on the device: this leg times the kernel only
        s.c.normal_(generator=gen)
        s.init()
        for _ in range(3):
            B.detag_step(s.state, stream)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(10):
            B.detag_step(s.state, stream)
        e1.record(stream)
        torch.cuda.synchronize(dev)
        s.status()
        ms = e0.elapsed_time(e1) / 10
        variant = VARIANT_NAMES.get(B.detag_get_variant(s.state), "other")
        s.close()
        del s
        torch.cuda.empty_cache()
        gbs = BYTES_PER_WC * n * d / (ms * 1e-3) / 1e9
        out = {"workload": f"{n} workers, random 4-regular graph (Metropolis weights), d = {d:,}, K = {K}",
               "variant": variant, "ms_per_step": ms, "value": n * d / (ms * 1e-3), "unit": UNIT, "achieved_gbs": gbs,
               "frac_of_measured_peak": gbs / peak, "frac_of_8TBps_nominal": gbs / 8000.0}
        if variant == "dense":
            fma = 2 * ((n + 7) // 8 * 8)
            out["fp64_fma_per_wc"] = fma
            out["fp64_pipe_frac"] = fma * out["value"] / (FP64_FMA_PER_CLK_SM * SM_COUNT * 1965e6)
        return out

    return {"picked_100": one(100, 0), "rounds_100": one(100, B.DETAG_VARIANT_CSR), "picked_72": one(72, 0)}


def run_host_only(args, rank: int, world: int) -> None:
    """The multi-rank plumbing without a GPU: the ranks meet over gloo, work out their shards and reduce the two
    scalars the real run reduces (slowest rank's time, sum of the shards' consensus errors)."""
    import torch.distributed as dist

    from paper_2006_08085_b200 import sharding

    if world > 1:
        dist.init_process_group("gloo")
    cfg = inputs.CONFIGS[args.config]
    offset = sharding.weak_scaling_offset(cfg.d, rank)
    slowest = sharding.reduce_max(1.0 + rank, dist if world > 1 else None)
    total = sharding.reduce_sum(float(offset), dist if world > 1 else None)
    if rank == 0:
        print(json.dumps({"host_only": True, "n_gpus": world, "slowest": slowest, "offset_sum": total,
                          "config": {"workload": cfg.name}}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def spawn_ranks(n: int) -> int:
    """Starts n ranks of this script through torch.distributed.run on the loopback address and waits for them."""
    import socket
    import subprocess

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def run_ours(args, rank: int, world: int, local_rank: int) -> None:
    import torch
    import torch.distributed as dist

    from paper_2006_08085_b200 import binding as B, build, sharding
    from paper_2006_08085_b200.session import Session

    build.build()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if args.leg == "general_graph":  # that leg alone (a small case of it with --d: what the ncu capture runs)
        if rank == 0:
            print(json.dumps({"general_graph": general_graph(dev, args)}), flush=True)
        return
    cfg = inputs.CONFIGS[args.config]
    if args.d:
        cfg = cfg.with_d(args.d)
    m = inputs.gossip_matrix(cfg)
    t_setup = time.perf_counter()

    # Objective data on the host (page-locked: the end-to-end leg copies from it), then to the device.
    ld = (cfg.d + 3) // 4 * 4
    pin = torch.cuda.is_available()
    host = {k: torch.empty((cfg.n, ld), dtype=torch.float32, pin_memory=pin) for k in ("a", "c", "x")}
    threads = max(1, min(32, (os.cpu_count() or 1) // max(1, world)))
    inputs.objective_data(cfg, threads=threads,
                          out=tuple(host[k].numpy()[:, : cfg.d] for k in ("a", "c", "x")))
    s = Session(m, cfg.d, cfg.K, float("nan"), cfg.alpha, None, None, None, cfg.sigma, cfg.seed,
                coord_offset=sharding.weak_scaling_offset(cfg.d, rank), ld=ld, device=str(dev))
    for k in ("a", "c", "x"):
        getattr(s, k).copy_(host[k], non_blocking=True)
    torch.cuda.synchronize(dev)
    if args.variant:
        B.detag_set_variant(s.state, {v: k for k, v in VARIANT_NAMES.items()}[args.variant])
    variant = VARIANT_NAMES[B.detag_get_variant(s.state)]
    t_setup = time.perf_counter() - t_setup

    stream = torch.cuda.current_stream(dev)
    s.init()
    for _ in range(max(args.warmup, 3)):
        B.detag_step(s.state, stream)
    torch.cuda.synchronize(dev)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize(dev)

    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    sampler.ready.wait(5.0)
    events = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    events[0].record(stream)
    for k in range(args.steps):
        B.detag_step(s.state, stream)  # one kernel launch per step
        events[k + 1].record(stream)
    torch.cuda.synchronize(dev)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize(dev)
    clocks = sampler.stop()
    s.status()
    total_ms = events[0].elapsed_time(events[-1])
    per_step = np.array([events[k].elapsed_time(events[k + 1]) for k in range(args.steps)])
    total_ms_max = sharding.reduce_max(total_ms, dist if world > 1 else None, dev)
    consensus = sharding.reduce_sum(s.consensus_error(), dist if world > 1 else None, dev)

    # ---- extra, not the headline: the same iterations through detag_step_many (on chip across steps where the
    # variant allows it: the state crosses HBM once per call instead of once per step)
    multi = None
    if world == 1 and args.steps_per_launch >= 2:
        T = args.steps_per_launch
        B.detag_step_many(s.state, T, stream)  # warm-up
        m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        m0.record(stream)
        for _ in range(args.multi_launches):
            B.detag_step_many(s.state, T, stream)
        m1.record(stream)
        torch.cuda.synchronize(dev)
        s.status()
        ms = m0.elapsed_time(m1) / (T * args.multi_launches)
        multi = {"api": "detag_step_many", "steps_per_launch": T, "launches": args.multi_launches,
                 "ms_per_step": ms, "value": cfg.wc / (ms * 1e-3), "unit": UNIT,
                 "hbm_bytes_per_wc_per_step": BYTES_PER_WC / T if variant == "dense" and cfg.n <= 32 else BYTES_PER_WC}

    # ---- extra: the other step modes on the same buffers (D-PSGD: 24 B/wc; caller-written gradients: 28 B/wc)
    modes = None
    if world == 1 and not args.no_modes:
        modes = {}
        m_steps = max(3, min(20, args.steps))

        def timed(label, bytes_per_wc):
            for _ in range(3):
                B.detag_step(s.state, stream)
            m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            m0.record(stream)
            for _ in range(m_steps):
                B.detag_step(s.state, stream)
            m1.record(stream)
            torch.cuda.synchronize(dev)
            s.status()
            ms = m0.elapsed_time(m1) / m_steps
            gbs = bytes_per_wc * cfg.wc / (ms * 1e-3) / 1e9
            modes[label] = {"ms_per_step": ms, "value": cfg.wc / (ms * 1e-3), "unit": UNIT, "steps": m_steps,
                            "bytes_per_wc": bytes_per_wc, "achieved_gbs": gbs,
                            "variant": VARIANT_NAMES.get(B.detag_get_variant(s.state), "other")}

        B.detag_set_algorithm(s.state, B.DETAG_ALGORITHM_DPSGD)
        timed("dpsgd", 24)
        B.detag_set_algorithm(s.state, B.DETAG_ALGORITHM_DETAG)
        g_new = torch.empty_like(s.g)
        g_new.copy_(s.g)
        B.detag_set_gradient_source(s.state, B.DETAG_GRADIENT_EXTERNAL, g_new)
        timed("external_gradient", 28)  # the same gradient array every step: the traffic is what is timed
        B.detag_set_gradient_source(s.state, B.DETAG_GRADIENT_SYNTHETIC, None)
        del g_new
        s.init()  # a clean DeTAG state for the legs below

    # ---- end to end through the host-buffer entry point: H2D of x, y, g, a, c and D2H of x, y, g every step
    e2e = None
    if not args.no_e2e:
        for k in ("y", "g"):
            host[k] = torch.empty((cfg.n, ld), dtype=torch.float32, pin_memory=pin)
        for k in ("x", "y", "g"):
            host[k].copy_(getattr(s, k))
        torch.cuda.synchronize(dev)
        chunk = 1 << 20
        while chunk > 128 and B.detag_host_staging_bytes(s.state, chunk) > (4 << 30):
            chunk >>= 1
        sbytes = B.detag_host_staging_bytes(s.state, chunk)
        staging = torch.empty(sbytes + 256, dtype=torch.uint8, device=dev)
        sptr = staging.data_ptr() + (-staging.data_ptr()) % 256
        e_steps = max(1, min(args.e2e_steps, args.steps))

        def host_step():
            B.detag_step_host(s.state, ld, host["x"], host["y"], host["g"], host["a"], host["c"], sptr, sbytes,
                              stream)

        host_step()  # warm-up
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e_steps):
            host_step()
        e1.record(stream)
        torch.cuda.synchronize(dev)
        te = sharding.reduce_max(e0.elapsed_time(e1), dist if world > 1 else None, dev)
        e2e = {"value": world * cfg.wc * e_steps / (te * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": 5 * 4 * cfg.wc, "d2h_bytes_per_step": 3 * 4 * cfg.wc, "steps": e_steps,
               "api": "detag_step_host (page-locked host state; chunked copy/step/copy on two streams)"}
        del staging

    line = None
    if rank == 0:
        peak, peak_src = measured_peak_gbs()
        kernel_ms = float(per_step.mean())
        achieved = BYTES_PER_WC * cfg.wc / (kernel_ms * 1e-3) / 1e9
        traffic = measured_traffic_bytes(variant, cfg.n, cfg.wc)
        key = kernel_key(variant, cfg.n)
        fp64, fp64_peak = None, None
        if key in FP64_FMA_PER_WC:  # second roofline: the FP64 pipe that carries both contractions
            fma = FP64_FMA_PER_WC[key] * cfg.wc / (kernel_ms * 1e-3)
            fp64_peak = FP64_FMA_PER_CLK_SM * SM_COUNT * (clocks.get("sm_max_mhz") or 1965) * 1e6
            fp64 = {"fma_per_wc": FP64_FMA_PER_WC[key], "achieved_tfma_s": fma / 1e12, "peak_tfma_s": fp64_peak / 1e12,
                    "frac": fma / fp64_peak, "peak_source": "64 FMA/clk/SM x 148 SMs x max SM clock"}
        line = {
            "metric": METRIC, "value": world * cfg.wc * args.steps / (total_ms_max * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": total_ms_max / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "n": cfg.n, "d": cfg.d, "K": cfg.K, "graph": cfg.graph,
                       "alpha": cfg.alpha, "sigma": cfg.sigma, "variant": variant,
                       "l2": f"state and objective arrays ({5 * 4 * cfg.wc / 1e9:.1f} GB per GPU) exceed the 126 MB L2"
                       if 20 * cfg.wc > 4 * 126e6 else "working set fits L2: not an HBM measurement",
                       "sharding": "each rank steps its own coordinate shard of d coordinates; no collective in the step"},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic, "peak_source": peak_src, "bytes_per_wc": BYTES_PER_WC,
                         "kernel_ms": kernel_ms, "kernel_ms_min": float(per_step.min()),
                         "kernel_ms_median": float(np.median(per_step)),
                         "frac_of_8TBps_nominal": achieved / 8000.0, "fp64_tensor_pipe": fp64},
            "clocks": clocks,
            "gpu_launches": args.steps,
            "consensus_error_after_run": consensus,
            "setup_s": t_setup,
        }
        if e2e is not None:
            line["e2e"] = e2e
        if multi is not None:
            if fp64_peak is not None:
                multi["fp64_tensor_pipe_frac"] = FP64_FMA_PER_WC[key] * multi["value"] / fp64_peak
            line["multi_step"] = multi
        if modes is not None:
            for v in modes.values():
                v["frac_of_measured_peak"] = v["achieved_gbs"] / peak
            line["modes"] = modes
    # the bench configuration's buffers go before the other configurations are set up
    s.close()
    del s, host
    torch.cuda.empty_cache()
    if rank == 0:
        if world == 1 and not args.no_per_config:
            line["per_config"] = [time_config(name, dev, args) for name in sorted(inputs.CONFIGS)
                                  if name != cfg.name or args.d]
            line["theorem3_regime"] = theorem3_regime(dev, args)
            line["general_graph"] = general_graph(dev, args)
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(inputs.CONFIGS[args.config], 10.0)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg5", choices=sorted(inputs.CONFIGS))
    ap.add_argument("--d", type=int, default=0, help="override the coordinate count (profiling a small case)")
    ap.add_argument("--variant", default="", choices=["", "csr", "dense", "ring", "torus"])
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--steps-per-launch", type=int, default=20,
                    help="also time detag_step_many with this many iterations per call (0: skip)")
    ap.add_argument("--multi-launches", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="skip the short runs of the other configurations")
    ap.add_argument("--no-modes", action="store_true", help="skip the D-PSGD and caller-written-gradient legs")
    ap.add_argument("--leg", default="", choices=["", "general_graph"], help="run this extra leg alone")
    ap.add_argument("--host-only", action="store_true",
                    help="multi-rank plumbing only (gloo, no CUDA call): what the CPU test of --gpus N runs")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        sys.exit(spawn_ranks(args.gpus))  # no launcher around this process: start the ranks here
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
    elif args.host_only:
        run_host_only(args, rank, world)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
