#!/usr/bin/env python
"""Benchmark of the fused parameter-server step (weighted aggregation + momentum SGD).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of the hot path over one batch of synthetic input: the host
controller chooses the batch sizes, then db_aggregate_update_ex combines the K
workers' gradients, applies the update and returns the squared gradient norm.
The workload is the ResNet-50-shaped one: 25,557,032 fp32 parameters in one arena,
K = 8 workers (4 fast, 4 slow), global batch 256, lr 0.1, mu 0.9.

Prints one JSON line (rank 0).  With several GPUs every rank runs an independent
replica of the same step (no data-path collective); `value` is all ranks' bytes over
the slowest rank's device time.  `--impl reference` times the fp64 CPU oracle instead.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2305_12213_b200 import inputs, replicas

METRIC = "aggregate+update HBM GB/s (% of B200 peak) and iterations/s at ResNet-50 size"
WORKLOAD = "resnet50_arena_N25557032_K8_fp32_gbatch256"
K_WORKERS = 8
N_PARAMS = inputs.RESNET50_N
THROUGHPUTS = [10.0] * 4 + [1.0] * 4
B0 = [32] * 8
KP, LR, MU = 1.0, 0.1, 0.9
GRAD_STD, PARAM_STD = 1e-3, 0.02
FALLBACK_HBM_GBS = 6650.0

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the aggregation kernel on this
# workload, from the ncu capture summarised under profiles/, with the digest of the kernel source
# the counters belong to.  Reported as null once the source has changed.
NCU_TRAFFIC = {"bytes_per_launch": 1200815616,
               "aggregate_cu_sha256": "a3bd1b313e6fbb98af38dea48f0e81ad2610b5b27e756cf20fc5ff0f69c4c2dc"}


def step_bytes(K: int, N: int, grad_bytes: int) -> int:
    """Algorithmic HBM bytes of one step: K gradient reads + read and write of params and momentum."""
    return K * N * grad_bytes + 4 * N * 4


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def kernel_traffic():
    src = os.path.join(ROOT, "paper_2305_12213_b200", "csrc", "aggregate.cu")
    try:
        digest = hashlib.sha256(open(src, "rb").read()).hexdigest()
    except OSError:
        return None
    if NCU_TRAFFIC["bytes_per_launch"] and digest == NCU_TRAFFIC["aggregate_cu_sha256"]:
        return NCU_TRAFFIC["bytes_per_launch"]
    return None


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while a region runs (read-only)."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int, period_s: float = 0.005):
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            if visible and visible.split(",")[index].strip().isdigit():
                index = int(visible.split(",")[index])
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------------------------
def run_ours(args):
    from paper_2305_12213_b200 import binding, build
    rank, local_rank, world = replicas.env_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; libdynbatch has no CPU fallback")
    dev = torch.device("cuda", local_rank if world > 1 else 0)
    torch.cuda.set_device(dev)
    replicas.init(device=dev)
    if rank == 0:
        build.build()
    replicas.barrier(dev)
    binding.lib()

    K, N = K_WORKERS, N_PARAMS
    seed = 2000 + 17 * rank
    grads = inputs.worker_gradients(K, N, GRAD_STD, seed, device=dev)
    p = inputs.normal(N, PARAM_STD, seed + 500, dev)
    v = torch.zeros(N, device=dev)
    sq = torch.zeros(1, dtype=torch.float64, device=dev)
    ws = torch.empty(binding.aggregate_workspace_bytes(K, N), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    b = list(B0)

    def step():
        nonlocal b
        b = binding.controller_step(b, THROUGHPUTS, KP)
        binding.aggregate_update(grads, b, p, v, LR, MU, sq, ws, stream)

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()

    # ---- timed region: device-resident inputs
    events = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    sampler = ClockSampler(dev.index)
    replicas.barrier(dev)
    torch.cuda.synchronize()
    with sampler:
        for i in range(args.steps):
            events[i].record(stream)
            step()
        events[args.steps].record(stream)
        torch.cuda.synchronize()
    replicas.barrier(dev)
    elapsed_ms = events[0].elapsed_time(events[args.steps])
    per_step_ms = [events[i].elapsed_time(events[i + 1]) for i in range(args.steps)]
    bytes_step = step_bytes(K, N, 4)
    job_bps, max_ms = replicas.job_throughput(bytes_step * args.steps, elapsed_ms, dev)
    final_sq = float(sq.item())
    assert np.isfinite(final_sq) and final_sq > 0 and bool(torch.isfinite(p[:1024]).all())

    # ---- end to end: gradients arrive in pinned host memory, parameters go back to the host
    e2e_steps = max(3, min(args.steps, 20))
    host_grads = [torch.empty(N, dtype=torch.float32).pin_memory() for _ in range(K)]
    for hg, g in zip(host_grads, grads):
        hg.copy_(g)
    host_p = torch.empty(N, dtype=torch.float32).pin_memory()
    host_sq = torch.empty(1, dtype=torch.float64).pin_memory()

    def e2e_step():
        nonlocal b
        for hg, g in zip(host_grads, grads):
            g.copy_(hg, non_blocking=True)
        b = binding.controller_step(b, THROUGHPUTS, KP)
        binding.aggregate_update(grads, b, p, v, LR, MU, sq, ws, stream)
        host_p.copy_(p, non_blocking=True)
        host_sq.copy_(sq, non_blocking=True)
        stream.synchronize()          # the step's result is on the host before the next one starts

    for _ in range(2):
        e2e_step()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    replicas.barrier(dev)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    torch.cuda.synchronize()
    replicas.barrier(dev)
    e2e_ms = e0.elapsed_time(e1)
    e2e_bps, _ = replicas.job_throughput(bytes_step * e2e_steps, e2e_ms, dev)

    peak, peak_kind = measured_peak()
    kernel_ms = float(np.mean(per_step_ms))
    achieved = bytes_step / (kernel_ms * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": job_bps / 1e9, "unit": "GB/s",
        "iterations_per_s": world * args.steps / (max_ms * 1e-3),
        "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
        "ms_per_step": max_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "K": K, "N": N, "grad_dtype": "f32", "global_batch": sum(B0),
                   "kp": KP, "lr": LR, "mu": MU, "grad_sqnorm": True,
                   "bytes_per_step": bytes_step, "l2": "inputs (1.23 GB per step) exceed the 126 MB L2",
                   "parallelism": f"{world} independent replica(s), no collective"},
        "e2e": {"value": e2e_bps / 1e9, "unit": "GB/s", "steps": e2e_steps,
                "ms_per_step": e2e_ms / e2e_steps,
                "h2d_bytes_per_step": K * N * 4, "d2h_bytes_per_step": N * 4 + 8},
        "gpu_launches": args.steps,
        "clocks": sampler.summary(),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": f"of {peak_kind}",
                     "kernel": "agg_vec_kernel<float, 8, 1, true>", "kernel_ms": kernel_ms,
                     "kernel_ms_min": float(np.min(per_step_ms)), "traffic": kernel_traffic()},
    }
    if rank == 0 and world == 1:
        del host_grads, host_p
        out["cpu_baseline"] = cpu_baseline([g.cpu().numpy() for g in grads], b)
    if rank == 0:
        print(json.dumps(out), flush=True)
    replicas.shutdown()


def cpu_baseline(host_grads, b, budget_s: float = 15.0):
    """The fp64 oracle, as it stands, on the host cores, over the same workload (all N, all K)."""
    import oracle
    N = host_grads[0].size
    p = inputs.normal(N, PARAM_STD, 1, "cpu").numpy().astype(np.float64)
    v = np.zeros(N, dtype=np.float64)
    oracle.aggregate_update(host_grads, b, p, v, LR, MU)          # warm-up pass
    t0 = time.perf_counter()
    passes = 0
    while passes < 3 or (time.perf_counter() - t0 < budget_s and passes < 50):
        oracle.aggregate_update(host_grads, b, p, v, LR, MU)
        passes += 1
    dt = time.perf_counter() - t0
    bytes_step = step_bytes(len(host_grads), N, 4)
    return {"value": bytes_step * passes / dt / 1e9, "unit": "GB/s", "cores": oracle.num_threads(),
            "kind": "oracle", "iterations_per_s": passes / dt,
            "sample": f"{passes} full passes of the workload (N={N}, K={len(host_grads)}), "
                      "fp64 state, OpenMP over elements"}


def run_reference(args):
    """The oracle on the host cores: each step is a bounded slice of the workload's parameters."""
    rank, _, _ = replicas.env_world()
    if rank != 0:
        return
    import oracle
    K, N = K_WORKERS, N_PARAMS
    steps, warm = args.steps, max(1, args.warmup)
    probe_n = 1 << 20
    host = [g.numpy() for g in inputs.worker_gradients(K, probe_n, GRAD_STD, 2000)]
    pp, vv = np.zeros(probe_n), np.zeros(probe_n)
    oracle.aggregate_update(host, B0, pp, vv, LR, MU)
    t0 = time.perf_counter()
    oracle.aggregate_update(host, B0, pp, vv, LR, MU)
    per_elem = (time.perf_counter() - t0) / probe_n
    n = int(min(N, max(1 << 16, 90.0 / (steps + warm) / per_elem)))
    host = [g.numpy() for g in inputs.worker_gradients(K, n, GRAD_STD, 2000)]
    p = inputs.normal(n, PARAM_STD, 2500).numpy().astype(np.float64)
    v = np.zeros(n)
    b = np.array(B0, dtype=np.int32)

    def step():
        nonlocal b
        b = oracle.controller_step(b, THROUGHPUTS, KP)
        oracle.aggregate_update(host, b, p, v, LR, MU)

    for _ in range(warm):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = time.perf_counter() - t0
    bytes_step = step_bytes(K, n, 4)
    val = bytes_step * steps / dt / 1e9
    sample = f"first {n} of {N} parameters per step, all K={K} workers, fp64 state"
    out = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s",
        "iterations_per_s": (n / N) * steps / dt,
        "n_gpus": args.gpus, "steps": steps, "warmup": warm, "ms_per_step": dt / steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "K": K, "N": N, "grad_dtype": "f32", "global_batch": sum(B0),
                   "kp": KP, "lr": LR, "mu": MU, "sample": sample},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    args = ap.parse_args()
    if args.steps < 1:
        raise SystemExit("--steps must be >= 1")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
