#!/usr/bin/env python
"""Benchmark of the fused parameter-server step (weighted aggregation + momentum SGD).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload resnet50|bert_base|small|sweep|softmax]

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
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126 * 1024 * 1024
PARAM_STD = 0.02


class Workload:
    """One synthetic configuration of the step: K workers, N parameters, gradient dtype, controller inputs."""

    def __init__(self, name, K, N, grad_dtype, b0, throughputs, kp, lr, mu, grad_std):
        self.name, self.K, self.N, self.grad_dtype = name, K, N, grad_dtype
        self.b0, self.throughputs, self.kp, self.lr, self.mu, self.grad_std = b0, throughputs, kp, lr, mu, grad_std

    @property
    def grad_bytes(self):
        return 2 if self.grad_dtype == torch.bfloat16 else 4

    @property
    def bytes_per_step(self):
        return step_bytes(self.K, self.N, self.grad_bytes)

    @property
    def working_set(self):
        return self.K * self.N * self.grad_bytes + 2 * self.N * 4


def resnet50_workload():
    return Workload("resnet50_arena_N25557032_K8_fp32_gbatch256", 8, inputs.RESNET50_N, torch.float32,
                    [32] * 8, [10.0] * 4 + [1.0] * 4, 1.0, 0.1, 0.9, 1e-3)


def bert_base_workload():
    return Workload("bert_base_arena_N109482240_K16_bf16_gbatch512", 16, inputs.BERT_BASE_N, torch.bfloat16,
                    [32] * 16, inputs.lognormal_throughputs(16, 0.5, 4242), 1.0, 0.05, 0.9, 1e-3)


def small_workload():
    return Workload("small_N1048576_K3_fp32_gbatch128", 3, 1 << 20, torch.float32, [16, 32, 80],
                    [1.0, 2.0, 5.0], 0.5, 0.1, 0.9, 1.0)


def sweep_workloads(grad_dtype=torch.float32):
    out = []
    tag = "fp32" if grad_dtype == torch.float32 else "bf16"
    for n in (1 << 20, 1 << 22, 1 << 24, 1 << 26, 1 << 28):
        for k in (2, 4, 8, 16, 32):
            if n * k <= (1 << 33):
                b = inputs.batch_sizes_uniform(k, 8, 256, 5000 + k)
                # throughputs proportional to b: the controller step runs and holds b fixed
                out.append(Workload(f"sweep_N{n}_K{k}_{tag}", k, n, grad_dtype, b, [float(x) for x in b],
                                    1.0, 0.1, 0.9, 1.0))
    return out


WORKLOADS = {"resnet50": resnet50_workload, "bert_base": bert_base_workload, "small": small_workload}

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the aggregation kernel on the
# resnet50 workload, from the ncu capture summarised under profiles/, with the digest of the kernel
# sources (agg_kernels.cuh, agg_device.cuh) the counters belong to.  Reported as null once the source has changed.
NCU_TRAFFIC = {"workload": "resnet50_arena_N25557032_K8_fp32_gbatch256", "bytes_per_launch": 1022299392 + 179061504,
               "kernel_source_sha256": "102a1c7047db046edaeae11a7d165cc5883ca2431a7d4e2e43615bfd83c20af8"}


NOMINAL_HBM_GBS = 8000.0   # NVIDIA's published HBM3e figure for B200 (not verifiable here): context beside the measured peak


def copy_probe(dev, nbytes: int = 1 << 30, reps: int = 10) -> float:
    """GB/s (read + write) of a plain device-to-device copy of 1 GiB, timed like the steps."""
    src = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    dst = torch.empty_like(src)
    src.zero_()
    for _ in range(3):
        dst.copy_(src)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        dst.copy_(src)
    e1.record()
    torch.cuda.synchronize()
    return 2.0 * nbytes * reps / (e0.elapsed_time(e1) * 1e-3) / 1e9


def read_probe(dev, nbytes: int = 1 << 30, reps: int = 10) -> float:
    """GB/s of a pure read stream over 1 GiB (the library's own probe kernel, 128-bit streaming loads)."""
    from paper_2305_12213_b200 import binding
    src = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    src.zero_()
    sink = torch.empty(binding.bench_read_probe_sink_bytes(nbytes), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    for _ in range(3):
        binding.bench_read_probe(src, sink, stream)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(reps):
        binding.bench_read_probe(src, sink, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    return float(nbytes) * reps / (e0.elapsed_time(e1) * 1e-3) / 1e9


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


def kernel_traffic(workload_name):
    if workload_name != NCU_TRAFFIC["workload"]:
        return None
    h = hashlib.sha256()
    try:
        for name in ("agg_kernels.cuh", "agg_device.cuh"):
            with open(os.path.join(ROOT, "paper_2305_12213_b200", "csrc", name), "rb") as f:
                h.update(f.read())
    except OSError:
        return None
    if NCU_TRAFFIC["bytes_per_launch"] and h.hexdigest() == NCU_TRAFFIC["kernel_source_sha256"]:
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
        self._go = threading.Event()
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
            # the first queries of a process take milliseconds: make them here, not inside a timed region
            pynvml.nvmlDeviceGetClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            pynvml.nvmlDeviceGetCurrentClocksEventReasons(self.h)
        except Exception:
            self.nv = None
        if self.nv is not None:
            # the thread exists before the region opens, so that entering the region costs the timed thread
            # one Event.set() and not a thread start
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def _loop(self):
        nv = self.nv
        self._go.wait()
        # An NVML query pair costs the running stream about 10 us (measured: a 20-step region of 3.5 ms sampled
        # every millisecond ran 1 - 2.5 us per step slower than unsampled).  So: the first sample one millisecond
        # into the region, then one every `period`.
        self._stop.wait(0.001)
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
        self._go.set()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        self._go.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------------------------
def measure(wl, args, dev, rank, world, with_e2e=True, with_cpu=True):
    """Times `args.steps` steps of workload `wl` on `dev`; returns the JSON record (all ranks)."""
    from paper_2305_12213_b200 import binding
    K, N = wl.K, wl.N
    seed = 2000 + 17 * rank
    grads = inputs.worker_gradients(K, N, wl.grad_std, seed, device=dev, dtype=wl.grad_dtype)
    p = inputs.normal(N, PARAM_STD, seed + 500, dev)
    v = torch.zeros(N, device=dev)
    sq = torch.zeros(1, dtype=torch.float64, device=dev)
    ws = torch.empty(binding.aggregate_workspace_bytes(K, N), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    b = list(wl.b0)
    # inputs smaller than twice the L2 would be served from it on the next step: flush in between
    flush = None
    if wl.working_set < 2 * L2_BYTES:
        flush = torch.empty(2 * L2_BYTES // 4, dtype=torch.int32, device=dev)

    variant = getattr(args, "variant", "momentum")
    state_bytes = 16                      # p and v read and written
    kernel_label = "agg_vec_kernel"
    adam_t = 0
    if variant == "adam":
        u = torch.zeros(N, device=dev)    # second moment; v serves as the first
        state_bytes = 24
    elif variant == "tensor_list":
        if N not in (inputs.RESNET50_N, inputs.BERT_BASE_N):
            raise SystemExit("--variant tensor_list needs a workload with a tensor list (resnet50, bert_base)")
        # the same memory seen as the model's separately allocated tensors, one launch through a plan
        shapes = inputs.resnet50_tensor_shapes() if N == inputs.RESNET50_N else inputs.bert_base_tensor_shapes()
        offs = inputs.tensor_offsets(shapes)
        assert offs[-1] == N
        cut = lambda t: [t[s:e] for s, e in zip(offs[:-1], offs[1:])]
        plan = binding.MultiTensorPlan([cut(g) for g in grads], cut(p), cut(v))
        kernel_label = f"agg_multi_kernel over {len(shapes)} tensors"
    elif variant in ("persistent", "staged"):
        # the launch shapes that were measured against the kept kernel and not adopted (no norm)
        if wl.grad_dtype != torch.float32 or K not in (2, 4, 8, 16) or N % 4:
            raise SystemExit(f"--variant {variant} covers fp32 gradients, K in 2, 4, 8, 16 and N % 4 == 0")
        vstatus = torch.zeros(1, dtype=torch.int32, device=dev)
        kernel_label = "persistent_kernel" if variant == "persistent" else f"bulk_staged_kernel[{args.stage_floats} floats]"
    with_norm = variant in ("momentum", "adam", "tensor_list")

    if variant == "momentum":
        call = binding.AggregateStep(grads, p, v, sq, ws, stream)      # the tensors' pointers, marshalled once

    def step():
        nonlocal b, adam_t
        b = binding.controller_step(b, wl.throughputs, wl.kp)
        if variant == "momentum":
            call.run(b, wl.lr, wl.mu)
        elif variant == "adam":
            adam_t += 1
            binding.aggregate_adam(grads, b, p, v, u, 1e-3, 0.9, 0.999, 1e-8, adam_t, sq, ws, stream)
        elif variant == "tensor_list":
            plan.step(b, wl.lr, wl.mu, sq, stream)
        elif variant == "nonorm":
            binding.aggregate_update(grads, b, p, v, wl.lr, wl.mu, None, None, stream)
        elif variant in ("persistent", "staged"):
            binding.bench_aggregate_variant(
                binding.DB_BENCH_PERSISTENT if variant == "persistent" else binding.DB_BENCH_BULK_STAGED,
                args.stage_floats, grads, b, p, v, wl.lr, wl.mu, vstatus, stream)
        else:
            binding.aggregate_update(grads, b, p, v, wl.lr, wl.mu, sq, ws, stream)

    # the sampler (NVML handle, thread) is set up before the warm-up steps, so that nothing but the barrier
    # lies between the last warm-up step and the first timed one
    sampler = ClockSampler(dev.index)
    warmup = max(3, args.warmup)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()

    # ---- timed region: device-resident inputs, one event before and one after all steps
    steps = args.steps
    replicas.barrier(dev)
    torch.cuda.synchronize()
    if flush is None:
        e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_probe = min(steps, 200)
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_probe)]
        with sampler:             # the clocks are sampled through the timed region and the per-call pass behind it
            e_begin.record(stream)
            for _ in range(steps):
                step()
            e_end.record(stream)
            torch.cuda.synchronize()
            # the kernel's own duration: a second pass with an event pair around every call
            for e0, e1 in pairs:
                e0.record(stream)
                step()
                e1.record(stream)
            torch.cuda.synchronize()
        elapsed_ms = e_begin.elapsed_time(e_end)
        per_step_ms = [e0.elapsed_time(e1) for e0, e1 in pairs]
    else:
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        with sampler:
            for e0, e1 in pairs:
                # write 252 MB (evicts the step's lines), then read it back so that the L2 is left
                # holding clean lines and the timed kernel does not pay for their write-back
                flush.fill_(1)
                flush.sum()
                e0.record(stream)
                step()
                e1.record(stream)
            torch.cuda.synchronize()
        per_step_ms = [e0.elapsed_time(e1) for e0, e1 in pairs]
        elapsed_ms = float(np.sum(per_step_ms))
    replicas.barrier(dev)
    bytes_step = wl.K * wl.N * wl.grad_bytes + state_bytes * wl.N
    job_bps, max_ms = replicas.job_throughput(bytes_step * steps, elapsed_ms, dev)
    if with_norm:
        final_sq = float(sq.item())
        assert np.isfinite(final_sq) and final_sq > 0
    if variant in ("persistent", "staged"):
        assert int(vstatus.item()) == 0, "a staged CTA gave up waiting for its copies"
    assert bool(torch.isfinite(p[:1024]).all())

    peak, peak_kind = measured_peak()
    # The dominant kernel's launch duration, from CUDA events on its stream.  Back-to-back mode: the timed
    # region's time per step (aggregation kernel + the norm fold scheduled under it, so it slightly
    # overstates the kernel); the per-call probe also pays an event pair per step and loses the overlap of
    # consecutive steps, it is reported beside it.  Flushed mode: the event pair around each step.
    kernel_ms = elapsed_ms / steps if flush is None else float(np.mean(per_step_ms))
    achieved = bytes_step / (kernel_ms * 1e-3) / 1e9
    gname = "float" if wl.grad_dtype == torch.float32 else "__nv_bfloat16"
    launches = 2 if with_norm else 1
    out = {
        "metric": METRIC if variant == "momentum" else f"{METRIC} [{variant} variant of the step]",
        "value": job_bps / 1e9, "unit": "GB/s",
        "iterations_per_s": world * steps / (max_ms * 1e-3),
        "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": max_ms / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None,
        "dtype": "f32" if wl.grad_dtype == torch.float32 else "bf16 gradients, f32 accumulation and state",
        "data": "synthetic",
        "config": {"workload": wl.name if variant == "momentum" else f"{wl.name}_{variant}", "K": K, "N": N,
                   "grad_dtype": "f32" if wl.grad_dtype == torch.float32 else "bf16",
                   "global_batch": sum(wl.b0), "kp": wl.kp, "lr": wl.lr, "mu": wl.mu, "grad_sqnorm": with_norm,
                   "bytes_per_step": bytes_step,
                   "l2": ("inputs (%.2f GB per step) exceed the 126 MB L2" % (wl.working_set / 1e9)) if flush is None
                   else "L2 flushed (252 MB written, then read) before every timed step",
                   "parallelism": f"{world} independent replica(s), no collective"},
        # the aggregation kernel, plus the one-CTA fold of its norm partials scheduled under it
        "gpu_launches": launches * steps,
        "clocks": sampler.summary(),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": f"of {peak_kind}",
                     "kernel": f"{kernel_label}<{gname}, K={K if K <= 16 else 0}, {'norm' if with_norm else 'no norm'}, {'adam' if variant == 'adam' else 'momentum'}>",
                     "kernel_ms": kernel_ms,
                     "kernel_ms_probe_mean": float(np.mean(per_step_ms)),
                     "kernel_ms_min": float(np.min(per_step_ms)),
                     "traffic": kernel_traffic(wl.name) if variant == "momentum" else None},
    }
    out["roofline"]["frac_of_nominal"] = achieved / NOMINAL_HBM_GBS
    out["roofline"]["nominal_peak"] = NOMINAL_HBM_GBS
    if variant != "momentum":
        return out                        # the end-to-end and CPU legs belong to the headline step
    if flush is not None:
        out["graph_replay"] = graph_replay(wl, args, dev, grads, p, v, list(wl.b0))
    if with_e2e:
        # context only: this run's own device-to-device copy, the kind of measurement the peak file holds
        out["roofline"]["copy_probe_gbs"] = copy_probe(dev)
        out["roofline"]["read_probe_gbs"] = read_probe(dev)
        out["e2e"] = measure_e2e(wl, args, dev, grads, p, v, b)
    if with_cpu and rank == 0 and world == 1:
        out["cpu_baseline"] = cpu_baseline(wl, host_gradients(grads), b)
    return out


def graph_replay(wl, args, dev, grads, p, v, b):
    """Small workloads, second measurement: `steps` steps captured once in a CUDA graph and replayed, which
    takes the host's launch cost and the event pair per step out of the figure.  The steps rotate over enough
    copies of the inputs (gradients, parameters, momentum) to exceed twice the L2, so every step still meets
    its data in DRAM.  The controller runs on the host while the graph is built; its batch sizes are in the
    captured launches."""
    from paper_2305_12213_b200 import binding
    K, N = wl.K, wl.N
    sets = min(64, -(-2 * L2_BYTES // wl.working_set) + 1)
    gsets = [grads] + [[g.clone() for g in grads] for _ in range(sets - 1)]
    psets = [p] + [p.clone() for _ in range(sets - 1)]
    vsets = [v] + [v.clone() for _ in range(sets - 1)]
    sq = torch.zeros(1, dtype=torch.float64, device=dev)
    ws = torch.empty(binding.aggregate_workspace_bytes(K, N), dtype=torch.uint8, device=dev)
    steps = args.steps
    binding.aggregate_update(gsets[0], b, psets[0], vsets[0], wl.lr, wl.mu, sq, ws)      # not the first call in capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for s in range(steps):
            b = binding.controller_step(b, wl.throughputs, wl.kp)
            i = s % sets
            binding.aggregate_update(gsets[i], b, psets[i], vsets[i], wl.lr, wl.mu, sq, ws)
    graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 5
    times = []
    for _ in range(reps):
        e0.record()
        graph.replay()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / steps)
    assert np.isfinite(float(sq.item()))
    ms = float(np.median(times))
    peak, _ = measured_peak()
    gbs = wl.bytes_per_step / (ms * 1e-3) / 1e9
    return {"us_per_step": ms * 1e3, "us_per_step_min": float(np.min(times)) * 1e3, "GB/s": gbs, "frac": gbs / peak,
            "steps_per_replay": steps, "replays": reps, "input_sets": sets,
            "l2": "steps rotate over %d copies of the inputs (%.0f MB in all, the L2 holds 126 MB)"
                  % (sets, sets * wl.working_set / 1e6)}


def measure_e2e(wl, args, dev, grads, p, v, b):
    """The same step through db_aggregate_update_host: the gradients are in pinned host memory, the
    updated parameters and the norm come back to the host; all copies are inside the timed region."""
    from paper_2305_12213_b200 import binding
    K, N = wl.K, wl.N
    stream = torch.cuda.current_stream()
    e2e_steps = max(3, min(args.steps, 20))
    host_grads = [torch.empty(N, dtype=wl.grad_dtype).pin_memory() for _ in range(K)]
    for hg, g in zip(host_grads, grads):
        hg.copy_(g)
    host_p = torch.empty(N, dtype=torch.float32).pin_memory()
    host_sq = torch.zeros(1, dtype=torch.float64).pin_memory()
    pipe = binding.HostPipeline()
    staging = torch.empty(binding.host_staging_bytes(K, wl.grad_dtype, N, 0), dtype=torch.uint8, device=dev)
    b = list(b)

    def e2e_step():
        nonlocal b
        b = binding.controller_step(b, wl.throughputs, wl.kp)
        pipe.aggregate_update(host_grads, b, p, v, wl.lr, wl.mu, host_p, host_sq, staging, 0, stream)
        stream.synchronize()          # the step's result is on the host before the next one starts

    for _ in range(2):
        e2e_step()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(dev.index)
    replicas.barrier(dev)
    torch.cuda.synchronize()
    with sampler:
        e0.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        e1.record(stream)
        torch.cuda.synchronize()
    replicas.barrier(dev)
    e2e_ms = e0.elapsed_time(e1)
    assert np.isfinite(float(host_sq[0])) and float(host_sq[0]) > 0 and bool(torch.isfinite(host_p[:1024]).all())
    e2e_bps, e2e_max_ms = replicas.job_throughput(wl.bytes_per_step * e2e_steps, e2e_ms, dev)
    nchunks = -(-N // (1 << 21))
    pipe.close()
    return {"value": e2e_bps / 1e9, "unit": "GB/s", "steps": e2e_steps, "ms_per_step": e2e_max_ms / e2e_steps,
            "h2d_bytes_per_step": K * N * wl.grad_bytes, "d2h_bytes_per_step": N * 4 + 8,
            "api": "db_aggregate_update_host, 2^21-element chunks, pinned host buffers",
            "gpu_launches_per_step": nchunks + 1, "clocks": sampler.summary()}


def measure_softmax(args, dev, rank, world):
    """Config 3: the four ragged workers' linear-softmax gradients (one grouped call, tensor cores) and
    their batch-weighted aggregation + update.  Reported per step; not the headline metric."""
    from paper_2305_12213_b200 import binding
    bs, D, C = [24, 40, 64, 128], 2048, 1000
    X, y, W = inputs.softmax_problem(bs, D, C, seed=3000 + rank, device=dev)
    offs = [0] + list(np.cumsum(bs))
    G = [torch.empty(D, C, device=dev) for _ in bs]
    flat = [g.reshape(-1) for g in G]
    losses = torch.zeros(len(bs), device=dev)
    ws = torch.empty(binding.worker_grad_grouped_workspace_bytes(offs[-1], len(bs), D, C), dtype=torch.uint8,
                     device=dev)
    N = D * C
    p, v = inputs.normal(N, 0.01, 1, dev), torch.zeros(N, device=dev)
    sq = torch.zeros(1, dtype=torch.float64, device=dev)
    aws = torch.empty(binding.aggregate_workspace_bytes(len(bs), N), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    flush = torch.empty(2 * L2_BYTES // 4, dtype=torch.int32, device=dev)

    def step():
        binding.worker_grad_grouped(X, y, W, offs, G, losses, ws, stream)
        binding.aggregate_update(flat, bs, p, v, 0.1, 0.9, sq, aws, stream)

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    steps = args.steps
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    sampler = ClockSampler(dev.index)
    replicas.barrier(dev)
    with sampler:
        for e0, e1 in pairs:
            flush.fill_(1)
            flush.sum()
            e0.record(stream)
            step()
            e1.record(stream)
        torch.cuda.synchronize()
    replicas.barrier(dev)
    per_step_ms = [e0.elapsed_time(e1) for e0, e1 in pairs]
    assert binding.worker_grad_status(ws) == 0 and bool(torch.isfinite(losses).all())
    ms = float(np.mean(per_step_ms))
    steps_per_s, max_ms = replicas.job_throughput(steps, float(np.sum(per_step_ms)), dev)
    replay = softmax_graph_replay(args, dev, rank, bs, D, C) if world == 1 else None
    flops = 4.0 * sum(bs) * D * C                      # two contractions, 2 b D C multiply-adds each
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            bf16_peak, kind = float(json.load(f)["bf16_tflops"]), "measured bf16 burst x 1.1/2.25 (nominal TF32 : bf16)"
    except Exception:
        bf16_peak, kind = 1590.0, "fallback bf16 x 1.1/2.25 (nominal TF32 : bf16)"
    peak = bf16_peak * 1.1 / 2.25
    achieved = flops / (ms * 1e-3) / 1e12
    return {
        "metric": "ragged linear-softmax worker gradients + weighted aggregation, steps/s", "value": steps_per_s,
        "unit": "steps/s", "n_gpus": world, "steps": steps, "warmup": max(3, args.warmup),
        "ms_per_step": max_ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32 (three TF32 tensor-core products per fp32 product)", "data": "synthetic",
        "config": {"workload": "softmax_D2048_C1000_b24_40_64_128", "D": D, "C": C, "batch_sizes": bs,
                   "l2": "L2 flushed (252 MB written, then read) before every timed step",
                   "calls": "db_worker_grad_grouped + db_aggregate_update_ex"},
        # logits, softmax, gradients, aggregation, norm fold
        "gpu_launches": 5 * steps,
        "clocks": sampler.summary(),
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                     "frac": achieved / peak, "peak_source": kind,
                     "note": "algorithmic FLOPs 4*sum(b)*D*C per step; the step is launch- and latency-bound "
                             "(reduction depth b_i <= 128), the tensor pipe is idle most of the time",
                     "kernel": "logits_tma_kernel (logits) / grad_tma_kernel (gradients)", "kernel_ms": ms,
                     "kernel_ms_min": float(np.min(per_step_ms)), "traffic": None},
        "graph_replay": replay,
    }


def softmax_graph_replay(args, dev, rank, bs, D, C):
    """Config 3, second measurement: the steps issued back to back, as a training loop issues them, captured
    once in a CUDA graph and replayed -- no event pair and no host launch cost per step, and each step's first
    kernel is scheduled under the previous step's last.  The steps rotate over enough complete copies of the
    problem (samples, labels, parameters, momentum, gradient buffers, workspaces) to exceed twice the L2, so
    every step still meets its data in DRAM."""
    from paper_2305_12213_b200 import binding
    offs = [0] + list(np.cumsum(bs))
    N = D * C
    ws_bytes = binding.worker_grad_grouped_workspace_bytes(offs[-1], len(bs), D, C)
    per_set = int(4 * (int(offs[-1]) * D + (3 + len(bs)) * N) + ws_bytes)
    sets = int(min(16, -(-2 * L2_BYTES // per_set) + 1))
    probs = []
    for i in range(sets):
        X, y, W = inputs.softmax_problem(bs, D, C, seed=3000 + rank + 17 * i, device=dev)
        G = [torch.empty(D, C, device=dev) for _ in bs]
        probs.append(dict(X=X, y=y, p=inputs.normal(N, 0.01, 1 + i, dev), W=W, G=G, flat=[g.reshape(-1) for g in G],
                          v=torch.zeros(N, device=dev), losses=torch.zeros(len(bs), device=dev),
                          ws=torch.empty(ws_bytes, dtype=torch.uint8, device=dev),
                          aws=torch.empty(binding.aggregate_workspace_bytes(len(bs), N), dtype=torch.uint8,
                                          device=dev)))
    sq = torch.zeros(1, dtype=torch.float64, device=dev)

    def step(q, stream):
        binding.worker_grad_grouped(q["X"], q["y"], q["W"], offs, q["G"], q["losses"], q["ws"], stream)
        binding.aggregate_update(q["flat"], bs, q["p"], q["v"], 0.1, 0.9, sq, q["aws"], stream)

    for q in probs:
        step(q, torch.cuda.current_stream())                  # not the first call in capture
    torch.cuda.synchronize()
    steps = args.steps
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for s_ in range(steps):
            step(probs[s_ % sets], torch.cuda.current_stream())
    graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    times = []
    for _ in range(5):
        e0.record()
        graph.replay()
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / steps)
    ok = all(binding.worker_grad_status(q["ws"]) == 0 and bool(torch.isfinite(q["losses"]).all()) for q in probs)
    assert ok and np.isfinite(float(sq.item()))
    ms = float(np.median(times))
    return {"us_per_step": ms * 1e3, "us_per_step_min": float(np.min(times)) * 1e3, "steps_per_s": 1e3 / ms,
            "steps_per_replay": steps, "replays": 5, "input_sets": sets,
            "l2": "steps rotate over %d complete copies of the problem (%.0f MB in all, the L2 holds 126 MB)"
                  % (sets, sets * per_set / 1e6)}


def measure_sharded(args, dev, rank, world):
    """Opt-in: the ResNet-50-shaped step with one parameter server per GPU (sharded.ShardedServer): every rank
    hosts K / world of the workers' gradient buffers and owns 1 / world of the parameters; per step a barrier,
    the fused kernel on the slice (peer loads for the other ranks' workers), an all-gather of the parameters and
    an all-reduce of the norm.  Strong scaling: the job is one model, whatever the number of GPUs."""
    from paper_2305_12213_b200 import binding, sharded
    wl = resnet50_workload()
    if wl.K % world:
        raise SystemExit(f"--mode sharded: {wl.K} workers do not divide over {world} ranks")
    k_local = wl.K // world
    local = inputs.worker_gradients(k_local, wl.N, wl.grad_std, 2000 + 100 * rank, device=dev, dtype=wl.grad_dtype)
    p0 = inputs.normal(wl.N, PARAM_STD, 2500, dev)
    server = sharded.ShardedServer(local, p0)
    b = list(wl.b0)
    stream = torch.cuda.current_stream()

    def step():
        nonlocal b
        b = binding.controller_step(b, wl.throughputs, wl.kp)
        server.step(b, wl.lr, wl.mu)

    warmup = max(3, args.warmup)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(dev.index)
    replicas.barrier(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with sampler:
        e0.record(stream)
        for _ in range(args.steps):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
    replicas.barrier(dev)
    ms = replicas.max_over_ranks(e0.elapsed_time(e1), dev)
    bytes_step = wl.bytes_per_step                       # the whole job's step, not per rank
    sq = float(server.sqnorm.item())
    assert np.isfinite(sq) and sq > 0
    peak, peak_kind = measured_peak()
    achieved = bytes_step / world / (ms / args.steps * 1e-3) / 1e9
    return {
        "metric": f"{METRIC} [one parameter server per GPU]", "value": bytes_step * args.steps / (ms * 1e-3) / 1e9,
        "unit": "GB/s", "iterations_per_s": args.steps / (ms * 1e-3), "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "strong",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name + "_sharded", "K": wl.K, "N": wl.N, "servers": world,
                   "parallelism": f"{world} parameter server(s), each owning N/{world} of params and momentum; "
                                  "gradients read through peer mappings; barrier + all-gather(params) + "
                                  "all-reduce(norm) per step",
                   "l2": "inputs exceed the 126 MB L2"},
        "gpu_launches": 2 * args.steps, "clocks": sampler.summary(),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_source": f"of {peak_kind}", "kernel": "agg_vec_kernel on this rank's slice; the step "
                     "also contains the collectives, so this is a lower bound of the kernel's own rate",
                     "traffic": None},
    }


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
    if args.mode == "sharded":
        out = measure_sharded(args, dev, rank, world)
        if rank == 0:
            print(json.dumps(out), flush=True)
    elif args.workload == "softmax":
        out = measure_softmax(args, dev, rank, world)
        if rank == 0:
            print(json.dumps(out), flush=True)
    elif args.workload == "sweep":
        points = sweep_workloads(torch.bfloat16 if args.sweep_dtype == "bf16" else torch.float32)
        if args.sweep_point:
            n_sel, k_sel = (int(x) for x in args.sweep_point.split(","))
            points = [w for w in points if w.N == n_sel and w.K == k_sel]
            if not points:
                raise SystemExit("--sweep-point: no such point (N in 2^20..2^28 by 4x, K in 2,4,8,16,32, K*N <= 2^33)")
        for wl in points:
            out = measure(wl, args, dev, rank, world, with_e2e=False, with_cpu=False)
            if rank == 0:
                print(json.dumps(out), flush=True)
            torch.cuda.empty_cache()
    else:
        out = measure(WORKLOADS[args.workload](), args, dev, rank, world)
        if rank == 0:
            print(json.dumps(out), flush=True)
    replicas.shutdown()


def host_gradients(grads):
    """Device gradient tensors -> the numpy arrays the oracle takes (fp32, or uint16 bf16 bit patterns)."""
    out = []
    for g in grads:
        t = g.detach().cpu().contiguous()
        out.append(t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy())
    return out


def cpu_baseline(wl, host_grads, b, budget_s: float = 12.0):
    """The fp64 oracle, as it stands, on the host cores, over the same workload (all N, all K): with all
    cores, and with one thread."""
    import oracle
    N = wl.N
    p = inputs.normal(N, PARAM_STD, 1, "cpu").numpy().astype(np.float64)
    v = np.zeros(N, dtype=np.float64)
    all_threads = oracle.num_threads()

    def timed(threads, budget, min_passes):
        oracle.set_num_threads(threads)
        oracle.aggregate_update(host_grads, b, p, v, wl.lr, wl.mu)          # warm-up pass
        t0 = time.perf_counter()
        passes = 0
        while passes < min_passes or (time.perf_counter() - t0 < budget and passes < 50):
            oracle.aggregate_update(host_grads, b, p, v, wl.lr, wl.mu)
            passes += 1
        dt = time.perf_counter() - t0
        return passes, dt

    try:
        passes, dt = timed(all_threads, budget_s, 3)
        passes1, dt1 = timed(1, budget_s / 2, 1)
    finally:
        oracle.set_num_threads(all_threads)
    return {"value": wl.bytes_per_step * passes / dt / 1e9, "unit": "GB/s", "cores": all_threads,
            "kind": "oracle", "iterations_per_s": passes / dt, "ms_per_iteration": dt / passes * 1e3,
            "sample": f"{passes} full passes of the workload (N={N}, K={wl.K}), "
                      "fp64 state, OpenMP over elements",
            "single_thread": {"value": wl.bytes_per_step * passes1 / dt1 / 1e9, "unit": "GB/s", "cores": 1,
                              "ms_per_iteration": dt1 / passes1 * 1e3,
                              "sample": f"{passes1} full pass(es) of the same workload"}}


def run_reference(args):
    """The oracle on the host cores: each step is a bounded slice of the workload's parameters."""
    rank, _, _ = replicas.env_world()
    if rank != 0:
        return
    import oracle
    wl = WORKLOADS[args.workload if args.workload in WORKLOADS else "resnet50"]()
    K, N = wl.K, wl.N
    steps, warm = args.steps, max(1, args.warmup)
    probe_n = 1 << 20
    host = host_gradients(inputs.worker_gradients(K, probe_n, wl.grad_std, 2000, dtype=wl.grad_dtype))
    pp, vv = np.zeros(probe_n), np.zeros(probe_n)
    oracle.aggregate_update(host, wl.b0, pp, vv, wl.lr, wl.mu)
    t0 = time.perf_counter()
    oracle.aggregate_update(host, wl.b0, pp, vv, wl.lr, wl.mu)
    per_elem = (time.perf_counter() - t0) / probe_n
    n = int(min(N, max(1 << 16, 90.0 / (steps + warm) / per_elem)))
    host = host_gradients(inputs.worker_gradients(K, n, wl.grad_std, 2000, dtype=wl.grad_dtype))
    p = inputs.normal(n, PARAM_STD, 2500).numpy().astype(np.float64)
    v = np.zeros(n)
    b = np.array(wl.b0, dtype=np.int32)

    def step():
        nonlocal b
        b = oracle.controller_step(b, wl.throughputs, wl.kp)
        oracle.aggregate_update(host, b, p, v, wl.lr, wl.mu)

    for _ in range(warm):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = time.perf_counter() - t0
    val = step_bytes(K, n, wl.grad_bytes) * steps / dt / 1e9
    sample = f"first {n} of {N} parameters per step, all K={K} workers, fp64 state"
    # the same sample once on a single thread, outside the timed region
    all_threads = oracle.num_threads()
    oracle.set_num_threads(1)
    try:
        t1 = time.perf_counter()
        step()
        dt1 = time.perf_counter() - t1
    finally:
        oracle.set_num_threads(all_threads)
    out = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s",
        "iterations_per_s": (n / N) * steps / dt,
        "n_gpus": args.gpus, "steps": steps, "warmup": warm, "ms_per_step": dt / steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": wl.name, "K": K, "N": N,
                   "grad_dtype": "f32" if wl.grad_dtype == torch.float32 else "bf16",
                   "global_batch": sum(wl.b0), "kp": wl.kp, "lr": wl.lr, "mu": wl.mu, "sample": sample},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": all_threads, "kind": "oracle",
                         "sample": sample,
                         "single_thread": {"value": step_bytes(K, n, wl.grad_bytes) / dt1 / 1e9, "unit": "GB/s",
                                           "cores": 1, "sample": "one step of the same sample"}},
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
    ap.add_argument("--variant", choices=["momentum", "adam", "tensor_list", "nonorm", "persistent", "staged"],
                    default="momentum",
                    help="the step's optimizer / entry point: momentum = db_aggregate_update_ex (headline), adam = "
                         "db_aggregate_adam_ex, tensor_list = db_aggregate_update_multi over the model's separate "
                         "tensors (resnet50, bert_base); nonorm = the headline kernel without the gradient norm, "
                         "persistent / staged = the launch shapes measured against it and not adopted "
                         "(db_bench_aggregate_variant; fp32, no norm)")
    ap.add_argument("--mode", choices=["replicas", "sharded"], default="replicas",
                    help="with several GPUs: replicas = every rank runs its own independent step (default, no "
                         "collective on the data path); sharded = one parameter server per GPU, each owning a slice "
                         "of the model (paper_2305_12213_b200.sharded), resnet50 workload only")
    ap.add_argument("--stage-floats", type=int, choices=[512, 1024, 2048], default=512,
                    help="with --variant staged: floats per stream and CTA staged in shared memory")
    ap.add_argument("--sweep-dtype", choices=["fp32", "bf16"], default="fp32",
                    help="gradient storage of the sweep's points (the named sweep configuration is fp32)")
    ap.add_argument("--sweep-point", default="", metavar="N,K",
                    help="with --workload sweep: run only this point (e.g. 67108864,2), for profiler captures")
    ap.add_argument("--workload", choices=["resnet50", "bert_base", "small", "sweep", "softmax"], default="resnet50",
                    help="resnet50 is the headline configuration; sweep prints one line per (N, K) point")
    args = ap.parse_args()
    if args.steps < 1:
        raise SystemExit("--steps must be >= 1")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
