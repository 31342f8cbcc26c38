"""Multi-GPU plumbing for independent parameter-server replicas.

The aggregation step is element-wise over the parameters and this library runs
it on one GPU per parameter server; with several GPUs each process owns a whole
replica (its own K gradient buffers, parameters and momentum).  No data-path
collective exists: ranks only meet at a barrier and to combine their timings.
Works with NCCL (one rank per GPU) and with gloo on CPU.
"""
from __future__ import annotations

import os
from typing import Optional, Tuple

import torch
import torch.distributed as dist


def env_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) if unset."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: Optional[str] = None, device: Optional[torch.device] = None) -> Tuple[int, int]:
    """Join the process group when launched with more than one rank; returns (rank, world_size)."""
    rank, _, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        if backend is None:
            backend = "nccl" if (device is not None and device.type == "cuda") else "gloo"
        kwargs = {}
        if backend == "nccl" and device is not None:
            kwargs["device_id"] = device
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kwargs)
    return rank, world


def barrier(device: Optional[torch.device] = None) -> None:
    if dist.is_initialized() and dist.get_world_size() > 1:
        if device is not None and device.type == "cuda":
            dist.barrier(device_ids=[device.index])
        else:
            dist.barrier()


def _reduce(value: float, op, device: Optional[torch.device]) -> float:
    if not (dist.is_initialized() and dist.get_world_size() > 1):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(value: float, device: Optional[torch.device] = None) -> float:
    """Slowest rank's time: the job is as slow as its slowest replica."""
    return _reduce(value, dist.ReduceOp.MAX, device)


def sum_over_ranks(value: float, device: Optional[torch.device] = None) -> float:
    return _reduce(value, dist.ReduceOp.SUM, device)


def job_throughput(units_this_rank: float, elapsed_ms_this_rank: float,
                   device: Optional[torch.device] = None) -> Tuple[float, float]:
    """(units per second over all ranks, max elapsed ms): total units / slowest rank's time."""
    total = sum_over_ranks(units_this_rank, device)
    ms = max_over_ranks(elapsed_ms_this_rank, device)
    return total / (ms * 1e-3), ms


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
