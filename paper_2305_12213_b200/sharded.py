"""Several parameter servers on the GPUs of one node (opt-in; the default multi-GPU mode is independent replicas).

The paper scales the number of parameter servers with the job (Section 4, experimental setup).  The step is
element-wise over the parameters, so server r of G owns one contiguous slice of params and momentum
(`binding.shard_range`) and runs the ordinary fused kernel on it: `db_aggregate_update_ex` with grads[k]
pointing at that slice of worker k's gradient buffer.  The workers' buffers live on the GPU that hosts the
worker; a server reads the slices of the other GPUs' workers through peer mappings of those buffers (CUDA IPC
handles exchanged once), with the kernel's own 128-bit loads -- no copy kernel, no TMA, no library kernel is
given a peer's memory.  Per step the ranks meet three times through `torch.distributed`:
  1. a barrier: every worker's gradients are written before any server reads them;
  2. an all-gather of the updated parameter slices, so that every GPU holds the whole model again (it also
     tells every rank that all servers have finished reading its gradient buffers);
  3. an all-reduce of the squared gradient norm (a scalar), when it is wanted.
Results are bit-identical to the one-GPU call over all N parameters; the norm is the sum of the slices' norms.

Collectives run on NCCL (one rank per GPU) or, for tests, on gloo through host copies.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch
import torch.distributed as dist

from . import binding


def chunk_elems(N: int, G: int, align: int = 8) -> int:
    """Stride between the servers' slices: ceil(N / G) rounded up to `align` elements, the rule of
    db_shard_range (whose slices are this long except for the last, shorter or empty ones)."""
    per = -(-N // G)
    return -(-per // align) * align


def _rank_world(group=None):
    """(rank, world) of the process group; (0, 1) when no group has been set up (one server)."""
    if not dist.is_initialized():
        return 0, 1
    return dist.get_rank(group), dist.get_world_size(group)


def exchange_gradient_buffers(local: Sequence[torch.Tensor], group=None) -> List[torch.Tensor]:
    """All workers' gradient buffers as tensors this process can hand to its kernels, in rank-major worker
    order: this rank's own tensors, and peer mappings (CUDA IPC) of the other ranks'.  Called once; the
    returned tensors alias the owners' memory."""
    from torch.multiprocessing.reductions import reduce_tensor
    rank, world = _rank_world(group)
    if world == 1:
        return list(local)
    mine = [reduce_tensor(t) for t in local]
    everyone: List[Optional[list]] = [None] * world
    dist.all_gather_object(everyone, mine, group=group)
    out: List[torch.Tensor] = []
    for r, handles in enumerate(everyone):
        if r == rank:
            out.extend(local)
        else:
            out.extend(rebuild(*args) for rebuild, args in handles)
    return out


def all_gather_slices(full_padded: torch.Tensor, chunk: int, group=None) -> None:
    """full_padded[r * chunk : (r + 1) * chunk] of every rank r -> the same range of every rank's tensor."""
    rank, world = _rank_world(group)
    if world == 1 or chunk == 0:
        return
    mine = full_padded[rank * chunk:(rank + 1) * chunk]
    if full_padded.is_cuda and dist.get_backend(group) == "nccl":
        send = mine.clone()                         # the gather's input may not alias its output
        dist.all_gather_into_tensor(full_padded, send, group=group)
        return
    # gloo (tests): through host memory
    host = mine.detach().cpu()
    parts = [torch.empty_like(host) for _ in range(world)]
    dist.all_gather(parts, host, group=group)
    for r, part in enumerate(parts):
        if r != rank:
            full_padded[r * chunk:(r + 1) * chunk].copy_(part)


def all_reduce_sum(value: torch.Tensor, group=None) -> None:
    """In-place sum over the ranks of a small tensor (the squared gradient norm)."""
    if _rank_world(group)[1] == 1:
        return
    if value.is_cuda and dist.get_backend(group) == "nccl":
        dist.all_reduce(value, group=group)
        return
    host = value.detach().cpu()
    dist.all_reduce(host, group=group)
    value.copy_(host)


def device_barrier(device: torch.device, group=None) -> None:
    """Every rank's work enqueued so far on `device` has finished before any rank goes on."""
    if _rank_world(group)[1] == 1:
        return
    if dist.get_backend(group) == "nccl":
        dist.barrier(group=group, device_ids=[device.index])
    else:
        torch.cuda.synchronize(device)
        dist.barrier(group=group)


class ShardedServer:
    """Parameter server `rank` of `world`: owns a slice of momentum, keeps the whole parameter vector.

    local_grads   this rank's workers' gradient buffers (N elements each, fp32 or bf16, same count and dtype on
                  every rank); the workers write them before each step
    params        N fp32 initial parameters (identical on every rank); kept, padded, in `self.params`
    """

    def __init__(self, local_grads: Sequence[torch.Tensor], params: torch.Tensor, group=None):
        self.group = group
        self.rank, self.world = _rank_world(group)
        self.device = params.device
        self.N = params.numel()
        for g in local_grads:
            if g.numel() != self.N or g.device != self.device:
                raise ValueError("every gradient buffer holds N elements on this rank's device")
        self.chunk = chunk_elems(self.N, self.world)
        self.begin, self.end = binding.shard_range(self.N, self.world, self.rank)
        self._padded = torch.zeros(max(self.chunk * self.world, self.N), dtype=torch.float32, device=self.device)
        self._padded[:self.N].copy_(params)
        self.params = self._padded[:self.N]
        self.momentum = torch.zeros(self.end - self.begin, dtype=torch.float32, device=self.device)
        self.grads = exchange_gradient_buffers(list(local_grads), group)
        self.K = len(self.grads)
        self.sqnorm = torch.zeros(1, dtype=torch.float64, device=self.device)
        n_slice = self.end - self.begin
        self._workspace = torch.empty(binding.aggregate_workspace_bytes(self.K, n_slice), dtype=torch.uint8,
                                      device=self.device)

    def step(self, b: Sequence[int], lr: float, mu: float, want_norm: bool = True) -> Optional[torch.Tensor]:
        """One parameter-server step over all K workers' gradients; returns the squared gradient norm
        (device tensor, valid on every rank) when wanted."""
        if len(b) != self.K:
            raise ValueError("one batch size per worker of the whole job")
        device_barrier(self.device, self.group)
        lo, hi = self.begin, self.end
        if hi > lo:
            binding.aggregate_update([g[lo:hi] for g in self.grads], b, self.params[lo:hi], self.momentum, lr, mu,
                                     self.sqnorm if want_norm else None, self._workspace if want_norm else None)
        elif want_norm:
            self.sqnorm.zero_()
        all_gather_slices(self._padded, self.chunk, self.group)
        if want_norm:
            all_reduce_sum(self.sqnorm, self.group)
            return self.sqnorm
        return None
