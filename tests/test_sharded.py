"""Several parameter servers (opt-in): slice arithmetic, the collectives' plumbing on gloo, and -- on a GPU --
the whole step with two server processes reading each other's gradient buffers through peer mappings."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

from paper_2305_12213_b200 import binding, build, inputs


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("N", [0, 1, 7, 8, 9, 1000, 1 << 20, inputs.RESNET50_N, inputs.BERT_BASE_N])
@pytest.mark.parametrize("G", [1, 2, 3, 8])
def test_slices_tile_the_parameters(N, G):
    build.build()
    from paper_2305_12213_b200 import sharded
    cuts = [binding.shard_range(N, G, r) for r in range(G)]
    assert cuts[0][0] == 0 and cuts[-1][1] == N
    for (a, b), (c, d) in zip(cuts[:-1], cuts[1:]):
        assert b == c and a <= b
    chunk = sharded.chunk_elems(N, G)
    assert chunk % 8 == 0 and chunk * G >= N
    for r, (a, b) in enumerate(cuts):
        assert a == min(r * chunk, N) and b == min((r + 1) * chunk, N)
    with pytest.raises(binding.DynbatchError):
        binding.shard_range(N, G, G)
    with pytest.raises(binding.DynbatchError):
        binding.shard_range(-1, G, 0)


def _gloo_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch.distributed as dist
    from paper_2305_12213_b200 import sharded
    dist.init_process_group("gloo", rank=rank, world_size=world)
    N = 1003
    chunk = sharded.chunk_elems(N, world)
    full = torch.zeros(chunk * world)
    lo, hi = binding.shard_range(N, world, rank)
    full[lo:hi] = torch.arange(lo, hi, dtype=torch.float32) + 1.0      # this server's updated slice
    sharded.all_gather_slices(full, chunk)
    sq = torch.tensor([float(rank + 1)], dtype=torch.float64)
    sharded.all_reduce_sum(sq)
    out.put((rank, bool(torch.equal(full[:N], torch.arange(N, dtype=torch.float32) + 1.0)), float(sq.item())))
    dist.barrier()
    dist.destroy_process_group()


def test_collectives_plumbing_on_gloo():
    build.build()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    world = 3
    procs = [ctx.Process(target=_gloo_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(r, True, 6.0) for r in range(world)]


def _server_worker(rank, world, port, out):
    """Both servers share one GPU here (one GPU per test machine): the peer mappings, the slices, the gather
    and the norm's reduction are the ones a node with one GPU per server uses; only NCCL is replaced by gloo."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch.distributed as dist
    from paper_2305_12213_b200 import sharded
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    N, K_local = 3_000_017, 2
    K = K_local * world
    b = [5, 9, 0, 18][:K] if K <= 4 else list(range(1, K + 1))
    local = [inputs.normal(N, 1e-3, 100 + 10 * rank + k, dev) for k in range(K_local)]
    p0 = inputs.normal(N, 0.02, 7, dev)
    server = sharded.ShardedServer(local, p0)
    assert server.K == K
    sq_steps = []
    for step in range(2):
        sq = server.step(b, 0.1, 0.9)
        sq_steps.append(float(sq.item()))
        for g in local:                       # the workers' next gradients, written only after the step's gather
            g.mul_(0.5)
    torch.cuda.synchronize()
    # the same two steps as one flat call over all N, from the same gradients (regenerated locally)
    allg = [inputs.normal(N, 1e-3, 100 + 10 * r + k, dev) for r in range(world) for k in range(K_local)]
    p, v = p0.clone(), torch.zeros(N, device=dev)
    ref_sq = torch.zeros(1, dtype=torch.float64, device=dev)
    ws = torch.empty(binding.aggregate_workspace_bytes(K, N), dtype=torch.uint8, device=dev)
    flat_sq = []
    for step in range(2):
        binding.aggregate_update(allg, b, p, v, 0.1, 0.9, ref_sq, ws)
        flat_sq.append(float(ref_sq.item()))
        for g in allg:
            g.mul_(0.5)
    torch.cuda.synchronize()
    lo, hi = server.begin, server.end
    ok = bool(torch.equal(server.params, p)) and bool(torch.equal(server.momentum, v[lo:hi]))
    rel = max(abs(a - c) / c for a, c in zip(sq_steps, flat_sq))
    out.put((rank, ok, rel))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.gpu
def test_two_servers_reproduce_the_one_gpu_step_bit_for_bit():
    build.build()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_server_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=300) for _ in procs)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    for rank, ok, rel in res:
        assert ok, f"server {rank}: parameters or momentum differ from the flat call"
        assert rel < 1e-12


@pytest.mark.gpu
def test_slices_on_one_gpu_equal_the_flat_call():
    """G calls on the G slices of one GPU's buffers: the arithmetic of the sharded form without processes."""
    dev = "cuda"
    N, K, G = 1_000_003, 5, 3
    b = [3, 9, 0, 18, 5]
    g = inputs.worker_gradients(K, N, 1e-3, 300, device=dev, dtype=torch.bfloat16)
    p0, v0 = inputs.normal(N, 0.02, 31, dev), inputs.normal(N, 0.01, 32, dev)
    p1, v1, p2, v2 = p0.clone(), v0.clone(), p0.clone(), v0.clone()
    sq1 = torch.zeros(1, dtype=torch.float64, device=dev)
    binding.aggregate_update(g, b, p1, v1, 0.1, 0.9, sq1,
                             torch.empty(binding.aggregate_workspace_bytes(K, N), dtype=torch.uint8, device=dev))
    total = 0.0
    for r in range(G):
        lo, hi = binding.shard_range(N, G, r)
        sq = torch.zeros(1, dtype=torch.float64, device=dev)
        ws = torch.empty(binding.aggregate_workspace_bytes(K, hi - lo), dtype=torch.uint8, device=dev)
        binding.aggregate_update([t[lo:hi] for t in g], b, p2[lo:hi], v2[lo:hi], 0.1, 0.9, sq, ws)
        total += float(sq.item())
    torch.cuda.synchronize()
    assert torch.equal(p1, p2) and torch.equal(v1, v2)
    assert abs(total - float(sq1.item())) <= 1e-12 * float(sq1.item())
