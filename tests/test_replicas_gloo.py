"""world_size-2 gloo test of the replica plumbing the multi-GPU benchmark uses."""
import os
import socket

import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2305_12213_b200 import binding, replicas
    r, w = replicas.init(backend="gloo")
    assert (r, w) == (rank, world)
    replicas.barrier()
    # each replica runs its own controller trajectory (host side of the step); no data is exchanged
    b = binding.controller_step([32] * 4, [1.0 + rank, 2.0, 3.0, 4.0], 1.0)
    assert sum(b) == 128
    slow_ms = 10.0 * (rank + 1)
    thr, ms = replicas.job_throughput(units_this_rank=100.0 * (rank + 1), elapsed_ms_this_rank=slow_ms)
    out.put((rank, thr, ms, replicas.max_over_ranks(float(rank)), replicas.sum_over_ranks(1.0), b))
    replicas.barrier()
    replicas.shutdown()


def test_two_replicas_combine_timings_without_data_exchange():
    from paper_2305_12213_b200 import build
    build.build()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, thr, ms, mx, sm, b in res:
        assert ms == 20.0 and mx == 1.0 and sm == 2.0
        assert abs(thr - 300.0 / 0.020) < 1e-6          # all units / slowest rank
    assert res[0][5] != res[1][5]                         # replicas are independent


def test_single_process_is_a_no_op():
    from paper_2305_12213_b200 import replicas
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert replicas.init() == (0, 1)
    replicas.barrier()
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.job_throughput(50.0, 10.0) == (5000.0, 10.0)
