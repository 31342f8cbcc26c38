"""GPU parity of db_worker_grad against the fp64 oracle, and the closed-form check that the
batch-weighted aggregate of per-worker gradients is the gradient of the concatenated batch."""
import numpy as np
import pytest
import torch

import oracle
from helpers import FP32_TOL, f64, rel_err
from paper_2305_12213_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


TENSOR, FFMA = 0, binding.DB_WORKER_GRAD_FFMA


def _worker_grad(X, y, W, flags=TENSOR):
    b_i, D = X.shape
    C = W.shape[1]
    G = torch.full((D, C), float("nan"), device=DEV)
    loss = torch.zeros(1, device=DEV)
    ws = torch.empty(binding.worker_grad_workspace_bytes(b_i, D, C), dtype=torch.uint8, device=DEV)
    binding.worker_grad(X, y, W, G, loss, ws, flags=flags)
    torch.cuda.synchronize()
    assert binding.worker_grad_status(ws) == 0, "a bounded wait inside the tensor-core kernel gave up"
    return G, float(loss.item())


@pytest.mark.parametrize("flags", [TENSOR, FFMA])
@pytest.mark.parametrize("b_i,D,C", [(1, 4, 4), (5, 6, 3), (7, 33, 10), (24, 128, 64), (3, 257, 130),
                                      (65, 200, 96), (130, 64, 1000), (40, 2048, 1000), (33, 100, 129),
                                      (300, 96, 40), (128, 2048, 1000)])
def test_shapes_including_ragged_tiles(b_i, D, C, flags):
    X, y, W = inputs.softmax_problem([b_i], D, C, seed=100 + b_i, w_std=0.05, device=DEV)
    G, loss = _worker_grad(X, y, W, flags)
    rG, rloss = oracle.worker_grad(X.cpu().numpy(), y.cpu().numpy(), W.cpu().numpy())
    assert rel_err(f64(G), rG) <= FP32_TOL
    assert abs(loss - rloss) <= FP32_TOL * abs(rloss)
    assert float(G.double().sum(dim=1).abs().max()) < 1e-5      # rows of P - Y sum to zero


def test_out_of_range_label_contributes_no_onehot():
    X, y, W = inputs.softmax_problem([4], 16, 8, seed=7, w_std=0.1, device=DEV)
    y2 = y.clone()
    y2[1] = 99
    G, _ = _worker_grad(X, y2, W, FFMA)
    # the row sums of P alone are 1: column-sum identity is broken exactly by sample 1's features
    excess = G.double().sum(dim=1) * 4
    assert rel_err(excess.cpu().numpy(), f64(X[1])) <= 1e-5


def test_misaligned_inputs_take_the_element_wise_loaders():
    b_i, D, C = 19, 70, 37                      # D, C not multiples of 4; X shifted off 16-byte alignment
    X, y, W = inputs.softmax_problem([b_i], D, C, seed=77, w_std=0.1, device=DEV)
    Xs = torch.empty(b_i * D + 1, device=DEV)[1:].view(b_i, D)
    Xs.copy_(X)
    for flags in (TENSOR, FFMA):
        G, loss = _worker_grad(Xs, y, W, flags)
        rG, rloss = oracle.worker_grad(X.cpu().numpy(), y.cpu().numpy(), W.cpu().numpy())
        assert rel_err(f64(G), rG) <= FP32_TOL and abs(loss - rloss) <= FP32_TOL * abs(rloss)


def test_tensor_and_ffma_paths_agree_and_repeat_bitwise():
    X, y, W = inputs.softmax_problem([64], 512, 250, seed=78, device=DEV)
    G1, _ = _worker_grad(X, y, W, TENSOR)
    G2, _ = _worker_grad(X, y, W, TENSOR)
    G3, _ = _worker_grad(X, y, W, FFMA)
    assert torch.equal(G1, G2)
    assert rel_err(f64(G1), f64(G3)) <= FP32_TOL


@pytest.mark.parametrize("flags", [TENSOR, FFMA])
def test_config_ragged_four_workers_against_the_concatenated_batch(flags):
    """D=2048, C=1000, b={24,40,64,128}: per-worker gradients, then the weighted aggregate,
    which must be the mean gradient of all 256 samples."""
    bs = [24, 40, 64, 128]
    D, C = 2048, 1000
    X, y, W = inputs.softmax_problem(bs, D, C, seed=3000, device=DEV)
    offs = np.concatenate([[0], np.cumsum(bs)])
    Xh, yh, Wh = X.cpu().numpy(), y.cpu().numpy(), W.cpu().numpy()
    Gs = []
    for i, b_i in enumerate(bs):
        s, e = int(offs[i]), int(offs[i + 1])
        G, loss = _worker_grad(X[s:e].contiguous(), y[s:e].contiguous(), W, flags)
        rG, rloss = oracle.worker_grad(Xh[s:e], yh[s:e], Wh)
        assert rel_err(f64(G), rG) <= FP32_TOL, f"worker {i}"
        assert abs(loss - rloss) <= FP32_TOL * abs(rloss)
        Gs.append(G.reshape(-1))
    N = D * C
    p, v = torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
    sq = torch.zeros(1, dtype=torch.float64, device=DEV)
    ws = torch.empty(binding.aggregate_workspace_bytes(4, N), dtype=torch.uint8, device=DEV)
    binding.aggregate_update(Gs, bs, p, v, 1.0, 0.0, sq, ws)      # p = -aggregate, v = aggregate
    torch.cuda.synchronize()
    full, _ = oracle.worker_grad(Xh, yh, Wh)                       # all 256 rows, divisor 256
    full = full.reshape(-1)
    assert rel_err(f64(v), full) <= FP32_TOL
    assert rel_err(f64(p), -full) <= FP32_TOL
    assert abs(float(sq.item()) - float(full @ full)) <= FP32_TOL * float(full @ full)
    # the uniform average of the four gradients is a different vector
    uniform = torch.stack(Gs).double().mean(0).cpu().numpy()
    assert rel_err(uniform, full) > 1e-2


# ------------------------------------------------------------------ grouped (all workers in three launches)
def _grouped(X, y, W, bs):
    offs = [0] + list(np.cumsum(bs))
    D, C = W.shape
    G = [torch.full((D, C), float("nan"), device=DEV) for _ in bs]
    losses = torch.zeros(len(bs), device=DEV)
    ws = torch.empty(binding.worker_grad_grouped_workspace_bytes(offs[-1], len(bs), D, C), dtype=torch.uint8,
                     device=DEV)
    binding.worker_grad_grouped(X, y, W, offs, G, losses, ws)
    torch.cuda.synchronize()
    assert binding.worker_grad_status(ws) == 0
    return G, losses.cpu().numpy(), offs


@pytest.mark.parametrize("bs,D,C", [([24, 40, 64, 128], 2048, 1000), ([1], 8, 4), ([1, 1, 1], 33, 10),
                                     ([5, 130, 2, 33, 70], 100, 130), ([300, 7], 64, 1030)])
def test_grouped_matches_the_oracle_per_worker(bs, D, C):
    X, y, W = inputs.softmax_problem(bs, D, C, seed=4000 + len(bs), w_std=0.02, device=DEV)
    G, losses, offs = _grouped(X, y, W, bs)
    Xh, yh, Wh = X.cpu().numpy(), y.cpu().numpy(), W.cpu().numpy()
    for w in range(len(bs)):
        rG, rloss = oracle.worker_grad(Xh[offs[w]:offs[w + 1]], yh[offs[w]:offs[w + 1]], Wh)
        assert rel_err(f64(G[w]), rG) <= FP32_TOL, f"worker {w}"
        assert abs(losses[w] - rloss) <= FP32_TOL * abs(rloss)


@pytest.mark.parametrize("bs,D,C", [
    ([1000, 3], 40, 72),                                   # 32 blocks of 32 samples: all seven main accumulators
    ([4096], 64, 36),                                      # the longest reduction the tensor-core path takes
    ([(7 * w) % 23 + 1 for w in range(64)], 130, 37),      # the maximum worker count; C % 4 != 0: element-wise stores
    ([385, 384], 129, 65),                                 # 13 and 12 blocks: four accumulators, ragged tiles
])
def test_grouped_long_reductions_and_many_workers(bs, D, C):
    X, y, W = inputs.softmax_problem(bs, D, C, seed=4100 + len(bs), w_std=0.05, device=DEV)
    G, losses, offs = _grouped(X, y, W, bs)
    Xh, yh, Wh = X.cpu().numpy(), y.cpu().numpy(), W.cpu().numpy()
    for w in range(len(bs)):
        rG, rloss = oracle.worker_grad(Xh[offs[w]:offs[w + 1]], yh[offs[w]:offs[w + 1]], Wh)
        assert rel_err(f64(G[w]), rG) <= FP32_TOL, f"worker {w}"
        assert abs(losses[w] - rloss) <= FP32_TOL * abs(rloss)


def test_grouped_outputs_off_the_16_byte_grid_take_ordinary_stores():
    # C is a multiple of 4 but the gradient buffers start one float past a 16-byte boundary: no TMA store
    bs, D, C = [9, 40], 160, 72
    X, y, W = inputs.softmax_problem(bs, D, C, seed=4300, w_std=0.05, device=DEV)
    offs = [0] + list(np.cumsum(bs))
    raw = [torch.full((D * C + 1,), float("nan"), device=DEV) for _ in bs]
    G = [r[1:].view(D, C) for r in raw]
    ws = torch.empty(binding.worker_grad_grouped_workspace_bytes(offs[-1], len(bs), D, C), dtype=torch.uint8,
                     device=DEV)
    binding.worker_grad_grouped(X, y, W, offs, G, None, ws)
    torch.cuda.synchronize()
    assert binding.worker_grad_status(ws) == 0
    Xh, yh, Wh = X.cpu().numpy(), y.cpu().numpy(), W.cpu().numpy()
    for w in range(len(bs)):
        rG, _ = oracle.worker_grad(Xh[offs[w]:offs[w + 1]], yh[offs[w]:offs[w + 1]], Wh)
        assert rel_err(f64(G[w]), rG) <= FP32_TOL
        assert bool(torch.isnan(raw[w][0]))                 # the element before the buffer is untouched


def test_grouped_keeps_a_workers_nan_in_that_workers_gradient():
    # worker 1's rows follow worker 0's in memory and share its last 16-sample copy; they must not leak
    bs = [5, 9, 3]
    X, y, W = inputs.softmax_problem(bs, 48, 20, seed=4200, w_std=0.05, device=DEV)
    X[5:14] = float("nan")
    G, _, offs = _grouped(X, y, W, bs)
    Xh, yh, Wh = X.cpu().numpy(), y.cpu().numpy(), W.cpu().numpy()
    for w in (0, 2):
        rG, _ = oracle.worker_grad(Xh[offs[w]:offs[w + 1]], yh[offs[w]:offs[w + 1]], Wh)
        assert rel_err(f64(G[w]), rG) <= FP32_TOL
    assert bool(torch.isnan(G[1]).all())


def test_grouped_then_aggregate_is_the_concatenated_batch_gradient():
    bs = [24, 40, 64, 128]
    D, C = 2048, 1000
    X, y, W = inputs.softmax_problem(bs, D, C, seed=3000, device=DEV)
    G, _, _ = _grouped(X, y, W, bs)
    N = D * C
    p, v = torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
    binding.aggregate_update([g.reshape(-1) for g in G], bs, p, v, 1.0, 0.0)
    torch.cuda.synchronize()
    full, _ = oracle.worker_grad(X.cpu().numpy(), y.cpu().numpy(), W.cpu().numpy())
    assert rel_err(f64(v), full.reshape(-1)) <= FP32_TOL


def test_back_to_back_calls_on_one_workspace_do_not_disturb_each_other():
    """Calls that share a workspace, enqueued without synchronising and with different samples: each call's
    kernels may be scheduled under the previous call's, but none may touch the workspace before those have
    finished.  Every call's gradients equal (bitwise) the ones it gives when run alone."""
    bs = [24, 40, 64, 128]
    D, C = 2048, 1000
    offs = [0] + list(np.cumsum(bs))
    problems = [inputs.softmax_problem(bs, D, C, seed=7000 + i, w_std=0.02, device=DEV) for i in range(3)]
    alone = [_grouped(X, y, W, bs)[0] for X, y, W in problems]
    ws = torch.empty(binding.worker_grad_grouped_workspace_bytes(offs[-1], len(bs), D, C), dtype=torch.uint8,
                     device=DEV)
    for rep in range(10):
        outs = [[torch.full((D, C), float("nan"), device=DEV) for _ in bs] for _ in problems]
        losses = [torch.zeros(len(bs), device=DEV) for _ in problems]
        torch.cuda.synchronize()
        for (X, y, W), G, l in zip(problems, outs, losses):
            binding.worker_grad_grouped(X, y, W, offs, G, l, ws)
        torch.cuda.synchronize()
        assert binding.worker_grad_status(ws) == 0
        for i, (G, ref) in enumerate(zip(outs, alone)):
            for w in range(len(bs)):
                assert torch.equal(G[w], ref[w]), f"repetition {rep}, call {i}, worker {w}"


def test_grouped_call_and_aggregation_replay_from_a_cuda_graph():
    """The three launches of the grouped call (tensor maps travel in the kernel parameters) and the aggregation
    behind it can be captured once and replayed: same bits as the eager calls, replay after replay."""
    bs = [24, 40, 64, 128]
    D, C = 2048, 1000
    offs = [0] + list(np.cumsum(bs))
    X, y, W = inputs.softmax_problem(bs, D, C, seed=7100, w_std=0.02, device=DEV)
    eager, eager_losses, _ = _grouped(X, y, W, bs)
    N = D * C
    ep, ev = torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
    binding.aggregate_update([g.reshape(-1) for g in eager], bs, ep, ev, 0.5, 0.9)
    torch.cuda.synchronize()

    G = [torch.full((D, C), float("nan"), device=DEV) for _ in bs]
    losses = torch.zeros(len(bs), device=DEV)
    ws = torch.empty(binding.worker_grad_grouped_workspace_bytes(offs[-1], len(bs), D, C), dtype=torch.uint8,
                     device=DEV)
    p, v = torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
    binding.worker_grad_grouped(X, y, W, offs, G, losses, ws)          # not the first call in capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        stream = torch.cuda.current_stream()
        binding.worker_grad_grouped(X, y, W, offs, G, losses, ws, stream)
        binding.aggregate_update([g.reshape(-1) for g in G], bs, p, v, 0.5, 0.9, None, None, stream)
    for rep in range(3):
        for g in G:
            g.fill_(float("nan"))
        p.zero_()
        v.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert binding.worker_grad_status(ws) == 0
        for w in range(len(bs)):
            assert torch.equal(G[w], eager[w]), f"replay {rep}, worker {w}"
        assert np.array_equal(losses.cpu().numpy(), eager_losses)
        assert torch.equal(p, ep) and torch.equal(v, ev)


def test_grouped_argument_errors():
    X, y, W = inputs.softmax_problem([4, 4], 16, 8, seed=9, device=DEV)
    G = [torch.empty(16, 8, device=DEV) for _ in range(2)]
    ws = torch.empty(binding.worker_grad_grouped_workspace_bytes(8, 2, 16, 8), dtype=torch.uint8, device=DEV)
    for offs in ([0, 4, 4], [1, 4, 8], [0, 5, 4]):           # empty worker, bad start, decreasing
        Xs = X[:max(offs[-1], 1)]
        with pytest.raises((binding.DynbatchError, ValueError)):
            binding.worker_grad_grouped(X[:offs[-1]], y[:offs[-1]], W, offs, G, None, ws)
    with pytest.raises(binding.DynbatchError):
        binding.worker_grad_grouped(X, y, W, [0, 4, 8], G, None, ws[:64])
