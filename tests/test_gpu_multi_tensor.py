"""db_aggregate_update_multi: one launch over a list of separately allocated tensors, against the flat
entry point applied tensor by tensor (bit-identical) and the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from helpers import FP32_TOL, f64, host_grad, rel_err
from paper_2305_12213_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _tensors(sizes, K, dtype, seed, shift=None):
    """Separate allocations per tensor; `shift` (elements) moves some of them off the 16-byte grid."""
    def alloc(n, std, s, dt, t):
        off = 0 if shift is None else shift[t % len(shift)]
        base = inputs.normal(n + 8, std, s, DEV, dt)
        return base[off:off + n]
    grads = [[alloc(n, 1e-3, seed + 100 * k + t, dtype, t) for t, n in enumerate(sizes)] for k in range(K)]
    params = [alloc(n, 0.02, seed + 7000 + t, torch.float32, t) for t, n in enumerate(sizes)]
    momentum = [alloc(n, 0.01, seed + 8000 + t, torch.float32, t) for t, n in enumerate(sizes)]
    return grads, params, momentum


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("shift", [None, [0, 1, 0, 3]])
def test_matches_per_tensor_calls_and_oracle(dtype, shift):
    sizes = [1, 64, 1000, 4099, 1024 * 8, 70001, 5, 300000, 2048]
    K, b = 5, [3, 9, 0, 18, 5]
    grads, params, momentum = _tensors(sizes, K, dtype, 11, shift)
    for t in range(len(sizes)):
        grads[2][t].fill_(float("nan"))                     # the zero-batch worker is never read
    ref_p = [p.clone() for p in params]
    ref_v = [v.clone() for v in momentum]
    p0 = [f64(p) for p in params]
    v0 = [f64(v) for v in momentum]
    plan = binding.MultiTensorPlan(grads, params, momentum)
    sq = torch.zeros(1, dtype=torch.float64, device=DEV)
    for step in range(2):
        plan.step(b, 0.1, 0.9, sq)
        torch.cuda.synchronize()
        total = 0.0
        for t, n in enumerate(sizes):
            binding.aggregate_update([grads[k][t].clone() for k in range(K)], b, ref_p[t], ref_v[t], 0.1, 0.9)
            _, s = oracle.aggregate_update([host_grad(grads[k][t]) for k in range(K)], b, p0[t], v0[t],
                                           float(np.float32(0.1)), float(np.float32(0.9)))
            total += s
        torch.cuda.synchronize()
        for t in range(len(sizes)):
            assert torch.equal(params[t], ref_p[t]) and torch.equal(momentum[t], ref_v[t]), f"tensor {t} step {step}"
            # the oracle keeps its own fp64 state over both steps (free-running), same gate as one step
            assert rel_err(f64(params[t]), p0[t]) <= FP32_TOL
            assert rel_err(f64(momentum[t]), v0[t]) <= FP32_TOL
        assert abs(float(sq.item()) - total) <= FP32_TOL * total
    plan.close()


def test_resnet50_tensor_list_equals_the_flat_arena_call():
    shapes = inputs.resnet50_tensor_shapes()
    offs = inputs.tensor_offsets(shapes)
    N, K, b = offs[-1], 8, [58] * 4 + [6] * 4
    g = inputs.worker_gradients(K, N, 1e-3, 2100, device=DEV)
    p0, v0 = inputs.normal(N, 0.02, 21, DEV), inputs.normal(N, 0.01, 22, DEV)
    p1, v1 = p0.clone(), v0.clone()
    sq1 = torch.zeros(1, dtype=torch.float64, device=DEV)
    ws = torch.empty(binding.aggregate_workspace_bytes(K, N), dtype=torch.uint8, device=DEV)
    binding.aggregate_update(g, b, p1, v1, 0.1, 0.9, sq1, ws)
    # the same memory seen as 161 tensors
    p2, v2 = p0.clone(), v0.clone()
    grads = [[g[k][s:e] for s, e in zip(offs[:-1], offs[1:])] for k in range(K)]
    params = [p2[s:e] for s, e in zip(offs[:-1], offs[1:])]
    momentum = [v2[s:e] for s, e in zip(offs[:-1], offs[1:])]
    plan = binding.MultiTensorPlan(grads, params, momentum)
    sq2 = torch.zeros(1, dtype=torch.float64, device=DEV)
    plan.step(b, 0.1, 0.9, sq2)
    torch.cuda.synchronize()
    assert torch.equal(p1, p2) and torch.equal(v1, v2)
    assert abs(float(sq1.item()) - float(sq2.item())) <= 1e-9 * float(sq1.item())
    plan.close()


def test_argument_errors():
    grads, params, momentum = _tensors([64, 128], 2, torch.float32, 3)
    plan = binding.MultiTensorPlan(grads, params, momentum)
    with pytest.raises(binding.DynbatchError):
        plan.step([0, 0], 0.1, 0.9)
    with pytest.raises(binding.DynbatchError):
        plan.step([1, -1], 0.1, 0.9)
    with pytest.raises(binding.DynbatchError):
        plan.step([1, 1], float("nan"), 0.9)
    plan.close()
