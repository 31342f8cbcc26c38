"""GPU parity of db_aggregate_adam_ex (weighted aggregation + Adam) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from helpers import FP32_TOL, f64, host_grad, rel_err
from paper_2305_12213_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"
LR, B1, B2, EPS = 1e-4, 0.9, 0.999, 1e-8


def _f32(x):
    return float(np.float32(x))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("K,N", [(1, 5), (2, 1023), (3, 70001), (8, 300_000), (17, 50_003), (33, 4099)])
def test_several_steps_teacher_forced_and_free_running(K, N, dtype):
    b = inputs.batch_sizes_uniform(K, 8, 256, 40 + K)
    p = inputs.normal(N, 0.02, 1, DEV)
    m, u = torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
    sq = torch.zeros(1, dtype=torch.float64, device=DEV)
    ws = torch.empty(binding.aggregate_workspace_bytes(K, N), dtype=torch.uint8, device=DEV)
    fp, fm, fu = f64(p), f64(m), f64(u)
    for t in range(1, 7):
        grads = inputs.worker_gradients(K, N, 1e-3, 600, t, DEV, dtype)
        hg = [host_grad(g) for g in grads]
        tp, tm, tu = f64(p), f64(m), f64(u)
        binding.aggregate_adam(grads, b, p, m, u, LR, B1, B2, EPS, t, sq, ws)
        torch.cuda.synchronize()
        _, rsq = oracle.aggregate_adam(hg, b, tp, tm, tu, _f32(LR), _f32(B1), _f32(B2), _f32(EPS), t)
        oracle.aggregate_adam(hg, b, fp, fm, fu, _f32(LR), _f32(B1), _f32(B2), _f32(EPS), t)
        for got, forced, free in ((p, tp, fp), (m, tm, fm), (u, tu, fu)):
            assert rel_err(f64(got), forced) <= FP32_TOL, f"step {t}"
            assert rel_err(f64(got), free) <= FP32_TOL, f"step {t} (free-running)"
        assert abs(float(sq.item()) - rsq) <= FP32_TOL * rsq


def test_misaligned_buffers_and_zero_batch_worker():
    N, K = 10_007, 3
    back = [inputs.normal(N + 8, 1e-3, 700 + k, DEV) for k in range(K)]
    grads = [back[0][1:N + 1], back[1][3:N + 3], back[2][2:N + 2]]      # incongruent: element-wise kernel
    grads[1].fill_(float("nan"))
    b = [5, 0, 9]
    p0 = inputs.normal(N, 0.02, 2, DEV)
    p, m, u = p0.clone(), torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
    binding.aggregate_adam(grads, b, p, m, u, LR, B1, B2, EPS, 1)
    torch.cuda.synchronize()
    rp, rm, ru = f64(p0), np.zeros(N), np.zeros(N)
    oracle.aggregate_adam([host_grad(g) for g in grads], b, rp, rm, ru, _f32(LR), _f32(B1), _f32(B2), _f32(EPS), 1)
    assert rel_err(f64(p), rp) <= FP32_TOL and rel_err(f64(m), rm) <= FP32_TOL and rel_err(f64(u), ru) <= FP32_TOL
    # same values through the vector kernel: identical bits
    p2, m2, u2 = p0.clone(), torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
    binding.aggregate_adam([g.clone() for g in grads], b, p2, m2, u2, LR, B1, B2, EPS, 1)
    torch.cuda.synchronize()
    assert torch.equal(p, p2) and torch.equal(m, m2) and torch.equal(u, u2)


def test_argument_errors():
    N = 64
    g = inputs.worker_gradients(2, N, 1.0, 710, device=DEV)
    p, m, u = (torch.zeros(N, device=DEV) for _ in range(3))
    for kw in (dict(beta1=1.0), dict(beta2=-0.1), dict(eps=-1.0), dict(step=0), dict(lr=float("nan"))):
        args = dict(lr=LR, beta1=B1, beta2=B2, eps=EPS, step=1)
        args.update(kw)
        with pytest.raises(binding.DynbatchError) as ei:
            binding.aggregate_adam(g, [1, 1], p, m, u, **args)
        assert ei.value.status == binding.DB_ERR_ARG
    with pytest.raises(binding.DynbatchError):
        binding.aggregate_adam(g, [1, 1], p, m, m, LR, B1, B2, EPS, 1)       # moments alias
