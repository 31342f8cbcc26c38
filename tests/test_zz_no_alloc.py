"""The allocation-free entry point, db_aggregate_update_static, against db_aggregate_update_ex.

Some users of the library may not allocate device memory at all (a plug-in whose host owns the whole
GPU heap, a loop where cudaMalloc's device-wide synchronisation is not acceptable).  For them the
norm's scratch lives in a fixed array inside the library.  The result must be the one the workspace
form gives -- also on a second call, when the shared array still holds the first call's partials.  This file sorts last so a failure here cannot hide another test's.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import FP32_TOL, f64, host_grad, rel_err
from paper_2305_12213_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _reference(grads, b, p0, v0, lr, mu):
    K, N = len(grads), p0.numel()
    p, v = p0.clone(), v0.clone()
    sq = torch.zeros(1, dtype=torch.float64, device=DEV)
    ws = torch.empty(binding.aggregate_workspace_bytes(K, N), dtype=torch.uint8, device=DEV)
    binding.aggregate_update(grads, b, p, v, lr, mu, sq, ws)
    torch.cuda.synchronize()
    return p, v, float(sq.item())


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_two_calls_in_a_row_match_the_workspace_form(dtype):
    K, N = 8, 3_000_017
    b = [58] * 4 + [6] * 4
    p_ref = inputs.normal(N, 0.02, 1, DEV)
    v_ref = torch.zeros(N, device=DEV)
    p, v = p_ref.clone(), v_ref.clone()
    sq = torch.full((1,), -1.0, dtype=torch.float64, device=DEV)
    for call in range(2):
        # a different problem each call: other gradients, and K shrinks so fewer slots are rewritten
        kk = K - 3 * call
        grads = inputs.worker_gradients(kk, N, 1e-3, 700 + call, device=DEV, dtype=dtype)
        p_ref, v_ref, sq_ref = _reference(grads, b[:kk], p_ref, v_ref, 0.1, 0.9)
        binding.aggregate_update_static(grads, b[:kk], p, v, 0.1, 0.9, sq)
        torch.cuda.synchronize()
        assert torch.equal(p, p_ref) and torch.equal(v, v_ref), f"call {call}"
        got = float(sq.item())
        assert got == sq_ref, f"call {call}: {got} vs {sq_ref}"      # same kernel, same grid: same bits
        assert abs(got - sq_ref) <= 1e-5 * sq_ref


def test_small_then_large_problem_reuses_the_array_cleanly():
    sq = torch.zeros(1, dtype=torch.float64, device=DEV)
    for N in (1000, 5_000_003, 7):
        g = [torch.ones(N, device=DEV) for _ in range(3)]
        p, v = torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
        binding.aggregate_update_static(g, [1, 2, 3], p, v, 0.5, 0.0, sq)
        torch.cuda.synchronize()
        assert float(sq.item()) == float(N)
        assert torch.equal(v, torch.ones(N, device=DEV)) and torch.equal(p, torch.full((N,), -0.5, device=DEV))


def test_without_norm_and_argument_errors():
    N = 4096
    g = inputs.worker_gradients(2, N, 1.0, 710, device=DEV)
    p0, v0 = inputs.normal(N, 0.02, 2, DEV), inputs.normal(N, 0.5, 3, DEV)
    p1, v1, p2, v2 = p0.clone(), v0.clone(), p0.clone(), v0.clone()
    binding.aggregate_update_static(g, [3, 5], p1, v1, 0.1, 0.9)
    binding.aggregate_update(g, [3, 5], p2, v2, 0.1, 0.9)
    torch.cuda.synchronize()
    assert torch.equal(p1, p2) and torch.equal(v1, v2)
    with pytest.raises(binding.DynbatchError) as ei:
        binding.aggregate_update_static(g, [0, 0], p1, v1, 0.1, 0.9)
    assert ei.value.status == binding.DB_ERR_ARG


def test_against_the_oracle_itself():
    """The same step judged by the fp64 definition, not by the library's other entry point."""
    K, N, b = 5, 1_500_011, [3, 9, 0, 18, 5]
    grads = inputs.worker_gradients(K, N, 1e-3, 720, device=DEV)
    p, v = inputs.normal(N, 0.02, 4, DEV), inputs.normal(N, 0.01, 5, DEV)
    rp, rv = f64(p), f64(v)
    sq = torch.zeros(1, dtype=torch.float64, device=DEV)
    for call in range(2):
        binding.aggregate_update_static(grads, b, p, v, 0.1, 0.9, sq)
        torch.cuda.synchronize()
        _, rsq = oracle.aggregate_update([host_grad(g) for g in grads], b, rp, rv,
                                         float(np.float32(0.1)), float(np.float32(0.9)))
        assert rel_err(f64(p), rp) <= FP32_TOL and rel_err(f64(v), rv) <= FP32_TOL, f"call {call}"
        assert abs(float(sq.item()) - rsq) <= FP32_TOL * rsq


def test_the_size_limit_is_reported_and_nothing_runs():
    """One parameter beyond what the built-in array serves with the norm: DB_ERR_UNSUPPORTED with a
    message that names the bytes, params / momentum / norm untouched.  At the limit, and at any size
    without the norm, the call goes through."""
    limit = (binding.DB_STATIC_SCRATCH_BYTES // 8 - 2) * 1024
    assert limit == 134_215_680
    N = limit + 1
    g = [torch.ones(N, device=DEV)]
    p, v = torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
    sq = torch.full((1,), -7.0, dtype=torch.float64, device=DEV)
    with pytest.raises(binding.DynbatchError) as ei:
        binding.aggregate_update_static(g, [4], p, v, 0.5, 0.0, sq)
    torch.cuda.synchronize()
    assert ei.value.status == binding.DB_ERR_UNSUPPORTED
    assert str(binding.DB_STATIC_SCRATCH_BYTES) in str(ei.value) and "bytes" in str(ei.value)
    assert float(sq.item()) == -7.0 and not p.any().item() and not v.any().item()
    # bad arguments are reported as such even when the size is over the limit too
    with pytest.raises(binding.DynbatchError) as ei:
        binding.aggregate_update_static(g, [0], p, v, 0.5, 0.0, sq)
    assert ei.value.status == binding.DB_ERR_ARG
    # without the norm there is no scratch and no limit
    binding.aggregate_update_static(g, [4], p, v, 0.5, 0.0)
    torch.cuda.synchronize()
    assert torch.equal(v, g[0]) and float(p[0]) == -0.5 and float(p[-1]) == -0.5
    # exactly at the limit, with the norm
    p.zero_(), v.zero_()
    binding.aggregate_update_static([g[0][:limit]], [4], p[:limit], v[:limit], 0.5, 0.0, sq)
    torch.cuda.synchronize()
    assert float(sq.item()) == float(limit) and float(v[limit - 1]) == 1.0 and float(v[limit]) == 0.0
