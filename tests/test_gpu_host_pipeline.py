"""db_aggregate_update_host: gradients in host memory, chunked and overlapped, against the
device-resident entry point (bit-identical update) and the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from helpers import FP32_TOL, f64, host_grad, rel_err
from paper_2305_12213_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("N,chunk", [(1, 0), (1000, 64), (300_001, 1 << 16), (5_000_003, 0), (1 << 21, 0)])
def test_matches_device_entry_and_oracle(N, chunk, dtype):
    K, b = 5, [3, 9, 0, 18, 5]
    pinned = [inputs.normal(N, 1e-3, 800 + k, "cpu", dtype).pin_memory() for k in range(K)]
    pinned[2].fill_(float("nan"))                      # zero-batch worker: never copied, never read
    p0, v0 = inputs.normal(N, 0.02, 31, DEV), inputs.normal(N, 0.01, 32, DEV)
    # device-resident reference run
    p_ref, v_ref = p0.clone(), v0.clone()
    sq_ref = torch.zeros(1, dtype=torch.float64, device=DEV)
    ws = torch.empty(binding.aggregate_workspace_bytes(K, N), dtype=torch.uint8, device=DEV)
    binding.aggregate_update([g.to(DEV) for g in pinned], b, p_ref, v_ref, 0.1, 0.9, sq_ref, ws)
    # host pipeline, two steps in a row on the same pipeline and staging
    pipe = binding.HostPipeline()
    staging = torch.empty(binding.host_staging_bytes(K, dtype, N, chunk), dtype=torch.uint8, device=DEV)
    p, v = p0.clone(), v0.clone()
    host_p = torch.empty(N, dtype=torch.float32).pin_memory()
    host_sq = torch.zeros(1, dtype=torch.float64).pin_memory()
    pipe.aggregate_update(pinned, b, p, v, 0.1, 0.9, host_p, host_sq, staging, chunk)
    torch.cuda.current_stream().synchronize()
    assert torch.equal(p, p_ref) and torch.equal(v, v_ref)
    assert torch.equal(host_p, p_ref.cpu())
    assert abs(float(host_sq[0]) - float(sq_ref.item())) <= 1e-9 * float(sq_ref.item())
    rp, rv = f64(p0), f64(v0)
    _, rsq = oracle.aggregate_update([host_grad(g) for g in pinned], b, rp, rv,
                                     float(np.float32(0.1)), float(np.float32(0.9)))
    assert rel_err(f64(p), rp) <= FP32_TOL and rel_err(f64(v), rv) <= FP32_TOL
    assert abs(float(host_sq[0]) - rsq) <= FP32_TOL * rsq
    # second step reuses slots that still hold the first step's chunks
    binding.aggregate_update([g.to(DEV) for g in pinned], b, p_ref, v_ref, 0.1, 0.9, sq_ref, ws)
    pipe.aggregate_update(pinned, b, p, v, 0.1, 0.9, host_p, host_sq, staging, chunk)
    torch.cuda.current_stream().synchronize()
    assert torch.equal(p, p_ref) and torch.equal(v, v_ref) and torch.equal(host_p, p_ref.cpu())
    pipe.close()


def test_optional_outputs_and_errors():
    N, K = 10_000, 2
    pinned = [inputs.normal(N, 1.0, 900 + k).pin_memory() for k in range(K)]
    p, v = torch.zeros(N, device=DEV), torch.zeros(N, device=DEV)
    pipe = binding.HostPipeline()
    staging = torch.empty(binding.host_staging_bytes(K, torch.float32, N, 4096), dtype=torch.uint8, device=DEV)
    pipe.aggregate_update(pinned, [1, 1], p, v, 1.0, 0.0, None, None, staging, 4096)
    torch.cuda.synchronize()
    assert rel_err(f64(v), 0.5 * (f64(pinned[0]) + f64(pinned[1]))) <= 1e-6
    with pytest.raises(binding.DynbatchError) as ei:          # staging too small for the default chunk
        pipe.aggregate_update(pinned, [1, 1], p, v, 1.0, 0.0, None, None, staging[:4096], 0)
    assert ei.value.status == binding.DB_ERR_ARG
    with pytest.raises(binding.DynbatchError):
        pipe.aggregate_update(pinned, [0, 0], p, v, 1.0, 0.0, None, None, staging, 4096)
    # params and momentum that overlap, or a non-finite step size: rejected before anything is
    # enqueued, so the state is untouched and the pipeline is still usable
    before = v.clone()
    for args in ((p, p[: N // 2], 1.0), (v, v, 1.0), (p, v, float("nan"))):
        with pytest.raises(binding.DynbatchError) as ei:
            pipe.aggregate_update([g[: args[1].numel()] for g in pinned], [1, 1], args[0][: args[1].numel()],
                                  args[1], args[2], 0.0, None, None, staging, 4096)
        assert ei.value.status == binding.DB_ERR_ARG
    torch.cuda.synchronize()
    assert torch.equal(v, before)
    pipe.aggregate_update(pinned, [1, 1], p, v, 1.0, 0.0, None, None, staging, 4096)
    torch.cuda.synchronize()
    pipe.close()
