"""db_contract_f32 (the tensor-core contraction under db_worker_grad) against numpy's fp64 matmul."""
import numpy as np
import pytest
import torch

from helpers import FP32_TOL, f64, rel_err
from paper_2305_12213_b200 import binding, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _operand(rows, K, layout, seed):
    """[rows, K] view that is k-contiguous, row-contiguous, or strided/misaligned."""
    if layout == "k":
        return inputs.normal((rows, K), 1.0, seed, DEV)
    if layout == "row":
        return inputs.normal((K, rows), 1.0, seed, DEV).t()
    base = inputs.normal((rows, 2 * K + 3), 1.0, seed, DEV)
    return base[:, 1:2 * K + 1:2]


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (5, 7, 3), (128, 32, 32), (129, 33, 65), (300, 130, 100),
                                   (1000, 24, 128), (257, 1000, 40), (2048, 1000, 128), (1000, 128, 2048)])
@pytest.mark.parametrize("la,lb", [("k", "k"), ("row", "k"), ("k", "row"), ("row", "row"), ("odd", "odd")])
def test_against_fp64_matmul(M, N, K, la, lb):
    A, B = _operand(M, K, la, 1), _operand(N, K, lb, 2)
    out = torch.full((M, N), float("nan"), device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.contract_f32(A, B, out, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = f64(A) @ f64(B).T
    assert rel_err(f64(out), ref) <= FP32_TOL


@pytest.mark.parametrize("M,N,K", [(4, 1, 4), (128, 32, 32), (132, 33, 68), (300, 130, 100), (1000, 24, 128),
                                   (260, 1000, 40), (1000, 256, 2048), (1000, 128, 4100)])
def test_operands_by_tma_in_the_logits_layout(M, N, K):
    """A contiguous along m, B along k, out along m (all 16-byte aligned, pitches multiples of 4): the
    layout of the logits, which takes the TMA-fed kernel; ragged tiles, a ragged last reduction block,
    reductions long enough for several accumulators."""
    A, B = _operand(M, K, "row", 5), _operand(N, K, "k", 6)
    out_t = torch.full((N, M), float("nan"), device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.contract_f32(A, B, out_t.t(), status)          # out(m, n) stored at [n, m]
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = f64(A) @ f64(B).T
    assert rel_err(f64(out_t.t()), ref) <= FP32_TOL


def test_empty_reduction_writes_zeros():
    import ctypes
    M, N = 70, 40
    dummy = torch.ones(8, device=DEV)
    out = torch.full((M, N), float("nan"), device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    st = binding.lib().db_contract_f32(dummy.data_ptr(), 0, 1, dummy.data_ptr(), 0, 1, out.data_ptr(), N, 1,
                                       M, N, 0, status.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert st == binding.DB_OK and int(status.item()) == 0 and torch.count_nonzero(out) == 0


def test_transposed_output_and_exact_small_integers():
    M, N, K = 200, 48, 64
    A = torch.randint(-8, 9, (M, K), device=DEV).float()
    B = torch.randint(-8, 9, (N, K), device=DEV).float()
    out_t = torch.empty(N, M, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.contract_f32(A, B, out_t.t(), status)          # out(m, n) stored at [n, m]
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(out_t.t().double(), A.double() @ B.double().T)   # integers: every step is exact
