"""Shared test utilities: the error metric and host/device conversions."""
import numpy as np
import torch

FP32_TOL = 1e-5     # max relative error of fp32 results against the fp64 oracle
BF16_TOL = 1e-2     # bf16 gradients against the oracle fed the unrounded fp32 gradients


def rel_err(x, r):
    """max_j |x_j - r_j| / max(|r_j|, rms(r)): relative error with a floor at the tensor's
    rms, so entries that cancel to almost zero are judged on the tensor's own scale."""
    x = np.asarray(x, dtype=np.float64).reshape(-1)
    r = np.asarray(r, dtype=np.float64).reshape(-1)
    if r.size == 0:
        return 0.0
    rms = float(np.sqrt(np.mean(r * r)))
    den = np.maximum(np.abs(r), rms)
    den[den == 0.0] = 1.0
    return float(np.max(np.abs(x - r) / den))


def host_grad(t: torch.Tensor):
    """Device/host gradient tensor -> the numpy array the oracle takes (f32, or u16 bf16 bits)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def f64(t: torch.Tensor):
    return t.detach().cpu().numpy().astype(np.float64)


def sample_indices(n: int, count: int, edges: int = 4096, extra=()):
    """Strided sample of about `count` indices plus the first/last `edges` and `extra`."""
    count = min(count, n)
    stride = max(1, n // count)
    idx = np.arange(0, n, stride, dtype=np.int64)
    e = min(edges, n)
    idx = np.concatenate([idx, np.arange(e), np.arange(n - e, n), np.asarray(list(extra), dtype=np.int64)])
    return np.unique(idx)
