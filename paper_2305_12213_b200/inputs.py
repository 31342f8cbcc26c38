"""Seeded synthetic inputs for the parameter-server step.

Shapes, sizes and value distributions of the workloads only; none of the
method's arithmetic lives here (no weights, no aggregation, no controller).
Both the CUDA library's tests/benchmark and the CPU oracle's tests draw their
inputs from this module, so the two sides see identical bytes.

The paper trains ResNet-50 (CIFAR-10), an MNIST CNN and a linear model; the
aggregation step is data-oblivious (its cost depends on K, N and the gradient
dtype only), so gradients are random normals laid out with the tensor shapes
of the named architectures.
"""
from __future__ import annotations

import math
from typing import List, Sequence, Tuple

import torch


# --------------------------------------------------------------------------
# Parameter-tensor shape lists
# --------------------------------------------------------------------------
def resnet50_tensor_shapes() -> List[Tuple[int, ...]]:
    """The 161 parameter tensors of ResNet-50 (ImageNet head), definition order.

    Stem 7x7 conv 3->64 + BN; bottleneck stages [3, 4, 6, 3] of widths
    64/128/256/512 (expansion 4), each block = 1x1, 3x3, 1x1 convs with a BN
    (scale, shift) after each, plus a 1x1 projection + BN on the first block
    of a stage; fully connected 2048 -> 1000 with bias.  25,557,032 elements.
    """
    shapes: List[Tuple[int, ...]] = [(64, 3, 7, 7), (64,), (64,)]
    inplanes = 64
    for planes, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for blk in range(blocks):
            out = planes * 4
            shapes += [(planes, inplanes, 1, 1), (planes,), (planes,)]
            shapes += [(planes, planes, 3, 3), (planes,), (planes,)]
            shapes += [(out, planes, 1, 1), (out,), (out,)]
            if blk == 0:
                shapes += [(out, inplanes, 1, 1), (out,), (out,)]
            inplanes = out
    shapes += [(1000, 2048), (1000,)]
    return shapes


def bert_base_tensor_shapes() -> List[Tuple[int, ...]]:
    """The 199 parameter tensors of BERT-base (encoder + pooler), 109,482,240 elements."""
    H, F, V = 768, 3072, 30522
    shapes: List[Tuple[int, ...]] = [(V, H), (512, H), (2, H), (H,), (H,)]
    for _ in range(12):
        for _ in range(4):                       # query, key, value, output
            shapes += [(H, H), (H,)]
        shapes += [(H,), (H,)]                   # attention LayerNorm
        shapes += [(F, H), (F,), (H, F), (H,)]   # feed-forward
        shapes += [(H,), (H,)]                   # output LayerNorm
    shapes += [(H, H), (H,)]                     # pooler
    return shapes


def tensor_offsets(shapes: Sequence[Tuple[int, ...]]) -> List[int]:
    """Start offset of every tensor in the flat arena, plus the total at the end."""
    offs = [0]
    for s in shapes:
        offs.append(offs[-1] + math.prod(s))
    return offs


RESNET50_N = 25_557_032
BERT_BASE_N = 109_482_240


# --------------------------------------------------------------------------
# Seeded draws
# --------------------------------------------------------------------------
def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def normal(n, std: float, seed: int, device="cpu", dtype=torch.float32) -> torch.Tensor:
    """n (int or shape) draws of N(0, std^2) as fp32, optionally rounded (RNE) to `dtype`."""
    shape = (n,) if isinstance(n, int) else tuple(n)
    x = torch.empty(shape, dtype=torch.float32, device=device)
    x.normal_(0.0, std, generator=_gen(seed, device))
    return x if dtype == torch.float32 else x.to(dtype)


def grad_seed(base: int, iteration: int, worker: int) -> int:
    """Seed of worker `worker`'s gradient at iteration `iteration`."""
    return int(base) + 1000 * int(iteration) + int(worker)


def worker_gradients(K: int, n: int, std: float, base_seed: int, iteration: int = 0,
                     device="cpu", dtype=torch.float32) -> List[torch.Tensor]:
    """K independent gradient buffers of n elements each."""
    return [normal(n, std, grad_seed(base_seed, iteration, k), device, dtype)
            for k in range(K)]


def batch_sizes_uniform(K: int, lo: int, hi: int, seed: int) -> List[int]:
    """K integer batch sizes uniform in [lo, hi]."""
    g = _gen(seed, "cpu")
    return torch.randint(lo, hi + 1, (K,), generator=g).tolist()


def lognormal_throughputs(K: int, sigma: float, seed: int) -> List[float]:
    """K worker throughputs exp(sigma * z), z standard normal (fp64)."""
    z = torch.empty(K, dtype=torch.float64).normal_(0.0, 1.0, generator=_gen(seed, "cpu"))
    return torch.exp(sigma * z).tolist()


def softmax_problem(batch_sizes: Sequence[int], D: int, C: int, seed: int,
                    w_std: float = 0.01, device="cpu"):
    """Linear-softmax inputs: features N(0,1) [sum b, D], labels uniform [0,C), W N(0,w_std^2) [D,C]."""
    n = int(sum(batch_sizes))
    X = normal((n, D), 1.0, seed, device)
    W = normal((D, C), w_std, seed + 1, device)
    y = torch.randint(0, C, (n,), generator=_gen(seed + 2, "cpu"), dtype=torch.int32).to(device)
    return X, y, W


def bf16_bits(t: torch.Tensor):
    """numpy uint16 view of a CPU bf16 tensor's bit patterns."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view("uint16")
