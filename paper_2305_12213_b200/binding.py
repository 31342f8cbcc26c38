"""Thin ctypes binding of libdynbatch (argument marshalling only).

Every function has the name and meaning of the C entry point declared in
include/dynbatch.h; tensors are torch tensors used purely as device memory
(`data_ptr()`), and the stream is torch's current stream unless given.  All
arithmetic runs inside the CUDA library: there is no Python or CPU fallback,
and a missing shared library is an error, not a reason to compute elsewhere.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_char_p, c_double, c_float, c_int32, c_int64, c_size_t, c_void_p
from typing import Optional, Sequence

import torch

DB_OK, DB_ERR_NULL, DB_ERR_ARG, DB_ERR_UNSUPPORTED, DB_ERR_INFEASIBLE, DB_ERR_CUDA = range(6)
DB_F32, DB_BF16 = 0, 1
DB_MAX_K = 64
DB_STATIC_SCRATCH_BYTES = 1 << 20     # the built-in scratch of aggregate_update_static

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "csrc", "libdynbatch.so")

_lib = None


class DynbatchError(RuntimeError):
    """A libdynbatch call returned a status other than DB_OK."""

    def __init__(self, status: int, message: str):
        super().__init__(f"libdynbatch status {status}: {message}")
        self.status = status


_SIGNATURES = {
    "db_aggregate_update": (c_int32, [c_void_p, c_void_p, c_int32, c_int64, c_void_p, c_void_p,
                                      c_float, c_float]),
    "db_aggregate_update_ex": (c_int32, [c_void_p, c_int32, c_void_p, c_int32, c_int64, c_void_p,
                                         c_void_p, c_float, c_float, c_void_p, c_void_p, c_size_t,
                                         c_void_p]),
    "db_aggregate_workspace_bytes": (c_size_t, [c_int32, c_int64]),
    "db_aggregate_adam_ex": (c_int32, [c_void_p, c_int32, c_void_p, c_int32, c_int64, c_void_p, c_void_p, c_void_p,
                                       c_float, c_float, c_float, c_float, c_int64, c_void_p, c_void_p, c_size_t,
                                       c_void_p]),
    "db_multi_plan_device_bytes": (c_size_t, [c_int32, c_int32, c_void_p, c_int32]),
    "db_multi_plan_create": (c_int32, [c_void_p, c_void_p, c_int32, c_int32, c_void_p, c_int32, c_void_p, c_void_p,
                                       c_void_p, c_size_t, c_void_p]),
    "db_aggregate_update_multi": (c_int32, [c_void_p, c_void_p, c_float, c_float, c_void_p, c_void_p]),
    "db_multi_plan_destroy": (c_int32, [c_void_p]),
    "db_aggregate_update_static": (c_int32, [c_void_p, c_int32, c_void_p, c_int32, c_int64, c_void_p,
                                             c_void_p, c_float, c_float, c_void_p, c_void_p]),
    "db_shard_range": (c_int32, [c_int64, c_int32, c_int32, c_int32, c_void_p, c_void_p]),
    "db_bench_read_probe_sink_bytes": (c_size_t, [c_size_t]),
    "db_bench_read_probe": (c_int32, [c_void_p, c_size_t, c_void_p, c_void_p]),
    "db_bench_wait_timeout": (c_int32, [c_void_p, c_int32, ctypes.c_uint64, c_void_p]),
    "db_bench_aggregate_variant": (c_int32, [c_int32, c_int32, c_void_p, c_void_p, c_int32, c_int64, c_void_p,
                                             c_void_p, c_float, c_float, c_void_p, c_void_p]),
    "db_host_pipeline_create": (c_int32, [c_void_p]),
    "db_host_pipeline_destroy": (c_int32, [c_void_p]),
    "db_host_staging_bytes": (c_size_t, [c_int32, c_int32, c_int64, c_int64]),
    "db_aggregate_update_host": (c_int32, [c_void_p, c_void_p, c_int32, c_void_p, c_int32, c_int64, c_void_p,
                                           c_void_p, c_float, c_float, c_void_p, c_void_p, c_void_p, c_size_t,
                                           c_int64, c_void_p]),
    "db_worker_grad": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p,
                                 c_void_p, c_void_p, c_size_t, c_void_p]),
    "db_worker_grad_ex": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p,
                                    c_void_p, c_void_p, c_size_t, ctypes.c_uint32, c_void_p]),
    "db_worker_grad_grouped": (c_int32, [c_void_p, c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32,
                                         c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "db_worker_grad_grouped_workspace_bytes": (c_size_t, [c_int32, c_int32, c_int32, c_int32]),
    "db_contract_f32": (c_int32, [c_void_p, c_int64, c_int64, c_void_p, c_int64, c_int64, c_void_p, c_int64,
                                  c_int64, c_int32, c_int32, c_int32, c_void_p, c_void_p]),
    "db_worker_grad_workspace_bytes": (c_size_t, [c_int32, c_int32, c_int32]),
    "db_controller_step": (c_int32, [c_void_p, c_void_p, c_int32, c_double]),
    "db_controller_step_ex": (c_int32, [c_void_p, c_void_p, c_int32, c_double, c_void_p, c_void_p]),
    "db_static_allocate": (c_int32, [c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p]),
    "db_controller_create": (c_int32, [c_void_p, c_void_p, c_int32, c_double, c_double, c_double, c_void_p,
                                       c_void_p, c_int32]),
    "db_controller_observe": (c_int32, [c_void_p, c_void_p, c_void_p, c_void_p]),
    "db_controller_destroy": (c_int32, [c_void_p]),
    "db_status_string": (c_char_p, [c_int32]),
    "db_last_cuda_error": (c_char_p, []),
}


def lib() -> ctypes.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2305_12213_b200.build`. "
                "libdynbatch has no CPU fallback.")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _check(status: int) -> None:
    if status != DB_OK:
        L = lib()
        msg = L.db_status_string(status).decode()
        if status in (DB_ERR_CUDA, DB_ERR_UNSUPPORTED):
            detail = L.db_last_cuda_error().decode()
            if detail:
                msg += ": " + detail
        raise DynbatchError(status, msg)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _i32_array(values: Sequence[int]):
    return (c_int32 * len(values))(*[int(x) for x in values])


def _dev_ptr(t: Optional[torch.Tensor], dtype: torch.dtype, name: str) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name} must be a contiguous CUDA tensor of {dtype}")
    return t.data_ptr()


def aggregate_workspace_bytes(K: int, N: int) -> int:
    return int(lib().db_aggregate_workspace_bytes(int(K), int(N)))


def aggregate_update(grads: Sequence[torch.Tensor], b: Sequence[int], params: torch.Tensor,
                     momentum: torch.Tensor, lr: float, mu: float,
                     grad_sqnorm: Optional[torch.Tensor] = None,
                     workspace: Optional[torch.Tensor] = None,
                     stream: Optional[torch.cuda.Stream] = None, N: Optional[int] = None) -> None:
    """db_aggregate_update_ex: fused weighted aggregation + momentum-SGD update, in place.

    grads: K CUDA tensors (all float32 or all bfloat16) of N elements; b: K batch sizes;
    params, momentum: float32 CUDA tensors; grad_sqnorm: optional float64 CUDA tensor of one
    element; workspace: uint8 CUDA tensor of aggregate_workspace_bytes(K, N) when the norm is wanted.
    """
    K = len(grads)
    if len(b) != K:
        raise ValueError("len(b) != len(grads)")
    gdt = grads[0].dtype
    if gdt == torch.float32:
        code = DB_F32
    elif gdt == torch.bfloat16:
        code = DB_BF16
    else:
        raise TypeError("gradients must be float32 or bfloat16")
    n = int(params.numel() if N is None else N)
    table = (c_void_p * K)(*[_dev_ptr(g, gdt, "grads[k]") for g in grads])
    _check(lib().db_aggregate_update_ex(
        ctypes.cast(table, c_void_p), code, ctypes.cast(_i32_array(b), c_void_p), K, n,
        _dev_ptr(params, torch.float32, "params"), _dev_ptr(momentum, torch.float32, "momentum"),
        float(lr), float(mu), _dev_ptr(grad_sqnorm, torch.float64, "grad_sqnorm"),
        None if workspace is None else workspace.data_ptr(),
        0 if workspace is None else workspace.numel() * workspace.element_size(),
        _stream_ptr(stream)))


class AggregateStep:
    """db_aggregate_update_ex with its tensor arguments marshalled once: for loops that call the step
    on the same buffers every iteration (the pointers, not the tensors' contents, are fixed here).
    `run(b, lr, mu)` then only converts the batch sizes and the two scalars."""

    def __init__(self, grads: Sequence[torch.Tensor], params: torch.Tensor, momentum: torch.Tensor,
                 grad_sqnorm: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                 stream: Optional[torch.cuda.Stream] = None):
        self.K = len(grads)
        gdt = grads[0].dtype
        if gdt not in (torch.float32, torch.bfloat16):
            raise TypeError("gradients must be float32 or bfloat16")
        self._keep = (list(grads), params, momentum, grad_sqnorm, workspace)       # the buffers stay alive
        self._table = (c_void_p * self.K)(*[_dev_ptr(g, gdt, "grads[k]") for g in grads])
        self._b = (c_int32 * self.K)()
        self._fn = lib().db_aggregate_update_ex
        self._args = (ctypes.cast(self._table, c_void_p), DB_F32 if gdt == torch.float32 else DB_BF16,
                      ctypes.cast(self._b, c_void_p), self.K, int(params.numel()),
                      _dev_ptr(params, torch.float32, "params"), _dev_ptr(momentum, torch.float32, "momentum"))
        self._tail = (_dev_ptr(grad_sqnorm, torch.float64, "grad_sqnorm"),
                      None if workspace is None else workspace.data_ptr(),
                      0 if workspace is None else workspace.numel() * workspace.element_size(),
                      _stream_ptr(stream))

    def run(self, b: Sequence[int], lr: float, mu: float) -> None:
        if len(b) != self.K:
            raise ValueError("len(b) != number of gradient buffers")
        self._b[:] = b
        _check(self._fn(*self._args, lr, mu, *self._tail))


def aggregate_adam(grads: Sequence[torch.Tensor], b: Sequence[int], params: torch.Tensor,
                   first_moment: torch.Tensor, second_moment: torch.Tensor, lr: float, beta1: float,
                   beta2: float, eps: float, step: int, grad_sqnorm: Optional[torch.Tensor] = None,
                   workspace: Optional[torch.Tensor] = None,
                   stream: Optional[torch.cuda.Stream] = None) -> None:
    """db_aggregate_adam_ex: fused weighted aggregation + Adam update (bias-corrected), in place."""
    K = len(grads)
    if len(b) != K:
        raise ValueError("len(b) != len(grads)")
    gdt = grads[0].dtype
    table = (c_void_p * K)(*[_dev_ptr(g, gdt, "grads[k]") for g in grads])
    code = DB_F32 if gdt == torch.float32 else DB_BF16 if gdt == torch.bfloat16 else -1
    _check(lib().db_aggregate_adam_ex(
        ctypes.cast(table, c_void_p), code, ctypes.cast(_i32_array(b), c_void_p), K, int(params.numel()),
        _dev_ptr(params, torch.float32, "params"), _dev_ptr(first_moment, torch.float32, "first_moment"),
        _dev_ptr(second_moment, torch.float32, "second_moment"), float(lr), float(beta1), float(beta2),
        float(eps), int(step), _dev_ptr(grad_sqnorm, torch.float64, "grad_sqnorm"),
        None if workspace is None else workspace.data_ptr(),
        0 if workspace is None else workspace.numel() * workspace.element_size(), _stream_ptr(stream)))


def aggregate_update_static(grads: Sequence[torch.Tensor], b: Sequence[int], params: torch.Tensor,
                            momentum: torch.Tensor, lr: float, mu: float,
                            grad_sqnorm: Optional[torch.Tensor] = None,
                            stream: Optional[torch.cuda.Stream] = None) -> None:
    """db_aggregate_update_static: aggregate_update for callers that cannot supply a workspace.

    The norm's scratch is a fixed array inside the library, shared by every call on the device, so
    calls that could overlap on the GPU must be serialised by the caller.  Nothing is allocated.
    """
    K = len(grads)
    if len(b) != K:
        raise ValueError("len(b) != len(grads)")
    gdt = grads[0].dtype
    if gdt not in (torch.float32, torch.bfloat16):
        raise TypeError("gradients must be float32 or bfloat16")
    table = (c_void_p * K)(*[_dev_ptr(g, gdt, "grads[k]") for g in grads])
    _check(lib().db_aggregate_update_static(
        ctypes.cast(table, c_void_p), DB_F32 if gdt == torch.float32 else DB_BF16,
        ctypes.cast(_i32_array(b), c_void_p), K, int(params.numel()),
        _dev_ptr(params, torch.float32, "params"), _dev_ptr(momentum, torch.float32, "momentum"),
        float(lr), float(mu), _dev_ptr(grad_sqnorm, torch.float64, "grad_sqnorm"), _stream_ptr(stream)))


def shard_range(N: int, G: int, r: int, align: int = 8):
    """db_shard_range: the slice [begin, end) of N parameters that parameter server r of G owns."""
    lo, hi = ctypes.c_int64(0), ctypes.c_int64(0)
    _check(lib().db_shard_range(int(N), int(G), int(r), int(align), ctypes.byref(lo), ctypes.byref(hi)))
    return int(lo.value), int(hi.value)


DB_BENCH_PERSISTENT, DB_BENCH_BULK_STAGED = 1, 2


def bench_read_probe_sink_bytes(nbytes: int) -> int:
    return int(lib().db_bench_read_probe_sink_bytes(int(nbytes)))


def bench_read_probe(src: torch.Tensor, sink: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """db_bench_read_probe: stream all of `src` through registers once (a measurement helper)."""
    if not (src.is_cuda and sink.is_cuda and src.is_contiguous() and sink.is_contiguous()):
        raise TypeError("src and sink must be contiguous CUDA tensors")
    nbytes = src.numel() * src.element_size()
    if sink.numel() * sink.element_size() < bench_read_probe_sink_bytes(nbytes):
        raise ValueError("sink too small")
    _check(lib().db_bench_read_probe(src.data_ptr(), nbytes, sink.data_ptr(), _stream_ptr(stream)))


def bench_wait_timeout(status: torch.Tensor, code: int, limit_ns: int,
                       stream: Optional[torch.cuda.Stream] = None) -> None:
    """db_bench_wait_timeout: run the kernels' bounded wait until it gives up and reports `code`."""
    _check(lib().db_bench_wait_timeout(_dev_ptr(status, torch.int32, "status"), int(code), int(limit_ns),
                                       _stream_ptr(stream)))


def bench_aggregate_variant(variant: int, stage_floats: int, grads: Sequence[torch.Tensor], b: Sequence[int],
                            params: torch.Tensor, momentum: torch.Tensor, lr: float, mu: float,
                            status: Optional[torch.Tensor] = None,
                            stream: Optional[torch.cuda.Stream] = None) -> None:
    """db_bench_aggregate_variant: the momentum step in a launch shape that was measured and not adopted."""
    K = len(grads)
    if len(b) != K:
        raise ValueError("len(b) != len(grads)")
    table = (c_void_p * K)(*[_dev_ptr(g, torch.float32, "grads[k]") for g in grads])
    _check(lib().db_bench_aggregate_variant(
        int(variant), int(stage_floats), ctypes.cast(table, c_void_p), ctypes.cast(_i32_array(b), c_void_p), K,
        int(params.numel()), _dev_ptr(params, torch.float32, "params"), _dev_ptr(momentum, torch.float32, "momentum"),
        float(lr), float(mu), _dev_ptr(status, torch.int32, "status"), _stream_ptr(stream)))


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.float32:
        return DB_F32
    if dt == torch.bfloat16:
        return DB_BF16
    raise TypeError("gradients must be float32 or bfloat16")


def host_staging_bytes(K: int, grad_dtype: torch.dtype, N: int, chunk_elems: int = 0) -> int:
    return int(lib().db_host_staging_bytes(int(K), _dtype_code(grad_dtype), int(N), int(chunk_elems)))


class HostPipeline:
    """db_host_pipeline: side streams and events for db_aggregate_update_host on the current device."""

    def __init__(self):
        self._h = c_void_p()
        _check(lib().db_host_pipeline_create(ctypes.byref(self._h)))

    def close(self) -> None:
        if self._h:
            lib().db_host_pipeline_destroy(self._h)
            self._h = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def aggregate_update(self, host_grads: Sequence[torch.Tensor], b: Sequence[int], params: torch.Tensor,
                         momentum: torch.Tensor, lr: float, mu: float,
                         host_params_out: Optional[torch.Tensor], host_sqnorm_out: Optional[torch.Tensor],
                         staging: torch.Tensor, chunk_elems: int = 0,
                         stream: Optional[torch.cuda.Stream] = None) -> None:
        """db_aggregate_update_host: gradients in (pinned) host tensors, parameters copied back to the host."""
        K = len(host_grads)
        if len(b) != K:
            raise ValueError("len(b) != len(host_grads)")
        gdt = host_grads[0].dtype
        for g in host_grads:
            if g.is_cuda or g.dtype != gdt or not g.is_contiguous():
                raise TypeError("host_grads must be contiguous CPU tensors of one dtype")
        for t, dt, name in ((host_params_out, torch.float32, "host_params_out"),
                            (host_sqnorm_out, torch.float64, "host_sqnorm_out")):
            if t is not None and (t.is_cuda or t.dtype != dt or not t.is_contiguous()):
                raise TypeError(f"{name} must be a contiguous CPU tensor of {dt}")
        table = (c_void_p * K)(*[g.data_ptr() for g in host_grads])
        _check(lib().db_aggregate_update_host(
            self._h, ctypes.cast(table, c_void_p), _dtype_code(gdt), ctypes.cast(_i32_array(b), c_void_p), K,
            int(params.numel()), _dev_ptr(params, torch.float32, "params"),
            _dev_ptr(momentum, torch.float32, "momentum"), float(lr), float(mu),
            None if host_params_out is None else host_params_out.data_ptr(),
            None if host_sqnorm_out is None else host_sqnorm_out.data_ptr(),
            staging.data_ptr(), staging.numel() * staging.element_size(), int(chunk_elems),
            _stream_ptr(stream)))


def worker_grad_workspace_bytes(b_i: int, D: int, C: int) -> int:
    return int(lib().db_worker_grad_workspace_bytes(int(b_i), int(D), int(C)))


DB_WORKER_GRAD_FFMA = 1


def worker_grad(X: torch.Tensor, y: torch.Tensor, W: torch.Tensor, G: torch.Tensor,
                loss: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                stream: Optional[torch.cuda.Stream] = None, flags: int = 0) -> None:
    """db_worker_grad_ex: G = X^T (softmax(X W) - onehot(y)) / b_i, optional mean cross-entropy."""
    b_i, D = X.shape
    D2, C = W.shape
    if D2 != D or tuple(G.shape) != (D, C) or y.numel() != b_i:
        raise ValueError("shape mismatch")
    _check(lib().db_worker_grad_ex(
        _dev_ptr(X, torch.float32, "X"), _dev_ptr(y, torch.int32, "y"), _dev_ptr(W, torch.float32, "W"),
        b_i, D, C, _dev_ptr(G, torch.float32, "G"), _dev_ptr(loss, torch.float32, "loss"),
        None if workspace is None else workspace.data_ptr(),
        0 if workspace is None else workspace.numel() * workspace.element_size(),
        int(flags), _stream_ptr(stream)))


def worker_grad_grouped_workspace_bytes(total_rows: int, K: int, D: int, C: int) -> int:
    return int(lib().db_worker_grad_grouped_workspace_bytes(int(total_rows), int(K), int(D), int(C)))


def worker_grad_grouped(X: torch.Tensor, y: torch.Tensor, W: torch.Tensor, offsets: Sequence[int],
                        G: Sequence[torch.Tensor], losses: Optional[torch.Tensor], workspace: torch.Tensor,
                        stream: Optional[torch.cuda.Stream] = None) -> None:
    """db_worker_grad_grouped: every worker's gradient (rows offsets[w]:offsets[w+1] of X, y) in three launches."""
    K = len(G)
    rows, D = X.shape
    D2, C = W.shape
    if len(offsets) != K + 1 or D2 != D or y.numel() != rows or int(offsets[-1]) != rows:
        raise ValueError("shape mismatch")
    for g in G:
        if tuple(g.shape) != (D, C):
            raise ValueError("G[w] must be [D, C]")
    table = (c_void_p * K)(*[_dev_ptr(g, torch.float32, "G[w]") for g in G])
    _check(lib().db_worker_grad_grouped(
        _dev_ptr(X, torch.float32, "X"), _dev_ptr(y, torch.int32, "y"), _dev_ptr(W, torch.float32, "W"),
        ctypes.cast(_i32_array(offsets), c_void_p), K, D, C, ctypes.cast(table, c_void_p),
        _dev_ptr(losses, torch.float32, "losses"), workspace.data_ptr(),
        workspace.numel() * workspace.element_size(), _stream_ptr(stream)))


def contract_f32(A: torch.Tensor, B: torch.Tensor, out: torch.Tensor, status: torch.Tensor,
                 stream: Optional[torch.cuda.Stream] = None) -> None:
    """db_contract_f32: out[m, n] = sum_k A[m, k] * B[n, k] for 2-D fp32 CUDA tensors of any strides."""
    M, K = A.shape
    N, K2 = B.shape
    if K2 != K or tuple(out.shape) != (M, N):
        raise ValueError("shape mismatch")
    for t in (A, B, out):
        if not t.is_cuda or t.dtype != torch.float32:
            raise TypeError("A, B, out must be float32 CUDA tensors")
    _check(lib().db_contract_f32(
        A.data_ptr(), A.stride(0), A.stride(1), B.data_ptr(), B.stride(0), B.stride(1), out.data_ptr(),
        out.stride(0), out.stride(1), M, N, K, _dev_ptr(status, torch.int32, "status"), _stream_ptr(stream)))


def worker_grad_status(workspace: torch.Tensor) -> int:
    """The status word at the start of a db_worker_grad workspace (0 = every internal wait completed)."""
    return int(workspace[:4].view(torch.int32).item())


def controller_step(b: Sequence[int], throughputs: Sequence[float], kp: float,
                    b_min: Optional[Sequence[int]] = None,
                    b_max: Optional[Sequence[int]] = None) -> list:
    """db_controller_step_ex: one proportional-control adjustment; returns the new batch sizes."""
    K = len(b)
    if len(throughputs) != K:
        raise ValueError("len(throughputs) != len(b)")
    arr = _i32_array(b)
    xs = (c_double * K)(*[float(x) for x in throughputs])
    lo = None if b_min is None else ctypes.cast(_i32_array(b_min), c_void_p)
    hi = None if b_max is None else ctypes.cast(_i32_array(b_max), c_void_p)
    _check(lib().db_controller_step_ex(ctypes.cast(arr, c_void_p), ctypes.cast(xs, c_void_p), K,
                                       float(kp), lo, hi))
    return list(arr)


def static_allocate(throughputs: Sequence[float], b0: int, b_min: Optional[Sequence[int]] = None,
                    b_max: Optional[Sequence[int]] = None) -> list:
    """db_static_allocate: throughput-proportional batch sizes that keep the global batch K * b0."""
    K = len(throughputs)
    xs = (c_double * K)(*[float(x) for x in throughputs])
    out = (c_int32 * K)()
    lo = None if b_min is None else ctypes.cast(_i32_array(b_min), c_void_p)
    hi = None if b_max is None else ctypes.cast(_i32_array(b_max), c_void_p)
    _check(lib().db_static_allocate(ctypes.cast(xs, c_void_p), K, int(b0), lo, hi, ctypes.cast(out, c_void_p)))
    return list(out)


class Controller:
    """db_controller: the stabilised batch-size controller (EWMA, bounds, dead-band)."""

    def __init__(self, b0: Sequence[int], kp: float = 1.0, alpha: float = 0.5, dead_band: float = 0.05,
                 b_min: Optional[Sequence[int]] = None, b_max: Optional[Sequence[int]] = None,
                 adaptive_b_max: bool = False):
        self.K = len(b0)
        self._h = c_void_p()
        lo = None if b_min is None else ctypes.cast(_i32_array(b_min), c_void_p)
        hi = None if b_max is None else ctypes.cast(_i32_array(b_max), c_void_p)
        _check(lib().db_controller_create(ctypes.byref(self._h), ctypes.cast(_i32_array(b0), c_void_p), self.K,
                                          float(kp), float(alpha), float(dead_band), lo, hi, int(adaptive_b_max)))

    def observe(self, iteration_times: Sequence[float]):
        """Returns (batch sizes in force, whether they were readjusted)."""
        ts = (c_double * self.K)(*[float(t) for t in iteration_times])
        out = (c_int32 * self.K)()
        changed = c_int32(0)
        _check(lib().db_controller_observe(self._h, ctypes.cast(ts, c_void_p), ctypes.cast(out, c_void_p),
                                           ctypes.byref(changed)))
        return list(out), bool(changed.value)

    def close(self) -> None:
        if self._h:
            lib().db_controller_destroy(self._h)
            self._h = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class MultiTensorPlan:
    """db_multi_plan: the momentum step over a fixed list of separately allocated tensors.

    grads[k][t] is worker k's gradient of tensor t; params[t], momentum[t] its fp32 state.
    """

    def __init__(self, grads: Sequence[Sequence[torch.Tensor]], params: Sequence[torch.Tensor],
                 momentum: Sequence[torch.Tensor], stream: Optional[torch.cuda.Stream] = None):
        K, T = len(grads), len(params)
        gdt = grads[0][0].dtype
        self.K = K
        sizes = (c_int64 * T)(*[int(p.numel()) for p in params])
        gtab = (c_void_p * (K * T))(*[_dev_ptr(grads[k][t], gdt, "grads[k][t]") for k in range(K) for t in range(T)])
        ptab = (c_void_p * T)(*[_dev_ptr(p, torch.float32, "params[t]") for p in params])
        vtab = (c_void_p * T)(*[_dev_ptr(v, torch.float32, "momentum[t]") for v in momentum])
        for k in range(K):
            for t in range(T):
                if grads[k][t].numel() != params[t].numel():
                    raise ValueError("gradient and parameter sizes differ")
        code = _dtype_code(gdt)
        nbytes = int(lib().db_multi_plan_device_bytes(K, code, ctypes.cast(sizes, c_void_p), T))
        self.table = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=params[0].device)
        self._keep = (list(params), list(momentum), [list(g) for g in grads])   # the plan stores raw pointers
        self._h = c_void_p()
        _check(lib().db_multi_plan_create(ctypes.byref(self._h), ctypes.cast(gtab, c_void_p), code, K,
                                          ctypes.cast(sizes, c_void_p), T, ctypes.cast(ptab, c_void_p),
                                          ctypes.cast(vtab, c_void_p), self.table.data_ptr(), self.table.numel(),
                                          _stream_ptr(stream)))

    def step(self, b: Sequence[int], lr: float, mu: float, grad_sqnorm: Optional[torch.Tensor] = None,
             stream: Optional[torch.cuda.Stream] = None) -> None:
        """db_aggregate_update_multi: one launch over every tensor of the plan."""
        if len(b) != self.K:
            raise ValueError("len(b) != K")
        _check(lib().db_aggregate_update_multi(self._h, ctypes.cast(_i32_array(b), c_void_p), float(lr), float(mu),
                                               _dev_ptr(grad_sqnorm, torch.float64, "grad_sqnorm"),
                                               _stream_ptr(stream)))

    def close(self) -> None:
        if self._h:
            lib().db_multi_plan_destroy(self._h)
            self._h = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
