"""fp64 CPU oracle -- TEST INFRASTRUCTURE ONLY.

ctypes front end of oracle/ref_oracle.c.  Importable by tests, the smoke check
and the CPU-baseline leg of the benchmark; never by the product package, and
it imports nothing from it.  Arrays are numpy; gradients are float32 arrays or
uint16 arrays holding bf16 bit patterns.
"""
import ctypes
import os
from ctypes import POINTER, c_double, c_int32, c_int64, c_void_p

import numpy as np

from .build import build as _build

REF_OK, REF_ERR_ARG, REF_ERR_INFEASIBLE = 0, 2, 4
F32, BF16 = 0, 1

_lib = None


def lib():
    global _lib
    if _lib is None:
        # REF_ORACLE_LIB: a library built elsewhere from a (deliberately altered) copy of
        # ref_oracle.c -- how tests/test_oracle_mutations.py shows that the pins catch mistakes.
        L = ctypes.CDLL(os.environ.get("REF_ORACLE_LIB") or _build())
        L.ref_weights.argtypes = [c_void_p, c_int32, c_void_p]
        L.ref_aggregate_update.argtypes = [
            c_void_p, c_int32, c_void_p, c_int32, c_int64, c_void_p, c_void_p,
            c_double, c_double, c_void_p, c_void_p]
        L.ref_aggregate_adam.argtypes = [
            c_void_p, c_int32, c_void_p, c_int32, c_int64, c_void_p, c_void_p,
            c_void_p, c_double, c_double, c_double, c_double, c_int64,
            c_void_p, c_void_p]
        L.ref_worker_grad.argtypes = [
            c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p,
            c_void_p]
        L.ref_controller_targets.argtypes = [
            c_void_p, c_void_p, c_int32, c_double, c_void_p]
        L.ref_controller_step.argtypes = [
            c_void_p, c_void_p, c_int32, c_double, c_void_p, c_void_p]
        L.ref_static_allocate.argtypes = [
            c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p]
        L.ref_controller_observe.argtypes = [
            c_void_p, c_void_p, c_int32, c_double, c_double, c_double,
            c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int32,
            c_void_p, c_void_p, c_void_p]
        L.ref_num_threads.restype = ctypes.c_int
        L.ref_set_num_threads.argtypes = [ctypes.c_int]
        _lib = L
    return _lib


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__(f"oracle returned status {code}")
        self.code = code


def _check(rc):
    if rc != REF_OK:
        raise OracleError(rc)


def _ptr(a):
    return None if a is None else a.ctypes.data


def _i32(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.int32))


def _f64(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _grad_table(grads):
    """K contiguous 1-D arrays (float32, or uint16 = bf16 bits) -> pointer table."""
    arrs = [np.ascontiguousarray(g).reshape(-1) for g in grads]
    dt = arrs[0].dtype
    if dt == np.float32:
        code = F32
    elif dt == np.uint16:
        code = BF16
    else:
        raise TypeError("gradients must be float32 or uint16 (bf16 bits)")
    n = arrs[0].size
    for a in arrs:
        if a.dtype != dt or a.size != n:
            raise ValueError("gradient buffers differ in dtype or length")
    table = (c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])
    return arrs, table, code, n


def weights(b):
    b = _i32(b)
    lam = np.empty(b.size, dtype=np.float64)
    _check(lib().ref_weights(_ptr(b), b.size, _ptr(lam)))
    return lam


def aggregate_update(grads, b, p, v, lr, mu, want_g=False):
    """In-place fp64 update of p, v (float64 arrays).  Returns (g or None, sum g^2)."""
    arrs, table, code, n = _grad_table(grads)
    b = _i32(b)
    if b.size != len(arrs):
        raise ValueError("len(b) != K")
    assert p.dtype == np.float64 and v.dtype == np.float64
    assert p.flags.c_contiguous and v.flags.c_contiguous
    assert p.size == n and v.size == n
    g = np.empty(n, dtype=np.float64) if want_g else None
    sq = c_double(0.0)
    _check(lib().ref_aggregate_update(
        ctypes.cast(table, c_void_p), code, _ptr(b), b.size, n, _ptr(p),
        _ptr(v), float(lr), float(mu), _ptr(g), ctypes.addressof(sq)))
    return g, sq.value


def aggregate_adam(grads, b, p, m, u, lr, beta1, beta2, eps, t, want_g=False):
    arrs, table, code, n = _grad_table(grads)
    b = _i32(b)
    for a in (p, m, u):
        assert a.dtype == np.float64 and a.flags.c_contiguous and a.size == n
    g = np.empty(n, dtype=np.float64) if want_g else None
    sq = c_double(0.0)
    _check(lib().ref_aggregate_adam(
        ctypes.cast(table, c_void_p), code, _ptr(b), b.size, n, _ptr(p),
        _ptr(m), _ptr(u), float(lr), float(beta1), float(beta2), float(eps),
        int(t), _ptr(g), ctypes.addressof(sq)))
    return g, sq.value


def worker_grad(X, y, W):
    """Mean CE gradient [D, C] (float64) and mean loss of a linear-softmax model."""
    X = np.ascontiguousarray(X, dtype=np.float32)
    W = np.ascontiguousarray(W, dtype=np.float32)
    y = _i32(y)
    n, D = X.shape
    D2, C = W.shape
    assert D == D2 and y.size == n
    G = np.empty((D, C), dtype=np.float64)
    loss = c_double(0.0)
    _check(lib().ref_worker_grad(_ptr(X), _ptr(y), _ptr(W), n, D, C, _ptr(G),
                                 ctypes.addressof(loss)))
    return G, loss.value


def controller_targets(b, X, kp):
    b = _i32(b)
    X = _f64(X)
    q = np.empty(b.size, dtype=np.float64)
    _check(lib().ref_controller_targets(_ptr(b), _ptr(X), b.size, float(kp),
                                        _ptr(q)))
    return q


def controller_step(b, X, kp, b_min=None, b_max=None):
    b = _i32(b).copy()
    X = _f64(X)
    lo = None if b_min is None else _i32(b_min)
    hi = None if b_max is None else _i32(b_max)
    _check(lib().ref_controller_step(_ptr(b), _ptr(X), b.size, float(kp),
                                     _ptr(lo), _ptr(hi)))
    return b


def static_allocate(X, b0, b_min=None, b_max=None):
    X = _f64(X)
    lo = None if b_min is None else _i32(b_min)
    hi = None if b_max is None else _i32(b_max)
    b = np.empty(X.size, dtype=np.int32)
    _check(lib().ref_static_allocate(_ptr(X), X.size, int(b0), _ptr(lo),
                                     _ptr(hi), _ptr(b)))
    return b


class ControllerState:
    """State of the stabilised controller: batch sizes, EWMA, samples since readjust."""

    def __init__(self, b, kp=1.0, alpha=0.5, dmin=0.05, b_min=None, b_max=None, adaptive=False):
        self.adaptive = bool(adaptive)
        self.b = _i32(b).copy()
        self.prev_b = np.zeros(self.b.size, dtype=np.int32)
        self.prev_X = np.zeros(self.b.size, dtype=np.float64)
        self.learnt_max = np.zeros(self.b.size, dtype=np.int32)
        self.kp, self.alpha, self.dmin = float(kp), float(alpha), float(dmin)
        self.lo = None if b_min is None else _i32(b_min)
        self.hi = None if b_max is None else _i32(b_max)
        self.ewma = np.zeros(self.b.size, dtype=np.float64)
        self.n_since = np.zeros(1, dtype=np.int32)

    def observe(self, t):
        t = _f64(t)
        changed = np.zeros(1, dtype=np.int32)
        _check(lib().ref_controller_observe(
            _ptr(self.b), _ptr(t), self.b.size, self.kp, self.alpha, self.dmin,
            _ptr(self.lo), _ptr(self.hi), _ptr(self.ewma), _ptr(self.n_since),
            _ptr(changed), int(self.adaptive), _ptr(self.prev_b), _ptr(self.prev_X),
            _ptr(self.learnt_max)))
        return bool(changed[0])


def num_threads():
    return lib().ref_num_threads()


def set_num_threads(n):
    lib().ref_set_num_threads(int(n))
