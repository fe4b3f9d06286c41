"""Python face of the CPU oracle (fp64, plain C loops).  TEST INFRASTRUCTURE ONLY.

Only the tests, ``__graft_entry__.smoke()`` and ``bench.py``'s CPU-baseline leg may import
this package.  It never imports the CUDA package and shares no code with it.  All
arithmetic lives in ``osdp_oracle.c``; this file only marshals numpy arrays.

Inputs are bf16 bit patterns (uint16 arrays) or fp32 arrays; they are widened exactly to
fp64 before any arithmetic.  Results are fp64 numpy arrays.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

from .build import build as _build

ACT_NONE, ACT_GELU_TANH, ACT_GELU_ERF = 0, 1, 2
SPLIT_OUT, SPLIT_RED = 0, 1
OK, BAD_SPLIT, BAD_ARG = 0, 1, 2

_lib = None
_dp = ctypes.POINTER(ctypes.c_double)


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build())
        _lib.orc_gelu.restype = ctypes.c_double
        _lib.orc_gelu.argtypes = [ctypes.c_double, ctypes.c_int]
        _lib.orc_gelu_grad.restype = ctypes.c_double
        _lib.orc_gelu_grad.argtypes = [ctypes.c_double, ctypes.c_int]
    return _lib


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__("oracle returned status %d" % code)
        self.code = code


def _check(rc):
    if rc != OK:
        raise OracleError(rc)


def _p(a):
    return None if a is None else a.ctypes.data_as(_dp)


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def bf16_to_f64(bits) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp64, via the C helper."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float64)
    lib().orc_bf16_to_f64(bits.ctypes.data_as(ctypes.c_void_p), _p(out), ctypes.c_size_t(bits.size))
    return out


def f32_to_bf16(x) -> np.ndarray:
    """fp32 -> bf16 bit patterns, round to nearest even, via the C helper."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().orc_f32_to_bf16(x.ctypes.data_as(ctypes.c_void_p), out.ctypes.data_as(ctypes.c_void_p),
                          ctypes.c_size_t(x.size))
    return out


def e4m3_to_f64(bits) -> np.ndarray:
    """Exact widening of fp8 e4m3 bit patterns (uint8) to fp64, via the C helper."""
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    out = np.empty(bits.shape, dtype=np.float64)
    lib().orc_e4m3_to_f64(bits.ctypes.data_as(ctypes.c_void_p), _p(out), ctypes.c_size_t(bits.size))
    return out


def as_f64(a) -> np.ndarray:
    """uint16 arrays are bf16 bit patterns, uint8 arrays fp8 e4m3 bit patterns; anything else is numeric."""
    if a is None:
        return None
    a = np.asarray(a)
    if a.dtype == np.uint16:
        return bf16_to_f64(a)
    if a.dtype == np.uint8:
        return e4m3_to_f64(a)
    return np.ascontiguousarray(a, dtype=np.float64)


def gelu(x: float, act: int) -> float:
    return lib().orc_gelu(float(x), int(act))


def gelu_grad(x: float, act: int) -> float:
    return lib().orc_gelu_grad(float(x), int(act))


def slice_range(D: int, k: int, s: int):
    b, e = ctypes.c_long(), ctypes.c_long()
    _check(lib().orc_slice_range(ctypes.c_long(D), int(k), int(s), ctypes.byref(b), ctypes.byref(e)))
    return b.value, e.value


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _l(v):
    return ctypes.c_long(int(v))


def linear_fwd(x, w, b=None, act=ACT_NONE, k=1, split_dim=None):
    """Returns (Z, Y) in fp64.  split_dim None -> the unsplit definition; else the slice loops."""
    X, W, B = as_f64(x), as_f64(w), as_f64(b)
    M, K = X.shape
    N = W.shape[0]
    assert W.shape == (N, K)
    Z = np.empty((M, N)); Y = np.empty((M, N))
    if split_dim is None:
        _check(lib().orc_linear_fwd(_p(X), _p(W), _p(B), _l(M), _l(N), _l(K), int(act), _p(Z), _p(Y)))
    else:
        _check(lib().orc_split_linear_fwd(_p(X), _p(W), _p(B), _l(M), _l(N), _l(K), int(k), int(split_dim),
                                          int(act), _p(Z), _p(Y)))
    return Z, Y


def linear_bwd(dy, x, w, z=None, act=ACT_NONE, k=1, split_dim=None):
    """Returns (dX, dW, db) in fp64; z is the forward's pre-activation (needed when act != none)."""
    DY, X, W, Z = as_f64(dy), as_f64(x), as_f64(w), _f64(z)
    M, K = X.shape
    N = W.shape[0]
    dX = np.empty((M, K)); dW = np.empty((N, K)); db = np.empty((N,))
    if split_dim is None:
        _check(lib().orc_linear_bwd(_p(DY), _p(X), _p(W), _p(Z), _l(M), _l(N), _l(K), int(act),
                                    _p(dX), _p(dW), _p(db)))
    else:
        _check(lib().orc_split_linear_bwd(_p(DY), _p(X), _p(W), _p(Z), _l(M), _l(N), _l(K), int(k),
                                          int(split_dim), int(act), _p(dX), _p(dW), _p(db)))
    return dX, dW, db


def mlp_fwd(x, w1, b1, w2, b2, act=ACT_GELU_TANH, k=None):
    """Y (fp64) of Linear->GeLU->Linear; k None -> unsplit (also returns Z1), else split along ffn."""
    X, W1, B1, W2, B2 = as_f64(x), as_f64(w1), as_f64(b1), as_f64(w2), as_f64(b2)
    M, H = X.shape
    F = W1.shape[0]
    assert W1.shape == (F, H) and W2.shape == (H, F)
    Y = np.empty((M, H))
    if k is None:
        Z1 = np.empty((M, F))
        _check(lib().orc_mlp_fwd(_p(X), _p(W1), _p(B1), _p(W2), _p(B2), _l(M), _l(H), _l(F), int(act),
                                 _p(Z1), _p(Y)))
        return Z1, Y
    _check(lib().orc_split_mlp_fwd(_p(X), _p(W1), _p(B1), _p(W2), _p(B2), _l(M), _l(H), _l(F), int(k),
                                   int(act), _p(Y)))
    return None, Y


def mlp_bwd(dy, x, w1, b1, w2, act=ACT_GELU_TANH, k=None):
    """(dX, dW1, db1, dW2, db2) in fp64; k None -> unsplit, else split along ffn."""
    DY, X, W1, B1, W2 = as_f64(dy), as_f64(x), as_f64(w1), as_f64(b1), as_f64(w2)
    M, H = X.shape
    F = W1.shape[0]
    dX = np.empty((M, H)); dW1 = np.empty((F, H)); db1 = np.empty((F,))
    dW2 = np.empty((H, F)); db2 = np.empty((H,))
    if k is None:
        _check(lib().orc_mlp_bwd(_p(DY), _p(X), _p(W1), _p(B1), _p(W2), _l(M), _l(H), _l(F), int(act),
                                 _p(dX), _p(dW1), _p(db1), _p(dW2), _p(db2)))
    else:
        _check(lib().orc_split_mlp_bwd(_p(DY), _p(X), _p(W1), _p(B1), _p(W2), _l(M), _l(H), _l(F), int(k),
                                       int(act), _p(dX), _p(dW1), _p(db1), _p(dW2), _p(db2)))
    return dX, dW1, db1, dW2, db2
