"""Python face of the CPU oracle (``sd2_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Compiles the C file with gcc on first use (``-O2``, no threads, no fast-math)
and exposes its functions on numpy arrays.  Nothing here imports or calls the
CUDA library; only tests, the smoke check and the benchmark's cpu_baseline /
reference arm may import this module.
"""

from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sd2_oracle.c")
_LIB = os.path.join(_HERE, "libsd2_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle; returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        p = ctypes.c_void_p
        i64 = ctypes.c_int64
        lib.sd2o_masked_linear.argtypes = [p, p, p, i64, i64, i64, p, p]
        lib.sd2o_masked_linear.restype = None
        lib.sd2o_roundtrip_ref.argtypes = [p, p, i64, i64, p]
        lib.sd2o_roundtrip_ref.restype = None
        lib.sd2o_nnz.argtypes = [p, p, i64, i64]
        lib.sd2o_nnz.restype = i64
        lib.sd2o_silu_mul.argtypes = [p, p, i64, p]
        lib.sd2o_silu_mul.restype = None
        lib.sd2o_f64_to_bf16_rne.argtypes = [ctypes.c_double]
        lib.sd2o_f64_to_bf16_rne.restype = ctypes.c_uint16
        _lib = lib
    return _lib


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def masked_linear(W, mask, X):
    """``(Y, S)`` fp64 ``[N, M]`` for bf16-pattern ``W [M,K]``, ``mask [M,K]``/None, ``X [N,K]``."""
    W = _u16(W)
    X = _u16(X)
    M, K = W.shape
    N, K2 = X.shape
    assert K == K2
    if mask is not None:
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
        assert mask.shape == (M, K)
    Y = np.empty((N, M), dtype=np.float64)
    S = np.empty((N, M), dtype=np.float64)
    _load().sd2o_masked_linear(_ptr(W), _ptr(mask), _ptr(X), M, K, N, _ptr(Y), _ptr(S))
    return Y, S


def roundtrip_ref(W, mask):
    W = _u16(W)
    M, K = W.shape
    if mask is not None:
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
    out = np.empty((M, K), dtype=np.uint16)
    _load().sd2o_roundtrip_ref(_ptr(W), _ptr(mask), M, K, _ptr(out))
    return out


def nnz(W, mask):
    W = _u16(W)
    M, K = W.shape
    if mask is not None:
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
    return int(_load().sd2o_nnz(_ptr(W), _ptr(mask), M, K))


def silu_mul(g, u):
    g = _u16(g).ravel()
    u = _u16(u).ravel()
    out = np.empty(g.shape, dtype=np.float64)
    _load().sd2o_silu_mul(_ptr(g), _ptr(u), g.size, _ptr(out))
    return out


def f64_to_bf16_rne(v: float) -> int:
    return int(_load().sd2o_f64_to_bf16_rne(float(v)))
