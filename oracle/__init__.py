"""CPU checker for the Ternary-SVD linear map (test infrastructure only).

`forward(U, S, V, x, x_dtype)` evaluates y = U (diag(S) (V x)) exactly as the
paper states it (display after Eq. 2; cost table S1): additions and
subtractions at the nonzeros of V, K multiplications by S, additions and
subtractions at the nonzeros of U.  The arithmetic is in `tsvd_oracle.c`
(plain C, IEEE double; 64-bit integers for the V-stage of int8 activations).

Nothing in the GPU library imports this package, and this package imports
nothing of the GPU library.  Only the tests, the smoke check and the CPU
baseline leg of the benchmark may call it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tsvd_oracle.c")
_LIB = os.path.join(_HERE, "libtsvd_oracle.so")
_lib: Optional[ctypes.CDLL] = None


def build(force: bool = False) -> str:
    """Compile the C checker with gcc (-O2 -fopenmp) next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i8p = ctypes.POINTER(ctypes.c_int8)
        f32p = ctypes.POINTER(ctypes.c_float)
        f64p = ctypes.POINTER(ctypes.c_double)
        i64p = ctypes.POINTER(ctypes.c_longlong)
        lib.tsvd_oracle_forward_f64.argtypes = [i8p, f32p, i8p, ctypes.c_int, ctypes.c_int,
                                                ctypes.c_int, f64p, ctypes.c_int, f32p, f64p, f64p, i64p]
        lib.tsvd_oracle_forward_f64.restype = ctypes.c_int
        lib.tsvd_oracle_forward_i8.argtypes = [i8p, f32p, i8p, ctypes.c_int, ctypes.c_int,
                                               ctypes.c_int, i8p, ctypes.c_int, f32p, f64p, i64p, i64p]
        lib.tsvd_oracle_forward_i8.restype = ctypes.c_int
        lib.tsvd_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the checker will use."""
    return int(_load().tsvd_oracle_threads())


@dataclass
class OracleResult:
    y: np.ndarray            # float64 [B,M]
    zraw: np.ndarray         # V x before the S scale: float64 [B,K], or int64 for int8 x
    adds: int                # additions + subtractions performed (Table S1, column "+")
    muls: int                # multiplications performed (Table S1, column "x")


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def forward(U: np.ndarray, S: np.ndarray, V: np.ndarray, x: np.ndarray,
            bias: Optional[np.ndarray] = None) -> OracleResult:
    """y = U (diag(S) (V x)) (+ bias) for a token-major batch x [B,N].

    U int8 [M,K], V int8 [K,N], S float32 [K].  x is float64 (already widened
    exactly from its storage type) or int8 (integer V-stage).  bias: None, or
    float32 [M] (the converted layer keeps the original layer's bias: the
    supplement's architecture listing has bias=True on every layer).
    """
    lib = _load()
    U = np.ascontiguousarray(U, dtype=np.int8)
    V = np.ascontiguousarray(V, dtype=np.int8)
    S = np.ascontiguousarray(S, dtype=np.float32)
    M, K = U.shape
    K2, N = V.shape
    if K2 != K or S.shape != (K,):
        raise ValueError("shape mismatch between U, S, V")
    if x.ndim != 2 or x.shape[1] != N:
        raise ValueError("x must be [B,N]")
    B = x.shape[0]
    bp = None
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.float32)
        if bias.shape != (M,):
            raise ValueError("bias must be [M]")
        bp = _ptr(bias, ctypes.c_float)
    y = np.zeros((B, M), dtype=np.float64)
    counts = np.zeros(2, dtype=np.int64)
    if x.dtype == np.int8:
        xx = np.ascontiguousarray(x)
        zraw = np.zeros((B, K), dtype=np.int64)
        rc = lib.tsvd_oracle_forward_i8(_ptr(U, ctypes.c_int8), _ptr(S, ctypes.c_float),
                                        _ptr(V, ctypes.c_int8), M, K, N,
                                        _ptr(xx, ctypes.c_int8), B, bp, _ptr(y, ctypes.c_double),
                                        _ptr(zraw, ctypes.c_longlong),
                                        _ptr(counts, ctypes.c_longlong))
    elif x.dtype == np.float64:
        xx = np.ascontiguousarray(x)
        zraw = np.zeros((B, K), dtype=np.float64)
        rc = lib.tsvd_oracle_forward_f64(_ptr(U, ctypes.c_int8), _ptr(S, ctypes.c_float),
                                         _ptr(V, ctypes.c_int8), M, K, N,
                                         _ptr(xx, ctypes.c_double), B, bp, _ptr(y, ctypes.c_double),
                                         _ptr(zraw, ctypes.c_double),
                                         _ptr(counts, ctypes.c_longlong))
    else:
        raise TypeError("x must be float64 (widened exactly) or int8")
    if rc == 1:
        raise ValueError("U and V must hold only -1, 0, +1")
    if rc != 0:
        raise MemoryError("oracle allocation failed")
    return OracleResult(y=y, zraw=zraw, adds=int(counts[0]), muls=int(counts[1]))
