"""The plain definition C = A.B in int64 (CPU oracle; test infrastructure only).

`matmul_i64` runs oracle/matmul_i64.c (built on first use with gcc -O2 -fopenmp into
oracle/liboracle_matmul.so) and `matmul_i64_numpy` is the same definition through
numpy's integer matmul, kept as an independent cross-check of the C loop nest.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "matmul_i64.c")
_LIB = os.path.join(_HERE, "liboracle_matmul.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle if it is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        i64, p = ctypes.c_int64, ctypes.c_void_p
        _lib.oracle_matmul_i64.argtypes = [p, p, p, i64, i64, i64]
        _lib.oracle_matmul_i64_ijk.argtypes = [p, p, p, i64, i64, i64]
        _lib.oracle_matmul_i64_rows.argtypes = [p, p, p, i64, i64, i64, i64]
        _lib.oracle_mod_symmetric.argtypes = [p, i64, i64]
        _lib.oracle_matmul_i64_s16_rows.argtypes = [p, p, p, i64, i64, i64, i64]
        _lib.oracle_threads.restype = ctypes.c_int
    return _lib


def threads() -> int:
    return int(_load().oracle_threads())


def _i8(x):
    x = np.ascontiguousarray(x)
    assert x.dtype == np.int8 and x.ndim == 2
    return x


def matmul_i64(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """A: M x K int8, B: K x N int8 -> M x N int64, the exact product."""
    A, B = _i8(A), _i8(B)
    M, K = A.shape
    K2, N = B.shape
    assert K == K2
    C = np.empty((M, N), dtype=np.int64)
    _load().oracle_matmul_i64(A.ctypes.data, B.ctypes.data, C.ctypes.data, M, N, K)
    return C


def matmul_i64_ijk(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """The same product by the textbook (i, j, k) loop nest on one thread."""
    A, B = _i8(A), _i8(B)
    M, K = A.shape
    K2, N = B.shape
    assert K == K2
    C = np.empty((M, N), dtype=np.int64)
    _load().oracle_matmul_i64_ijk(A.ctypes.data, B.ctypes.data, C.ctypes.data, M, N, K)
    return C


def matmul_i64_rows(A: np.ndarray, B: np.ndarray, i0: int, i1: int) -> np.ndarray:
    """Rows i0..i1-1 of the exact product."""
    A, B = _i8(A), _i8(B)
    M, K = A.shape
    _, N = B.shape
    assert 0 <= i0 <= i1 <= M
    C = np.empty((i1 - i0, N), dtype=np.int64)
    _load().oracle_matmul_i64_rows(A.ctypes.data, B.ctypes.data, C.ctypes.data, i0, i1, N, K)
    return C


def matmul_i64_s16(A: np.ndarray, B: np.ndarray, i0: int = 0, i1: int = None) -> np.ndarray:
    """Rows i0..i1-1 (default: all) of the exact product of int16 matrices, int64."""
    A, B = np.ascontiguousarray(A), np.ascontiguousarray(B)
    assert A.dtype == np.int16 and B.dtype == np.int16 and A.shape[1] == B.shape[0]
    M, K = A.shape
    N = B.shape[1]
    i1 = M if i1 is None else i1
    C = np.empty((i1 - i0, N), dtype=np.int64)
    _load().oracle_matmul_i64_s16_rows(A.ctypes.data, B.ctypes.data, C.ctypes.data, i0, i1, N, K)
    return C


def mod_symmetric(C: np.ndarray, m: int) -> np.ndarray:
    """Entrywise symmetric residue mod m (Section 5.3 result form)."""
    out = np.ascontiguousarray(C, dtype=np.int64).copy()
    _load().oracle_mod_symmetric(out.ctypes.data, out.size, m)
    return out


def matmul_i64_numpy(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    return np.asarray(A).astype(np.int64) @ np.asarray(B).astype(np.int64)
