"""TEST INFRASTRUCTURE: Python face of the fp64 GEMM oracle (see gemm_oracle.c).

C[i][j] = sum_k A[i][k] * B[k][j] with A (M x K) and B (K x N) given as bf16 bit
patterns (numpy uint16, row-major) and C in float64 - the plain definition of the
product that the persistent GEMM of Section 7.1.2 must reproduce.
"""
from __future__ import annotations

import ctypes

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        i64 = ctypes.c_int64
        p = ctypes.c_void_p
        lib.oracle_gemm_bruteforce.argtypes = [p, p, p, i64, i64, i64]
        lib.oracle_gemm_bruteforce.restype = None
        lib.oracle_gemm_blocked.argtypes = [p, p, p, i64, i64, i64]
        lib.oracle_gemm_blocked.restype = None
        lib.oracle_gemm_block.argtypes = [p, p, p, i64, i64, i64, i64, i64, i64, i64]
        lib.oracle_gemm_block.restype = None
        lib.oracle_gemm_entry.argtypes = [p, p, i64, i64, i64, i64]
        lib.oracle_gemm_entry.restype = ctypes.c_double
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _check(A, B):
    A = np.ascontiguousarray(A, dtype=np.uint16)
    B = np.ascontiguousarray(B, dtype=np.uint16)
    assert A.ndim == 2 and B.ndim == 2 and A.shape[1] == B.shape[0]
    return A, B


def gemm_bruteforce(A, B) -> np.ndarray:
    """Single-thread triple loop; use for shapes up to about 256^3."""
    A, B = _check(A, B)
    M, K = A.shape
    N = B.shape[1]
    C = np.empty((M, N), dtype=np.float64)
    _load().oracle_gemm_bruteforce(A.ctypes.data, B.ctypes.data, C.ctypes.data, M, N, K)
    return C


def gemm_blocked(A, B) -> np.ndarray:
    """Same sums in the same (ascending-k) order, row panels spread over host threads."""
    A, B = _check(A, B)
    M, K = A.shape
    N = B.shape[1]
    C = np.empty((M, N), dtype=np.float64)
    _load().oracle_gemm_blocked(A.ctypes.data, B.ctypes.data, C.ctypes.data, M, N, K)
    return C


def gemm_block(A, B, row0, row1, col0, col1) -> np.ndarray:
    """Rows [row0,row1) x columns [col0,col1) of C only."""
    A, B = _check(A, B)
    M, K = A.shape
    N = B.shape[1]
    out = np.empty((row1 - row0, col1 - col0), dtype=np.float64)
    _load().oracle_gemm_block(A.ctypes.data, B.ctypes.data, out.ctypes.data, M, N, K,
                              row0, row1, col0, col1)
    return out


def gemm_entries(A, B, rows, cols) -> np.ndarray:
    """C[rows[t]][cols[t]] one entry at a time (sampled checks at full size)."""
    A, B = _check(A, B)
    K = A.shape[1]
    N = B.shape[1]
    lib = _load()
    return np.array([lib.oracle_gemm_entry(A.ctypes.data, B.ctypes.data, N, K, int(i), int(j))
                     for i, j in zip(rows, cols)], dtype=np.float64)


def num_threads() -> int:
    return int(_load().oracle_num_threads())
