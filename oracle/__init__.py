"""ctypes binding of the CPU oracle (plain Gustavson SpGEMM, Algorithm 1 / Eq. 1 of the paper).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU-baseline / reference
legs may import this package; the CUDA product never does, and this package imports nothing from
the product.  See ``gustavson_oracle.cpp`` for what is computed and in which precision.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gustavson_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA, no third-party code)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        p, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        lib.oracle_row_products.restype = i64
        lib.oracle_row_products.argtypes = [i64, p, p, p, p]
        common = [i64, i64, p, p, p, i64, i64, p, p, p, i32, i64, i64, i32]
        lib.oracle_spgemm_count.restype = i32
        lib.oracle_spgemm_count.argtypes = common + [p]
        lib.oracle_spgemm_fill.restype = i32
        lib.oracle_spgemm_fill.argtypes = common + [p, p, p, p]
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _dtype_code(dt) -> int:
    dt = np.dtype(dt)
    if dt == np.float32:
        return 0
    if dt == np.float64:
        return 1
    raise TypeError(f"unsupported value dtype {dt}")


def _check(M) -> None:
    assert M.row_ptr.dtype == np.int64 and M.col.dtype == np.int32
    assert M.row_ptr.flags.c_contiguous and M.col.flags.c_contiguous and M.val.flags.c_contiguous


@dataclass
class OracleRows:
    """Rows [r0, r1) of C: local ``row_ptr`` (starts at 0), ascending ``col`` per row, ``val`` =
    sum of products and ``abs`` = sum of |products| (both float64)."""

    r0: int
    r1: int
    row_ptr: np.ndarray
    col: np.ndarray
    val: np.ndarray
    abs: np.ndarray
    threads: int

    @property
    def nnz(self) -> int:
        return int(self.row_ptr[-1])


def row_products(A, B) -> np.ndarray:
    """IP_i = sum over stored entries j of A[i,:] of nnz(B[A.col[j],:]) (Section III-A)."""
    _check(A), _check(B)
    assert A.n_cols == B.n_rows
    ip = np.empty(A.n_rows, dtype=np.int64)
    _load().oracle_row_products(A.n_rows, _ptr(A.row_ptr), _ptr(A.col), _ptr(B.row_ptr), _ptr(ip))
    return ip


def _common_args(A, B, r0, r1, threads):
    return [A.n_rows, A.n_cols, _ptr(A.row_ptr), _ptr(A.col), _ptr(A.val),
            B.n_rows, B.n_cols, _ptr(B.row_ptr), _ptr(B.col), _ptr(B.val),
            _dtype_code(A.val.dtype), r0, r1, threads]


def spgemm_row_counts(A, B, r0: int = 0, r1: int | None = None, threads: int = 0) -> np.ndarray:
    """Number of entries of C[i,:] for i in [r0, r1) (symbolic product)."""
    _check(A), _check(B)
    assert A.val.dtype == B.val.dtype and A.n_cols == B.n_rows
    r1 = A.n_rows if r1 is None else r1
    counts = np.empty(r1 - r0, dtype=np.int64)
    rc = _load().oracle_spgemm_count(*_common_args(A, B, r0, r1, threads), _ptr(counts))
    if rc < 0:
        raise ValueError(f"oracle_spgemm_count failed ({rc})")
    return counts


def spgemm(A, B, r0: int = 0, r1: int | None = None, threads: int = 0) -> OracleRows:
    """Rows [r0, r1) of C = A * B by Algorithm 1 (sorted rows, structural zeros kept)."""
    r1 = A.n_rows if r1 is None else r1
    counts = spgemm_row_counts(A, B, r0, r1, threads)
    row_ptr = np.zeros(r1 - r0 + 1, dtype=np.int64)
    np.cumsum(counts, out=row_ptr[1:])
    nnz = int(row_ptr[-1])
    col = np.empty(nnz, dtype=np.int32)
    val = np.empty(nnz, dtype=np.float64)
    ab = np.empty(nnz, dtype=np.float64)
    used = _load().oracle_spgemm_fill(*_common_args(A, B, r0, r1, threads), _ptr(row_ptr),
                                      _ptr(col), _ptr(val), _ptr(ab))
    if used < 0:
        raise ValueError(f"oracle_spgemm_fill failed ({used})")
    return OracleRows(r0, r1, row_ptr, col, val, ab, used)
