"""Small host-side helpers for the tests (no SpGEMM arithmetic of the product or the oracle)."""
import numpy as np

from gen import CSR


def csr_from_pattern(pattern: np.ndarray, values: np.ndarray, dtype) -> CSR:
    """CSR holding exactly the entries where ``pattern`` is True (explicit zeros allowed)."""
    n, m = pattern.shape
    rows, cols = np.nonzero(pattern)  # row-major order => ascending columns per row
    row_ptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(np.bincount(rows, minlength=n), out=row_ptr[1:])
    return CSR(n, m, row_ptr, cols.astype(np.int32), values[rows, cols].astype(dtype))


def random_csr(rng, n, m, density, dtype, zero_fraction=0.0) -> CSR:
    pattern = rng.random((n, m)) < density
    values = rng.uniform(-1, 1, size=(n, m))
    if zero_fraction:
        values[rng.random((n, m)) < zero_fraction] = 0.0
    return csr_from_pattern(pattern, values, dtype)


def identity(n, dtype) -> CSR:
    return CSR(n, n, np.arange(n + 1, dtype=np.int64), np.arange(n, dtype=np.int32), np.ones(n, dtype=dtype))


def permutation(perm: np.ndarray, dtype) -> CSR:
    """P with P[i, perm[i]] = 1, so (P*A)[i,:] = A[perm[i],:]."""
    n = perm.size
    return CSR(n, n, np.arange(n + 1, dtype=np.int64), perm.astype(np.int32), np.ones(n, dtype=dtype))


def transpose(A: CSR) -> CSR:
    rows = np.repeat(np.arange(A.n_rows, dtype=np.int64), np.diff(A.row_ptr))
    order = np.lexsort((rows, A.col))
    row_ptr = np.zeros(A.n_cols + 1, dtype=np.int64)
    np.cumsum(np.bincount(A.col, minlength=A.n_cols), out=row_ptr[1:])
    return CSR(A.n_cols, A.n_rows, row_ptr, rows[order].astype(np.int32), A.val[order].copy())


def dense_product(A: CSR, B: CSR):
    """Brute force on densified inputs: (pattern, sum, abs-sum) by the textbook triple loop,
    written with dense float64 matrix products (exact for fp32 inputs up to summation order)."""
    def dense(M):
        D = np.zeros((M.n_rows, M.n_cols), dtype=np.float64)
        P = np.zeros((M.n_rows, M.n_cols), dtype=np.float64)
        rows = np.repeat(np.arange(M.n_rows), np.diff(M.row_ptr))
        D[rows, M.col] = M.val.astype(np.float64)
        P[rows, M.col] = 1.0
        return D, P
    Ad, Ap = dense(A)
    Bd, Bp = dense(B)
    return (Ap @ Bp) > 0, Ad @ Bd, np.abs(Ad) @ np.abs(Bd)
