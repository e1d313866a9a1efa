"""Pins for the CPU oracle: every check compares it with something other than itself — brute force
on densified inputs, algebraic identities, closed forms that follow from the stencil geometry, the
definition of the product count, and an independent library routine."""
import numpy as np
import pytest

import gen
import oracle
from helpers import (csr_from_pattern, dense_product, identity, permutation, random_csr, transpose)


def _assert_matches_dense(A, B):
    res = oracle.spgemm(A, B)
    pat, val, ab = dense_product(A, B)
    # structure: exactly the positions reachable by at least one product, ascending per row
    exp_rows, exp_cols = np.nonzero(pat)
    exp_ptr = np.zeros(A.n_rows + 1, dtype=np.int64)
    np.cumsum(np.bincount(exp_rows, minlength=A.n_rows), out=exp_ptr[1:])
    assert np.array_equal(res.row_ptr, exp_ptr)
    assert np.array_equal(res.col, exp_cols.astype(np.int32))
    ev, ea = val[exp_rows, exp_cols], ab[exp_rows, exp_cols]
    assert np.all(np.abs(res.abs - ea) <= 1e-14 * ea + 1e-300)
    assert np.all(np.abs(res.val - ev) <= 4e-15 * ea + 1e-300)


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
@pytest.mark.parametrize("seed", range(6))
def test_brute_force_random_tiny(dtype, seed):
    rng = np.random.default_rng(seed)
    n, k, m = rng.integers(1, 48, size=3)
    A = random_csr(rng, n, k, rng.uniform(0.02, 0.5), dtype, zero_fraction=0.1)
    B = random_csr(rng, k, m, rng.uniform(0.02, 0.5), dtype, zero_fraction=0.1)
    _assert_matches_dense(A, B)


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_brute_force_special_shapes(dtype):
    rng = np.random.default_rng(7)
    # 1x1, empty operands, a fully dense row of A against dense B, empty rows/columns in between
    one = csr_from_pattern(np.ones((1, 1), bool), np.full((1, 1), -0.75), dtype)
    _assert_matches_dense(one, one)
    empty = csr_from_pattern(np.zeros((5, 7), bool), np.zeros((5, 7)), dtype)
    _assert_matches_dense(empty, random_csr(rng, 7, 3, 0.5, dtype))
    _assert_matches_dense(random_csr(rng, 4, 5, 0.5, dtype), csr_from_pattern(np.zeros((5, 6), bool), np.zeros((5, 6)), dtype))
    pat = rng.random((9, 11)) < 0.2
    pat[3, :] = True
    pat[5, :] = False
    A = csr_from_pattern(pat, rng.uniform(-1, 1, pat.shape), dtype)
    B = csr_from_pattern(np.ones((11, 13), bool), rng.uniform(-1, 1, (11, 13)), dtype)
    _assert_matches_dense(A, B)


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_exact_cancellation_keeps_structural_zero(dtype):
    # row 0 of A hits column 2 of C twice with a*b and (-a)*b: the sum is exactly 0 but the entry
    # must exist; an explicit zero in A also creates entries.
    A = csr_from_pattern(np.array([[1, 1, 0], [0, 0, 1]], bool), np.array([[0.5, -0.5, 0], [0, 0, 0.0]]), dtype)
    B = csr_from_pattern(np.array([[0, 0, 1], [0, 0, 1], [1, 0, 0]], bool),
                         np.array([[0, 0, 0.25], [0, 0, 0.25], [0.3, 0, 0]]), dtype)
    res = oracle.spgemm(A, B)
    assert res.row_ptr.tolist() == [0, 1, 2]
    assert res.col.tolist() == [2, 0]
    assert res.val.tolist() == [0.0, 0.0]
    assert res.abs[0] == 0.25 and res.abs[1] == 0.0


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_identity_and_permutation(dtype):
    rng = np.random.default_rng(11)
    A = random_csr(rng, 40, 40, 0.15, dtype)
    I = identity(40, dtype)
    for res in (oracle.spgemm(A, I), oracle.spgemm(I, A)):
        assert np.array_equal(res.row_ptr, A.row_ptr) and np.array_equal(res.col, A.col)
        assert np.array_equal(res.val, A.val.astype(np.float64))  # one term per sum: bit exact
    perm = rng.permutation(40)
    P = permutation(perm, dtype)
    res = oracle.spgemm(P, A)  # rows permuted
    for i in range(40):
        s, e = A.row_ptr[perm[i]], A.row_ptr[perm[i] + 1]
        rs, re = res.row_ptr[i], res.row_ptr[i + 1]
        assert np.array_equal(res.col[rs:re], A.col[s:e])
        assert np.array_equal(res.val[rs:re], A.val[s:e].astype(np.float64))
    res = oracle.spgemm(A, transpose(P))  # columns permuted: (A P^T)[i, j'] = A[i, j], perm[j'] = j
    inv = np.empty(40, dtype=np.int64)
    inv[perm] = np.arange(40)
    for i in range(40):
        s, e = A.row_ptr[i], A.row_ptr[i + 1]
        cols = inv[A.col[s:e]]
        order = np.argsort(cols)
        rs, re = res.row_ptr[i], res.row_ptr[i + 1]
        assert np.array_equal(res.col[rs:re], cols[order].astype(np.int32))
        assert np.array_equal(res.val[rs:re], A.val[s:e][order].astype(np.float64))


def test_product_count_identity():
    # sum_i IP_i = sum over stored A[i,k] of nnz(B[k,:]) = sum_k colcount_A(k) * nnz(B[k,:]),
    # and nnz(C[i,:]) <= min(IP_i, C.m)
    A, B, _ = gen.config_inputs(4, shrink=8)
    ip = oracle.row_products(A, B)
    b_len = np.diff(B.row_ptr)
    col_count = np.bincount(A.col, minlength=A.n_cols)
    assert ip.sum() == int((col_count * b_len).sum())
    per_nz = b_len[A.col]
    rows = np.repeat(np.arange(A.n_rows), np.diff(A.row_ptr))
    assert np.array_equal(ip, np.bincount(rows, weights=per_nz, minlength=A.n_rows).astype(np.int64))
    counts = oracle.spgemm_row_counts(A, B)
    assert np.all(counts <= np.minimum(ip, B.n_cols))
    assert np.all((counts == 0) == (ip == 0))


def _laplacian_square_expected(N):
    """A^2 for the 5-point stencil from grid geometry alone: (A^2)[p, q] = number of length-2
    stencil walks weighted by the stencil values.  diagonal: 16 + deg(p); distance-1 neighbour:
    4*(-1) + (-1)*4 = -8; straight distance-2: (-1)(-1) = 1; diagonal neighbour: two walks = 2."""
    entries = {}
    for y in range(N):
        for x in range(N):
            p = y * N + x
            deg = (y > 0) + (y < N - 1) + (x > 0) + (x < N - 1)
            row = {p: 16.0 + deg}
            for dy, dx, v in [(-1, 0, -8), (1, 0, -8), (0, -1, -8), (0, 1, -8), (-2, 0, 1), (2, 0, 1),
                              (0, -2, 1), (0, 2, 1), (-1, -1, 2), (-1, 1, 2), (1, -1, 2), (1, 1, 2)]:
                yy, xx = y + dy, x + dx
                if 0 <= yy < N and 0 <= xx < N:
                    row[yy * N + xx] = float(v)
            entries[p] = row
    return entries


@pytest.mark.parametrize("N", [3, 8, 21])
def test_laplacian_square_closed_form(N):
    A = gen.laplacian_2d(N, np.float64)
    assert A.nnz == 5 * N * N - 4 * N
    ip = oracle.row_products(A, A)
    assert ip.sum() == 25 * (N - 2) ** 2 + 64 * (N - 2) + 36
    res = oracle.spgemm(A, A)
    assert res.nnz == 13 * N * N - 20 * N + 4
    exp = _laplacian_square_expected(N)
    for p in range(N * N):
        s, e = res.row_ptr[p], res.row_ptr[p + 1]
        cols = sorted(exp[p])
        assert res.col[s:e].tolist() == cols
        assert res.val[s:e].tolist() == [exp[p][c] for c in cols]  # small integers: bit exact


def test_laplacian_counts_at_benchmark_size():
    # the benchmark's grid (N = 1024): counts from the closed forms, structure only (fast)
    N = 1024
    A = gen.laplacian_2d(N, np.float64)
    assert A.nnz == 5_238_784
    assert oracle.row_products(A, A).sum() == 26_177_544
    counts = oracle.spgemm_row_counts(A, A)
    assert counts.sum() == 13_611_012 and counts.max() == 13 and counts.min() == 6


def test_fixed_degree_random_matrix():
    # every row of A has exactly 8 entries => IP_i = 64 for every row, IP = 8 * nnz(A), and the
    # expected number of distinct columns per row is 4096*(1-(1-8/4096)^8)-ish ~ 63.5
    A, _, _ = gen.config_inputs(0)
    ip = oracle.row_products(A, A)
    assert np.all(ip == 64) and ip.sum() == 8 * A.nnz == 262_144
    counts = oracle.spgemm_row_counts(A, A)
    assert counts.max() <= 64
    assert abs(counts.mean() - 63.5) < 0.3


@pytest.mark.parametrize("cfg,shrink", [(2, 8), (3, 9), (4, 7), (0, 2)])
def test_against_library_routine(cfg, shrink):
    # independent implementation: scipy's CSR product (values), and its product with all-ones
    # values (structure: no cancellation possible, so nothing is pruned)
    A, B, _ = gen.config_inputs(cfg, shrink=shrink)
    res = oracle.spgemm(A, B)
    As, Bs = A.to_scipy().astype(np.float64), B.to_scipy().astype(np.float64)
    ones = lambda M: type(M)((np.ones_like(M.data), M.indices, M.indptr), shape=M.shape)
    S = (ones(As) @ ones(Bs)).tocsr()
    S.sort_indices()
    assert np.array_equal(res.row_ptr, S.indptr.astype(np.int64))
    assert np.array_equal(res.col, S.indices.astype(np.int32))
    V = (As @ Bs).tocsr()
    Ab = (abs(As) @ abs(Bs)).tocsr()
    rows = np.repeat(np.arange(A.n_rows), np.diff(res.row_ptr))
    ev = np.asarray(V[rows, res.col]).ravel()
    ea = np.asarray(Ab[rows, res.col]).ravel()
    assert np.all(np.abs(res.abs - ea) <= 1e-13 * ea)
    assert np.all(np.abs(res.val - ev) <= 1e-13 * ea)


def test_symmetry_and_transpose_identity():
    A = gen.laplacian_2d(12, np.float64)
    res = oracle.spgemm(A, A)
    from gen import CSR
    C = CSR(A.n_rows, A.n_cols, res.row_ptr, res.col, res.val)
    Ct = transpose(C)
    assert np.array_equal(Ct.row_ptr, C.row_ptr) and np.array_equal(Ct.col, C.col) and np.array_equal(Ct.val, C.val)
    # (A*A)^T = A^T * A^T on a small R-MAT graph
    R = gen.rmat(9, 8, seed=3, dtype=np.float32)
    r1 = oracle.spgemm(R, R)
    Rt = transpose(R)
    r2 = oracle.spgemm(Rt, Rt)
    C1t = transpose(CSR(R.n_rows, R.n_cols, r1.row_ptr, r1.col, r1.val))
    assert np.array_equal(C1t.row_ptr, r2.row_ptr) and np.array_equal(C1t.col, r2.col)
    ab = transpose(CSR(R.n_rows, R.n_cols, r1.row_ptr, r1.col, r1.abs)).val
    assert np.all(np.abs(C1t.val - r2.val) <= 1e-14 * ab)


def test_row_range_and_thread_count_do_not_change_the_result():
    A, B, _ = gen.config_inputs(2, shrink=9)
    full = oracle.spgemm(A, B, threads=1)
    multi = oracle.spgemm(A, B, threads=4)
    assert np.array_equal(full.col, multi.col) and np.array_equal(full.val, multi.val)
    r0, r1 = 100, 777
    part = oracle.spgemm(A, B, r0, r1)
    s, e = full.row_ptr[r0], full.row_ptr[r1]
    assert np.array_equal(part.row_ptr, full.row_ptr[r0:r1 + 1] - s)
    assert np.array_equal(part.col, full.col[s:e]) and np.array_equal(part.val, full.val[s:e])
