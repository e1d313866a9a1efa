"""The seeded generators: determinism, CSR validity, and the distributions the recipes promise."""
import numpy as np

import gen


def test_counter_generator_is_a_pure_function():
    idx = np.arange(1000, dtype=np.int64)
    a = gen.counter_uniform(5, 7, idx)
    b = gen.counter_uniform(5, 7, idx[::-1])[::-1]
    assert np.array_equal(a, b)
    assert not np.array_equal(a, gen.counter_uniform(6, 7, idx))
    assert not np.array_equal(a, gen.counter_uniform(5, 8, idx))
    # fixed values guard against silent changes of the mixing constants
    assert gen.matrices.counter_bits(1, 2, np.array([0, 1, 2])).tolist() == \
        [2132609893017788125, 18058456146663585017, 17349919185937834186]
    u = gen.counter_uniform(1, 2, np.arange(200000))
    assert abs(u.mean() - 0.5) < 5e-3 and abs(u.var() - 1 / 12) < 2e-3 and 0 <= u.min() and u.max() < 1


def test_all_configs_are_valid_csr_and_deterministic():
    for cfg, shrink in [(0, 0), (1, 4), (2, 8), (3, 9), (4, 7)]:
        A, B, desc = gen.config_inputs(cfg, shrink)
        A.validate(), B.validate()
        A2, B2, _ = gen.config_inputs(cfg, shrink)
        assert np.array_equal(A.col, A2.col) and np.array_equal(A.val, A2.val)
        assert np.array_equal(B.row_ptr, B2.row_ptr)
        assert A.n_cols == B.n_rows and A.val.dtype == B.val.dtype
        assert A.val.min() >= -1 and A.val.max() <= 4


def test_er_has_exactly_k_distinct_columns_per_row():
    A = gen.erdos_renyi_k(512, 8, seed=1)
    assert np.all(np.diff(A.row_ptr) == 8)
    A.validate()
    # dense corner case: k close to n forces many redraws
    D = gen.erdos_renyi_k(16, 15, seed=2)
    D.validate()
    assert np.all(np.diff(D.row_ptr) == 15)


def test_rmat_shape_and_skew():
    A = gen.rmat(12, 16, seed=3)
    A.validate()
    deg = np.diff(A.row_ptr)
    assert A.nnz <= 16 << 12 and A.nnz > 0.8 * (16 << 12)   # merging removes some duplicates
    # (a+b) = 0.76 of the mass falls in the upper half of the rows at every level: hubs at low ids
    assert deg[: 1 << 11].sum() > 0.7 * A.nnz
    assert deg.max() > 20 * deg.mean()


def test_zipf_lengths_follow_the_clipped_law():
    lens = gen.matrices._zipf_lengths(5, 200000, 1.8, 4096)
    assert lens.min() == 1 and lens.max() == 4096
    from scipy.special import zeta
    p1 = 1.0 / zeta(1.8)
    assert abs((lens == 1).mean() - p1) < 0.01
    assert abs((lens == 2).mean() - p1 * 2 ** -1.8) < 0.01
    tail = 1.0 - np.sum(np.arange(1, 4096, dtype=np.float64) ** -1.8) / zeta(1.8)
    assert abs((lens == 4096).mean() - tail) < 5e-4 and (lens == 4096).sum() > 0


def test_block_dense_rows_is_the_second_workload_class():
    # most rows heavy, nearly every product in a heavy row, column space of a few accumulator widths
    import oracle
    A, B, _ = gen.config_inputs(5, shrink=4)
    A.validate()
    assert B is A and A.n_rows == A.n_cols == 4096
    A2, _, _ = gen.config_inputs(5, shrink=4)
    assert np.array_equal(A.col, A2.col) and np.array_equal(A.val, A2.val)   # same seed, same matrix
    ip = oracle.row_products(A, A)
    heavy = ip > 512
    assert 0.3 <= heavy.mean() <= 0.9 and ip[heavy].sum() >= 0.98 * ip.sum()
    assert np.diff(A.row_ptr).min() >= 1 and np.diff(A.row_ptr).max() <= 6 * 64
