"""GPU parity tests: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Structure (row_ptr, col_idx) bit-exact; values within tau * sum|a*b| with
tau = 1e-5 (fp32) / 1e-12 (fp64)."""
import numpy as np
import pytest
import torch

import gen
import oracle
from helpers import csr_from_pattern, random_csr
from parity import check_product, run_gpu, compare_rows

pytestmark = pytest.mark.gpu


def test_row_analysis_matches_definition():
    import paper_2607_22866_b200 as gm
    A, B, _ = gen.config_inputs(4, shrink=6)
    dA, dB = gm.DeviceCSR.from_host(A), gm.DeviceCSR.from_host(B)
    plan = gm.spgemm_plan(dA, dB)
    ip = plan.row_products().cpu().numpy()
    ref = oracle.row_products(A, B)
    assert np.array_equal(ip, ref)
    info = plan.info()
    assert info.products_total == ref.sum() and info.products_max_row == ref.max()
    assert info.rows_empty == int((ref == 0).sum())
    assert info.c_nnz_upper == int(np.minimum(ref, B.n_cols).sum())
    plan.destroy()


def test_config0_er_all_light():
    A, B, _ = gen.config_inputs(0)
    C, info, stats = check_product(A, B)
    assert info.rows_heavy == 0 and info.rows_light == 4096 and info.products_total == 262144


@pytest.mark.parametrize("shrink", [4, 0])
def test_config1_laplacian_bit_exact(shrink):
    A, B, _ = gen.config_inputs(1, shrink=shrink)
    C, info, stats = check_product(A, B)
    N = 1024 >> shrink
    assert C.nnz == 13 * N * N - 20 * N + 4
    # small integers: fp64 sums are exact whatever the order
    ref = oracle.spgemm(A, B)
    assert np.array_equal(C.val.cpu().numpy(), ref.val)


@pytest.mark.parametrize("cfg,shrink", [(2, 8), (2, 6), (3, 8), (4, 6)])
def test_scaled_down_configs_default_plan(cfg, shrink):
    A, B, _ = gen.config_inputs(cfg, shrink=shrink)
    check_product(A, B)


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
@pytest.mark.parametrize("levels", [0, 1, 2, 3])
def test_forced_levels_give_identical_structure(dtype, levels):
    A = gen.rmat(12, 16, seed=3, dtype=dtype)
    width = {0: 4096, 1: 1024, 2: 256, 3: 64}[levels]
    fan = {0: 0, 1: 4, 2: 4, 3: 4}[levels]
    C, info, stats = check_product(A, A, tau=256, chunk_width=width, max_fanout=fan)
    assert info.params.n_levels == levels
    assert info.rows_heavy > 100 and stats.final_chunks == info.rows_heavy * info.params.chunks_required


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_many_batches_append_in_row_order(dtype):
    A = gen.rmat(12, 16, seed=5, dtype=dtype)
    ip = oracle.row_products(A, A)
    # staging barely larger than the biggest row: dozens of batches, some holding a single row
    C, info, stats = check_product(A, A, tau=128, chunk_width=512, max_fanout=8, stage_elems=int(ip.max()) + 1000)
    assert info.n_batches > 8
    assert stats.c_capacity >= C.nnz


def test_capacity_error_is_reported_not_faulted():
    import paper_2607_22866_b200 as gm
    A = gen.rmat(11, 16, seed=6, dtype=np.float32)
    ip = oracle.row_products(A, A)
    with pytest.raises(gm.GmError) as ei:
        run_gpu(A, A, tau=128, chunk_width=512, stage_elems=int(ip.max()) + 100, c_capacity=1000)
    assert ei.value.status == -6
    with pytest.raises(gm.GmError) as ei:
        run_gpu(A, A, tau=128, stage_elems=int(ip.max()) - 1)   # a row is never split across batches
    assert ei.value.status == -6
    # the context is still usable
    check_product(A, A, tau=128, chunk_width=512)


@pytest.mark.parametrize("smem", [49152, 101376, 232448])
def test_smem_budget_sweep(smem):
    A = gen.rmat(13, 16, seed=7, dtype=np.float32)
    C, info, stats = check_product(A, A, smem_bytes=smem)
    assert info.params.tau <= 8192


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_light_heavy_boundary_and_degenerate_rows(dtype):
    rng = np.random.default_rng(3)
    n, m = 300, 1000
    # B: row 0 has a single entry (column 999), row 1 is dense, row 2 is empty, the rest random
    patB = rng.random((n, m)) < 0.05
    patB[0, :] = False; patB[0, 999] = True
    patB[1, :] = True
    patB[2, :] = False
    B = csr_from_pattern(patB, rng.uniform(-1, 1, patB.shape), dtype)
    patA = rng.random((64, n)) < 0.03
    patA[5, :] = False; patA[5, 0] = True                  # one product
    patA[6, :] = False; patA[6, [0, 2]] = True             # references an empty row of B
    patA[7, :] = False                                      # empty row between heavy rows
    patA[8, :] = True                                       # very heavy row (hits the dense row)
    patA[9, :] = False; patA[9, 1] = True                  # exactly m products, all distinct columns
    A = csr_from_pattern(patA, rng.uniform(-1, 1, patA.shape), dtype)
    ip = oracle.row_products(A, B)
    for tau in (int(ip[9]), int(ip[9]) - 1, 1, 40):        # IP_i == tau is light, tau + 1 is heavy
        C, info, stats = check_product(A, B, tau=tau, chunk_width=128, max_fanout=2)
        assert info.rows_heavy == int((ip > tau).sum())


def test_heavy_row_whose_products_hit_one_column_or_one_chunk():
    dtype = np.float32
    n = 600
    # every row of B is the same single entry in column 77 => a heavy row of A gives ONE entry of C
    patB = np.zeros((n, 4096), bool); patB[:, 77] = True
    rng = np.random.default_rng(5)
    B = csr_from_pattern(patB, rng.uniform(-1, 1, patB.shape), dtype)
    patA = np.zeros((4, n), bool); patA[1, :] = True; patA[3, :500] = True
    A = csr_from_pattern(patA, rng.uniform(-1, 1, patA.shape), dtype)
    C, info, stats = check_product(A, B, tau=64, chunk_width=256, max_fanout=4)
    assert info.rows_heavy == 2 and C.nnz == 2
    # exactly one product per chunk: B rows are single entries at columns c*W
    patB2 = np.zeros((16, 4096), bool)
    for k in range(16):
        patB2[k, k * 256] = True
    B2 = csr_from_pattern(patB2, np.ones(patB2.shape), dtype)
    A2 = csr_from_pattern(np.ones((2, 16), bool), rng.uniform(-1, 1, (2, 16)), dtype)
    check_product(A2, B2, tau=8, chunk_width=256, max_fanout=4)


@pytest.mark.parametrize("c_cols", [1, 31, 255, 256, 257, 100003])
def test_column_counts_that_are_not_chunk_multiples(c_cols):
    rng = np.random.default_rng(c_cols)
    k = 200
    dens = min(0.5, 60.0 / c_cols) if c_cols > 1 else 1.0
    B = random_csr(rng, k, c_cols, dens, np.float64)
    A = random_csr(rng, 50, k, 0.3, np.float64)
    check_product(A, B, tau=16, chunk_width=256 if c_cols > 256 else 32, max_fanout=4)


def test_empty_operands():
    for shape_a, shape_b in [((0, 5), (5, 7)), ((4, 0), (0, 7)), ((4, 5), (5, 0)), ((3, 3), (3, 3))]:
        A = csr_from_pattern(np.zeros(shape_a, bool), np.zeros(shape_a), np.float32)
        B = csr_from_pattern(np.zeros(shape_b, bool), np.zeros(shape_b), np.float32)
        C, info, stats = run_gpu(A, B)
        assert C.nnz == 0 and C.row_ptr.numel() == shape_a[0] + 1 and int(C.row_ptr.abs().sum()) == 0


def test_argument_errors():
    import paper_2607_22866_b200 as gm
    A = gen.erdos_renyi_k(64, 4, seed=1, dtype=np.float32)
    B = gen.erdos_renyi_k(32, 4, seed=1, dtype=np.float32)
    with pytest.raises(gm.GmError) as ei:
        run_gpu(A, B)
    assert ei.value.status == -2
    A64 = gen.erdos_renyi_k(64, 4, seed=1, dtype=np.float64)
    with pytest.raises(gm.GmError) as ei:
        gm.spgemm(gm.DeviceCSR.from_host(A), gm.DeviceCSR.from_host(A64))
    assert ei.value.status == -3
    with pytest.raises(gm.GmError) as ei:
        run_gpu(A, A, smem_bytes=1 << 19)
    assert ei.value.status == -9
    bad = gen.erdos_renyi_k(64, 4, seed=1, dtype=np.float32)
    bad.col[1] = bad.col[0]        # duplicate column in row 0
    with pytest.raises(gm.GmError) as ei:
        run_gpu(bad, A, validate_inputs=1)
    assert ei.value.status == -4


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_single_stream_and_debug_validation(dtype):
    # light rows next to the heavy path on the plan's second stream (default) or everything on the caller's stream;
    # debug mode checks the inputs and every product's chunk on the device and finds nothing to complain about
    A = gen.rmat(13, 16, seed=4, dtype=dtype)
    kw = dict(tau=256, chunk_width=1024, max_fanout=4, stage_elems=1 << 21)
    C1, info, _ = check_product(A, A, **kw)
    assert info.rows_light > 0 and info.rows_heavy > 0 and info.n_batches > 1 and info.params.n_levels == 2
    C2, _, _ = check_product(A, A, single_stream=1, validate_inputs=1, **kw)
    assert torch.equal(C1.row_ptr, C2.row_ptr) and torch.equal(C1.col, C2.col)
    A1, B1, _ = gen.config_inputs(4, shrink=6)      # one batch: gather and the light rows' numeric pass side by side
    check_product(A1, B1, validate_inputs=1)
    check_product(A1, B1, single_stream=1)


def test_two_runs_same_structure_values_close():
    A = gen.rmat(12, 16, seed=9, dtype=np.float32)
    C1, _, _ = run_gpu(A, A, tau=256, chunk_width=1024, max_fanout=4)
    C2, _, _ = run_gpu(A, A, tau=256, chunk_width=1024, max_fanout=4)
    assert torch.equal(C1.row_ptr, C2.row_ptr) and torch.equal(C1.col, C2.col)
    ref = oracle.spgemm(A, A)
    d = (C1.val.double() - C2.val.double()).abs().cpu().numpy()
    assert np.all(d <= 2e-5 * ref.abs)


def test_plan_reuse_with_new_values():
    import paper_2607_22866_b200 as gm
    A = gen.rmat(11, 16, seed=2, dtype=np.float64)
    dA = gm.DeviceCSR.from_host(A)
    plan = gm.spgemm_plan(dA, dA, opts=None)
    C1 = gm.spgemm_execute(plan)
    compare_rows(C1, oracle.spgemm(A, A), np.float64)
    dA.val.mul_(-0.5)
    A.val[:] = A.val * -0.5
    C2 = gm.spgemm_execute(plan)
    compare_rows(C2, oracle.spgemm(A, A), np.float64)
    plan.destroy()


def test_host_entry_point():
    import paper_2607_22866_b200 as gm
    A, B, _ = gen.config_inputs(4, shrink=7)
    ref = oracle.spgemm(A, B)
    rp = np.empty(A.n_rows + 1, np.int64)
    col = np.empty(ref.nnz + 10, np.int32)
    val = np.empty(ref.nnz + 10, np.float32)
    nnz = gm.spgemm_host(A, B, rp, col, val)
    assert nnz == ref.nnz and np.array_equal(rp, ref.row_ptr) and np.array_equal(col[:nnz], ref.col)
    assert np.all(np.abs(val[:nnz].astype(np.float64) - ref.val) <= 1e-5 * ref.abs)
    with pytest.raises(gm.GmError) as ei:
        gm.spgemm_host(A, B, rp, col[:5], val[:5])
    assert ei.value.status == -6


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_host_entry_point_streams_batches_to_the_host(dtype):
    # several batches: every batch's rows (light ones included) are finished and copied out while the next
    # batch computes; pinned and pageable destinations, and a destination that is too small
    import paper_2607_22866_b200 as gm
    A = gen.rmat(12, 16, seed=9, dtype=dtype)
    ref = oracle.spgemm(A, A)
    o = gm.PlanOpts(); o.tau = 128; o.stage_elems = 1 << 17
    tol = 1e-5 if dtype == np.float32 else 1e-12
    for pinned in (False, True):
        rp = np.empty(A.n_rows + 1, np.int64)
        if pinned:
            tcol = torch.empty(ref.nnz + 7, dtype=torch.int32, pin_memory=True)
            tval = torch.empty(ref.nnz + 7, dtype=torch.float32 if dtype == np.float32 else torch.float64, pin_memory=True)
            col, val = tcol.numpy(), tval.numpy()
        else:
            col = np.empty(ref.nnz + 7, np.int32)
            val = np.empty(ref.nnz + 7, dtype)
        col[:] = -1
        nnz = gm.spgemm_host(A, A, rp, col, val, opts=o)
        assert nnz == ref.nnz and np.array_equal(rp, ref.row_ptr) and np.array_equal(col[:nnz], ref.col)
        assert np.all(np.abs(val[:nnz].astype(np.float64) - ref.val) <= tol * ref.abs)
        assert np.all(col[nnz:] == -1)
    dA = gm.DeviceCSR.from_host(A)
    plan = gm.spgemm_plan(dA, dA, 232448, o)
    assert plan.info().n_batches > 3
    plan.destroy()
    with pytest.raises(gm.GmError) as ei:
        gm.spgemm_host(A, A, rp, col[:ref.nnz // 2], val[:ref.nnz // 2], opts=o)
    assert ei.value.status == -6


def test_host_entry_point_with_chunks_that_left_the_hierarchy_early():
    # three levels with early exit, several batches, result streamed to the host: the gather reads the chunks that
    # stayed behind from the other staging buffer
    import paper_2607_22866_b200 as gm
    A = gen.rmat(12, 16, seed=21, dtype=np.float32)
    ref = oracle.spgemm(A, A)
    o = gm.PlanOpts()
    o.tau, o.chunk_width, o.max_fanout, o.stage_elems, o.validate_inputs = 128, 128, 4, 1 << 18, 1
    rp = np.empty(A.n_rows + 1, np.int64)
    col = np.empty(ref.nnz, np.int32)
    val = np.empty(ref.nnz, np.float32)
    nnz = gm.spgemm_host(A, A, rp, col, val, opts=o)
    assert nnz == ref.nnz and np.array_equal(rp, ref.row_ptr) and np.array_equal(col, ref.col)
    assert np.all(np.abs(val.astype(np.float64) - ref.val) <= 1e-5 * ref.abs)
    dA = gm.DeviceCSR.from_host(A)
    C, info, stats = gm.spgemm(dA, dA, 232448, o)
    assert info.params.n_levels == 3 and info.n_batches > 1 and stats.early_exit_products > 0


def _check_sampled_rows(A, B, n_random=200, n_heavy=60, whole_row_ptr=False, **opts):
    """Full-size check in the launch configuration the benchmark times: structure and values of
    sampled rows (random rows, the heaviest rows, random heavy rows) against the row-range oracle,
    plus whole-matrix invariants that need no reference."""
    import gc
    from parity import TOL
    # the results of these products take most of the device: hand cached blocks of earlier tests back first
    gc.collect()
    torch.cuda.empty_cache()
    C, info, stats = run_gpu(A, B, **opts)
    ip = oracle.row_products(A, B)
    assert info.products_total == int(ip.sum()) and info.rows_heavy == int((ip > info.params.tau).sum())
    rp = C.row_ptr.cpu().numpy()
    assert rp[0] == 0 and rp[-1] == C.nnz == stats.c_nnz and np.all(np.diff(rp) >= 0)
    assert np.all(np.diff(rp) <= np.minimum(ip, B.n_cols)) and np.all((np.diff(rp) == 0) == (ip == 0))
    if whole_row_ptr:
        # every row's entry count against the oracle's count-only (symbolic) pass over the whole matrix
        assert np.array_equal(np.diff(rp), oracle.spgemm_row_counts(A, B))
    rng = np.random.default_rng(0)
    rows = set(rng.integers(0, A.n_rows, n_random).tolist()) | set(np.argsort(-ip)[:3].tolist())
    heavy = np.nonzero(ip > info.params.tau)[0]
    if heavy.size:
        rows |= set(rng.choice(heavy, min(n_heavy, heavy.size), replace=False).tolist())
    for r in sorted(rows):
        ref = oracle.spgemm(A, B, r, r + 1, threads=1)
        s, e = rp[r], rp[r + 1]
        assert e - s == ref.nnz, r
        assert np.array_equal(C.col[s:e].cpu().numpy(), ref.col), r
        val = C.val[s:e].cpu().numpy().astype(np.float64)
        assert np.all(np.abs(val - ref.val) <= TOL[np.dtype(A.val.dtype)] * ref.abs), r
    return info, stats


def test_config2_rmat20_full_size_sampled_rows():
    # the benchmark's default workload: 2.1e10 products, 9.7e9 entries of C, about ten batches of up to 2^31 products;
    # sampled rows in full, and the entry count of every row
    A, B, _ = gen.config_inputs(2)
    info, stats = _check_sampled_rows(A, B, whole_row_ptr=True)
    assert info.n_batches >= 8 and info.params.levels() == [32] and stats.c_capacity >= stats.c_nnz
    assert info.level0_direct == 1


def test_config3_rmat21_fp64_full_size_default_plan():
    # R-MAT scale 21, edge factor 8, fp64, exactly as the benchmark runs it (no plan options): one level of 128
    # children written by the expansion kernel, several batches, a result of more than 100 GB
    A, B, _ = gen.config_inputs(3)
    info, stats = _check_sampled_rows(A, B, n_random=150, n_heavy=50)
    assert info.params.levels() == [128] and info.level0_direct == 1 and info.n_batches > 1


def test_config4_zipf_pair_full_size_default_plan():
    # the rectangular clipped-Zipf pair (2^24 columns) exactly as the benchmark runs it: two levels, the first as
    # separate passes (short segments) with its histogram counted by the expansion kernel, 256 children
    A, B, _ = gen.config_inputs(4)
    info, stats = _check_sampled_rows(A, B, n_random=150, n_heavy=60, whole_row_ptr=True)
    assert info.params.levels() == [256, 2] and info.level0_direct == 0 and info.rows_heavy > 0
    # after the first split nearly every chunk of these rows is light: the second level moves a fraction of the products
    assert stats.early_exit_products > 0 and stats.split_products < 2 * stats.staged_products


def test_second_workload_class_dense_heavy_rows():
    # block-structured product (the shape of the paper's structural matrices): 70 % of the rows heavy, 99.99 % of the
    # products in them, two chunks per row, rows of C of a thousand entries from tens of thousands of products.
    # Whole matrix against the oracle at 1/16 size, sampled rows and every row's entry count at full size.
    A, B, _ = gen.config_inputs(5, shrink=4)
    C, info, stats = check_product(A, B)
    assert info.rows_heavy > 0.5 * A.n_rows
    A, B, _ = gen.config_inputs(5)
    info, stats = _check_sampled_rows(A, B, n_random=100, n_heavy=60, whole_row_ptr=True)
    assert info.params.levels() == [2] and info.products_heavy > 0.98 * info.products_total
    assert stats.c_nnz * 20 < info.products_total   # dense accumulation: dozens of products per entry


def test_config3_rmat_fp64_two_levels_sampled_rows():
    # fp64 R-MAT (scale 18 here, scale 21 in the config) with the fan-out capped so that the split takes two levels
    A, B, _ = gen.config_inputs(3, shrink=3)
    info, stats = _check_sampled_rows(A, B, max_fanout=8, stage_elems=1 << 26)
    assert info.params.n_levels == 2 and info.n_batches > 1


def test_config4_zipf_wide_columns_three_levels_sampled_rows():
    # rectangular clipped-Zipf product, 2^22 columns here (2^24 in the config), three multisplit levels
    A, B, _ = gen.config_inputs(4, shrink=2)
    info, stats = _check_sampled_rows(A, B, n_random=60, n_heavy=40, max_fanout=8, chunk_width=8192)
    assert info.params.n_levels == 3 and info.rows_heavy > 0
    assert stats.early_exit_products > 0  # most chunks of these rows are light after the first split


@pytest.mark.parametrize("separate", [0, 1])
@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_first_level_of_256_children_as_separate_passes(dtype, separate):
    # fan-out 256 with the first level run as histogram + multisplit passes over the staging buffer (the shape of the
    # Zipf pair's default plan): rows of B are short, so the planner does not let the expansion place the products
    A, B, _ = gen.config_inputs(4, shrink=5)
    C, info, stats = check_product(A, B, tau=256, chunk_width=1024, separate_histogram=separate, stage_elems=1 << 18)
    assert info.params.levels()[0] == 256 and info.params.n_levels == 2 and info.level0_direct == 0
    assert info.n_batches > 1 and info.rows_heavy > 100


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
@pytest.mark.parametrize("level0", [1, 2])
@pytest.mark.parametrize("separate", [0, 1])
def test_light_chunks_leave_the_hierarchy_early(dtype, level0, separate):
    # Algorithm 3's early exit: from the second level on a chunk with few products is not split further.  Four levels
    # (fan-out 4, 4, 4, 2), several batches; the same product with every chunk carried through every level must
    # give the same C, and the multisplit passes must have moved fewer products.
    A = gen.rmat(13, 16, seed=5, dtype=dtype)
    common = dict(tau=256, chunk_width=64, max_fanout=4, level0_multisplit=level0, separate_histogram=separate,
                  stage_elems=1 << 20)
    C0, info0, st0 = check_product(A, A, early_exit=-1, **common)
    C1, info1, st1 = check_product(A, A, **common)
    C2, info2, st2 = check_product(A, A, early_exit=24, **common)
    assert info1.params.n_levels == 4 and info1.n_batches > 1 and info1.level0_direct == level0 - 1
    passes = info1.params.n_levels - info1.level0_direct
    assert st0.early_exit_products == 0 and st0.early_exit_chunks == 0
    assert st0.split_products == passes * st0.staged_products
    assert 0 < st2.early_exit_products < st1.early_exit_products <= st1.staged_products
    assert st1.split_products < st2.split_products < st0.split_products
    # a chunk leaves at most once, and one that left at level l is moved by l - 1 passes fewer than the rest
    assert st1.split_products >= passes * st1.staged_products - (info1.params.n_levels - 1) * st1.early_exit_products
    for C in (C1, C2):
        assert torch.equal(C.row_ptr, C0.row_ptr) and torch.equal(C.col, C0.col)  # (values: each against the oracle above)


@pytest.mark.parametrize("separate", [0, 1])
def test_fused_and_stand_alone_histogram_agree(separate):
    # first level as separate passes over the staging buffer (Algorithm 5 as printed); its counts come either
    # from the expansion kernel or from the histogram kernel
    A = gen.rmat(13, 16, seed=11, dtype=np.float32)
    C, info, stats = check_product(A, A, tau=512, chunk_width=512, max_fanout=4, separate_histogram=separate,
                                   level0_multisplit=1, stage_elems=1 << 20)
    assert info.params.n_levels == 2 and info.n_batches > 1 and info.level0_direct == 0


@pytest.mark.parametrize("dtype,fanout,width", [(np.float32, 4, 512), (np.float64, 32, 256), (np.float32, 256, 32)])
def test_expansion_straight_into_the_first_level(dtype, fanout, width):
    # default path: the expansion kernel places every product in its level-0 child from counts alone.
    # Several batches, one to three levels, and (narrow chunks with fan-out 256) tiles with more
    # (segment, child) pairs than the per-tile table of run starts holds.
    A = gen.rmat(13, 16, seed=11, dtype=dtype)
    C, info, stats = check_product(A, A, tau=256, chunk_width=width, max_fanout=fanout, stage_elems=1 << 20,
                                   level0_multisplit=2)
    assert info.level0_direct == 1 and info.n_batches > 1 and info.params.n_levels >= 1


@pytest.mark.parametrize("dtype,fanout,width", [(np.float32, 32, 512), (np.float64, 128, 128), (np.float32, 2, 8192)])
def test_bulk_copy_expansion_and_plain_loads_agree(dtype, fanout, width):
    # expand_staging = 1: rows of B reach the expansion through bulk asynchronous copies into shared memory (pieces
    # that start and end at every alignment, warps whose range holds one segment or hundreds, short segments by the
    # kernel of their own, the last elements of B's arrays); default: the tile-per-block kernel with plain loads.
    # Both against the oracle.
    A = gen.rmat(14, 16, seed=13, dtype=dtype)
    kw = dict(tau=512, chunk_width=width, max_fanout=fanout, stage_elems=1 << 22, level0_multisplit=2)
    C1, info, _ = check_product(A, A, expand_staging=1, **kw)
    assert info.level0_direct == 1 and info.n_batches > 1 and info.params.levels()[0] == fanout
    C2, info2, _ = check_product(A, A, **kw)
    assert torch.equal(C1.row_ptr, C2.row_ptr) and torch.equal(C1.col, C2.col)


def test_bounded_wait_on_bulk_copies_runs_out_cleanly():
    # the copies are announced to the barrier but withheld (nothing completes it), so every wait gives up after 200
    # polls: the call returns GM_ERR_TIMEOUT, nothing faults or hangs, and the same context then computes the product
    import paper_2607_22866_b200 as gm
    A = gen.rmat(13, 16, seed=13, dtype=np.float32)
    kw = dict(tau=512, chunk_width=1024, max_fanout=8, level0_multisplit=2)
    with pytest.raises(gm.GmError) as ei:
        run_gpu(A, A, expand_staging=1, debug_spin_limit=-200, **kw)
    assert ei.value.status == -8
    check_product(A, A, expand_staging=1, **kw)


@pytest.mark.parametrize("dtype,width,fanout", [(np.float32, 8192, 0), (np.float64, 512, 16), (np.float32, 128, 8)])
def test_outer_product_order_expansion(dtype, width, fanout):
    # expand_order = 1: the batch's segments sorted by row of B (masked CSR -> CSC), products generated column of A by
    # column of A as in Eq. 2 / Algorithm 4; zero, one and two multisplit levels, several batches
    A = gen.rmat(13, 16, seed=17, dtype=dtype)
    kw = dict(tau=256, chunk_width=width, stage_elems=1 << 20)
    if fanout:
        kw["max_fanout"] = fanout
    C1, info, _ = check_product(A, A, expand_order=1, **kw)
    assert info.level0_direct == 0 and info.n_batches > 1
    C2, _, _ = run_gpu(A, A, **kw)
    assert torch.equal(C1.row_ptr, C2.row_ptr) and torch.equal(C1.col, C2.col)
    # rows of B of 0 to 3 entries: tiles with more segments than the shared window holds, empty segments
    rng = np.random.default_rng(29)
    Bs = random_csr(rng, 3000, 5000, 0.0004, dtype)
    As = random_csr(rng, 40, 3000, 0.6, dtype)
    check_product(As, Bs, tau=64, chunk_width=256, max_fanout=4, expand_order=1)


def test_expansion_straight_into_the_first_level_short_rows_of_b():
    # rows of B with 0 to 3 entries: tiles with thousands of segments, empty segments, heavy rows made of them
    rng = np.random.default_rng(23)
    B = random_csr(rng, 3000, 5000, 0.0004, np.float32)
    A = random_csr(rng, 40, 3000, 0.6, np.float32)
    C, info, stats = check_product(A, B, tau=64, chunk_width=256, max_fanout=4, level0_multisplit=2)
    assert info.level0_direct == 1 and info.rows_heavy == 40
    C, info, stats = check_product(A, B, tau=64, chunk_width=256, max_fanout=4)  # short segments: separate passes
    assert info.level0_direct == 0


@pytest.mark.parametrize("ctas", [1, 2, 4, 8])
def test_accumulators_per_sm_with_many_tiny_chunks(ctas):
    # narrow blocks (fewer warps than the 32-chunk look-ahead of the small-chunk path) and chunks of a few
    # products each: every chunk must still be visited exactly once
    A, B, _ = gen.config_inputs(4, shrink=4)
    C, info, stats = check_product(A, B, acc_ctas_per_sm=ctas, tau=256)
    assert info.rows_heavy > 100 and info.params.acc_ctas_per_sm == ctas


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_chunk_sizes_around_the_warp_sort_widths(dtype):
    # Chunks of 1 ... 600 products, with repeated columns, on both sides of every width of the one-warp sort
    # (32, 64, 128, 256, 512 products) and of the hand-over to the block-wide accumulator.  Row r of B holds
    # 2^r entries in chunk 1 (columns 1024..2047, drawn from 300 columns so that rows overlap) and one entry
    # in chunk 0; a row of A picks the rows of B that spell its target size in binary.
    rng = np.random.default_rng(17)
    pool = 1024 + rng.choice(1024, 300, replace=False)
    patB = np.zeros((10, 4096), bool)
    for r in range(10):
        patB[r, rng.choice(pool, min(1 << r, 300), replace=False)] = True
        patB[r, r] = True
    sizes_of_b = patB[:, 1024:2048].sum(axis=1)
    B = csr_from_pattern(patB, rng.uniform(-1, 1, patB.shape), dtype)
    targets = [1, 2, 31, 32, 33, 63, 64, 65, 127, 128, 129, 255, 256, 257, 300, 511]
    patA = np.zeros((len(targets) + 3, 10), bool)
    for i, n in enumerate(targets):
        patA[i] = [(n >> r) & 1 for r in range(10)]
    patA[len(targets)] = True                     # all rows: the largest chunk
    patA[len(targets) + 1, [8, 9]] = True
    patA[len(targets) + 2, [9]] = True
    A = csr_from_pattern(patA, rng.uniform(-1, 1, patA.shape), dtype)
    chunk1 = patA.astype(np.int64) @ sizes_of_b
    assert chunk1.min() == 1 and (chunk1 > 512).any() and {32, 33, 256, 257}.issubset(set(chunk1.tolist()))
    C, info, stats = check_product(A, B, tau=1, chunk_width=1024, max_fanout=4)
    assert info.rows_heavy == int((chunk1 + patA.sum(axis=1) > 1).sum())


@pytest.mark.parametrize("seed", list(range(48)))
def test_random_plans_against_the_oracle(seed):
    # seeded draws of matrix shape and of every plan option that changes how the work is split: whatever the split,
    # C must be the oracle's (debug validation on: inputs checked, every product checked against its chunk)
    rng = np.random.default_rng(1000 + seed)
    dtype = [np.float32, np.float64][seed % 2]
    kind = seed % 3
    if kind == 0:
        A = gen.rmat(int(rng.integers(9, 13)), int(rng.integers(4, 20)), seed=100 + seed, dtype=dtype)
        B = A
    elif kind == 1:
        m = int(rng.integers(300, 2000))
        A = random_csr(rng, int(rng.integers(20, 400)), m, float(rng.uniform(0.01, 0.3)), dtype)
        B = random_csr(rng, m, int(rng.integers(100, 5000)), float(rng.uniform(0.002, 0.05)), dtype,
                       zero_fraction=0.05)
    else:
        A = gen.zipf_rows(int(rng.integers(200, 3000)), 4000, 1.6, 600, seed=200 + seed, dtype=dtype)
        B = gen.zipf_rows(4000, int(rng.integers(500, 200000)), 1.8, 300, seed=300 + seed, dtype=dtype)
    opts = dict(
        tau=int(rng.choice([8, 32, 128, 512])),
        chunk_width=int(rng.choice([32, 64, 256, 1024, 4096])),
        max_fanout=int(rng.choice([2, 4, 16, 256])),
        stage_elems=int(rng.choice([0, 1 << 16, 1 << 19])),
        level0_multisplit=int(rng.integers(0, 3)),
        separate_histogram=int(rng.integers(0, 2)),
        early_exit=int(rng.choice([0, -1, 16])),
        small_chunk_max=int(rng.choice([0, 32, 512, -1])),
        mid_chunk_max=int(rng.choice([0, 64, 1024, -1])),
        expand_order=int(rng.choice([0, 0, 1])),
        single_stream=int(rng.integers(0, 2)),
        acc_ctas_per_sm=int(rng.choice([1, 2, 4])),
    )
    ip = oracle.row_products(A, B)
    if opts["stage_elems"]:
        opts["stage_elems"] = max(opts["stage_elems"], int(ip.max()))
    while opts["max_fanout"] ** 8 < -(-B.n_cols // opts["chunk_width"]):  # the split may take at most eight levels
        opts["max_fanout"] *= 4
    check_product(A, B, **opts)
