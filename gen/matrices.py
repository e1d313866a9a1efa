"""Seeded, platform-independent generators for the synthetic SpGEMM workloads.

Every random number comes from one counter-based generator, ``counter_uniform(seed, stream,
index)``: a pure function of its three integer arguments built from 64-bit integer mixing only, so
the same seed gives bit-identical matrices on any machine and in any evaluation order.

All matrices are returned as :class:`CSR` with int64 ``row_ptr``, int32 ``col`` (ascending and
distinct inside every row) and float32/float64 ``val``.  Values are drawn *after* the structure is
fixed, one per stored entry in CSR order, uniform on [-1, 1).

Workload recipes (the paper evaluates A*A on R-MAT graphs made with the Graph500 parameters
a=0.57, b=c=0.19, Section IV-A; the R-MAT generators below stand in for those, and the clipped-Zipf
rectangular pair stands in for its web/social-graph matrices):

* ``erdos_renyi_k``   every row has exactly k distinct uniform columns.
* ``laplacian_2d``    5-point stencil on an N x N grid, point (x, y) -> row y*N + x.
* ``rmat``            ``edge_factor * 2**scale`` draws, ``scale`` quadrant picks per draw (most
                      significant bit first, no noise, no vertex permutation, self loops kept),
                      duplicate edges merged before values are drawn.
* ``zipf_rows``       row lengths min(X, cap) with P(X = k) proportional to k**-s (k >= 1),
                      columns uniform and distinct inside a row.
* ``block_dense_rows`` block rows that couple to a handful of block columns with dense blocks (the shape of the
                      paper's structural and power-network matrices, Table II: few thousand rows per pattern, most
                      rows heavy, nearly every product in a heavy row, a narrow column space).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

_U64 = np.uint64
_GOLDEN = _U64(0x9E3779B97F4A7C15)
_M1 = _U64(0xBF58476D1CE4E5B9)
_M2 = _U64(0x94D049BB133111EB)
_STREAM_MUL = _U64(0xD1B54A32D192ED03)

# stream ids (kept apart so structure and values never share a counter)
_STREAM_VALUES = 1 << 40
_STREAM_LENGTHS = 1 << 41
_STREAM_COLUMNS = 1 << 42


@dataclass
class CSR:
    """Plain CSR container (host side, numpy)."""

    n_rows: int
    n_cols: int
    row_ptr: np.ndarray  # int64, n_rows + 1
    col: np.ndarray  # int32, nnz
    val: np.ndarray  # float32 / float64, nnz

    @property
    def nnz(self) -> int:
        return int(self.row_ptr[-1])

    @property
    def dtype(self):
        return self.val.dtype

    def to_scipy(self):
        import scipy.sparse as sp

        return sp.csr_matrix((self.val, self.col, self.row_ptr), shape=(self.n_rows, self.n_cols))

    def validate(self) -> None:
        rp = self.row_ptr
        assert rp.dtype == np.int64 and self.col.dtype == np.int32
        assert rp.shape == (self.n_rows + 1,) and rp[0] == 0 and rp[-1] == self.col.size == self.val.size
        assert np.all(np.diff(rp) >= 0)
        if self.col.size:
            assert self.col.min() >= 0 and self.col.max() < self.n_cols
            d = np.diff(self.col.astype(np.int64))
            inner = np.ones(self.col.size - 1, dtype=bool)
            starts = rp[1:-1]
            starts = starts[(starts > 0) & (starts < self.col.size)]
            inner[starts - 1] = False  # position p-1 | p straddles a row boundary
            assert np.all(d[inner] > 0), "columns must be strictly ascending inside a row"


def _mix64(x: np.ndarray) -> np.ndarray:
    x = (x ^ (x >> _U64(30))) * _M1
    x = (x ^ (x >> _U64(27))) * _M2
    return x ^ (x >> _U64(31))


def counter_bits(seed: int, stream: int, index) -> np.ndarray:
    """64 pseudo-random bits as a pure function of (seed, stream, index)."""
    with np.errstate(over="ignore"):
        idx = np.asarray(index).astype(np.uint64)
        key = _mix64(np.asarray([seed], dtype=np.uint64) * _GOLDEN + _GOLDEN)
        key = _mix64(key ^ (np.asarray([stream], dtype=np.uint64) * _STREAM_MUL))
        return _mix64(_mix64(idx * _GOLDEN + key) + key)


def counter_uniform(seed: int, stream: int, index) -> np.ndarray:
    """Uniform float64 on [0, 1) with 53 random bits."""
    return (counter_bits(seed, stream, index) >> _U64(11)).astype(np.float64) * (1.0 / (1 << 53))


def _draw_values(seed: int, nnz: int, dtype) -> np.ndarray:
    out = np.empty(nnz, dtype=dtype)
    step = 1 << 22
    for s in range(0, nnz, step):
        e = min(nnz, s + step)
        u = counter_uniform(seed, _STREAM_VALUES, np.arange(s, e, dtype=np.int64))
        out[s:e] = (2.0 * u - 1.0).astype(dtype)
    return out


def _csr_from_sorted_keys(keys: np.ndarray, n_rows: int, n_cols: int, seed: int, dtype) -> CSR:
    """keys = row * n_cols + col, sorted and unique."""
    rows = keys // n_cols
    col = (keys - rows * n_cols).astype(np.int32)
    counts = np.bincount(rows, minlength=n_rows).astype(np.int64)
    row_ptr = np.zeros(n_rows + 1, dtype=np.int64)
    np.cumsum(counts, out=row_ptr[1:])
    return CSR(n_rows, n_cols, row_ptr, col, _draw_values(seed, keys.size, dtype))


def _distinct_uniform_columns(seed: int, stream: int, row_nnz: np.ndarray, n_cols: int) -> np.ndarray:
    """For every row r, ``row_nnz[r]`` distinct uniform columns.  Slot t of row r draws candidate
    number a = 0, 1, ... from counter index (r << 36) + (a << 13) + t until it differs from every
    column kept so far in that row; among equal candidates the lowest slot keeps its value.
    Returns sorted unique keys ``row * n_cols + col``."""
    row_nnz = np.asarray(row_nnz, dtype=np.int64)
    assert row_nnz.max(initial=0) < (1 << 13) and row_nnz.max(initial=0) <= n_cols
    n_rows = row_nnz.size
    rows = np.repeat(np.arange(n_rows, dtype=np.int64), row_nnz)
    starts = np.zeros(n_rows + 1, dtype=np.int64)
    np.cumsum(row_nnz, out=starts[1:])
    slot = np.arange(rows.size, dtype=np.int64) - starts[rows]
    attempt = np.zeros(rows.size, dtype=np.int64)
    cols = np.empty(rows.size, dtype=np.int64)
    todo = np.arange(rows.size, dtype=np.int64)
    while todo.size:
        idx = (rows[todo] << 36) + (attempt[todo] << 13) + slot[todo]
        u = counter_uniform(seed, stream, idx)
        cols[todo] = np.minimum((u * n_cols).astype(np.int64), n_cols - 1)
        key = ((rows * n_cols + cols) << 13) | slot  # unique: sorts by (row, col, slot)
        order = np.argsort(key, kind="stable")
        ks = key[order] >> 13
        dup = np.zeros(rows.size, dtype=bool)
        dup[1:] = ks[1:] == ks[:-1]
        todo = np.sort(order[dup])
        attempt[todo] += 1
        assert attempt.max(initial=0) < (1 << 23)
    return np.sort(rows * n_cols + cols)


def erdos_renyi_k(n: int, k: int, seed: int, dtype=np.float32, n_cols: int | None = None) -> CSR:
    """Every row holds exactly ``k`` distinct uniform-random columns."""
    n_cols = n if n_cols is None else n_cols
    keys = _distinct_uniform_columns(seed, _STREAM_COLUMNS, np.full(n, k, dtype=np.int64), n_cols)
    return _csr_from_sorted_keys(keys, n, n_cols, seed, dtype)


def laplacian_2d(N: int, dtype=np.float64) -> CSR:
    """5-point Laplacian on an N x N grid: diagonal 4, the (up to four) grid neighbours -1."""
    n = N * N
    y, x = np.divmod(np.arange(n, dtype=np.int64), N)
    cand = [
        (y > 0, -N, -1.0),
        (x > 0, -1, -1.0),
        (np.ones(n, dtype=bool), 0, 4.0),
        (x < N - 1, 1, -1.0),
        (y < N - 1, N, -1.0),
    ]
    counts = sum(m.astype(np.int64) for m, _, _ in cand)
    row_ptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(counts, out=row_ptr[1:])
    col = np.empty(row_ptr[-1], dtype=np.int32)
    val = np.empty(row_ptr[-1], dtype=dtype)
    cursor = row_ptr[:-1].copy()
    rows = np.arange(n, dtype=np.int64)
    for mask, off, v in cand:  # candidates are listed in ascending column order
        pos = cursor[mask]
        col[pos] = (rows[mask] + off).astype(np.int32)
        val[pos] = v
        cursor[mask] += 1
    return CSR(n, n, row_ptr, col, val)


def rmat(scale: int, edge_factor: int, seed: int, dtype=np.float32,
         a: float = 0.57, b: float = 0.19, c: float = 0.19, d: float = 0.05) -> CSR:
    """R-MAT graph with 2**scale vertices and ``edge_factor * 2**scale`` edge draws; duplicate
    edges are merged (one stored entry), self loops are kept.  Level ``bit`` (0 = most significant)
    of draw ``e`` uses counter (seed, stream=bit, index=e); quadrant a = (row bit 0, col bit 0),
    b = (0, 1), c = (1, 0), d = (1, 1)."""
    assert abs(a + b + c + d - 1.0) < 1e-12
    n = 1 << scale
    m = edge_factor * n
    block = 1 << 22
    parts = []
    for s in range(0, m, block):
        e = np.arange(s, min(m, s + block), dtype=np.int64)
        r = np.zeros(e.size, dtype=np.int64)
        cc = np.zeros(e.size, dtype=np.int64)
        for bit in range(scale):
            u = counter_uniform(seed, bit, e)
            rb = u >= a + b
            cb = ((u >= a) & (u < a + b)) | (u >= a + b + c)
            r = (r << 1) | rb
            cc = (cc << 1) | cb
        parts.append(r * n + cc)
    keys = np.unique(np.concatenate(parts))
    return _csr_from_sorted_keys(keys, n, n, seed, dtype)


def _zipf_lengths(seed: int, n_rows: int, s: float, cap: int) -> np.ndarray:
    """min(X, cap) with P(X = k) = k**-s / zeta(s), k = 1, 2, ...: inverse CDF over a table of
    ``cap`` entries whose last entry absorbs the whole tail."""
    from scipy.special import zeta

    k = np.arange(1, cap + 1, dtype=np.float64)
    cdf = np.cumsum(k ** (-s)) / float(zeta(s))
    cdf[-1] = 1.0
    u = counter_uniform(seed, _STREAM_LENGTHS, np.arange(n_rows, dtype=np.int64))
    return np.minimum(np.searchsorted(cdf, u, side="right") + 1, cap).astype(np.int64)


def zipf_rows(n_rows: int, n_cols: int, s: float, cap: int, seed: int, dtype=np.float32) -> CSR:
    lens = np.minimum(_zipf_lengths(seed, n_rows, s, cap), n_cols)
    keys = _distinct_uniform_columns(seed, _STREAM_COLUMNS, lens, n_cols)
    return _csr_from_sorted_keys(keys, n_rows, n_cols, seed, dtype)


def zipf_rectangular_pair(n_a: int, m_a: int, m_b: int, seed: int, dtype=np.float32,
                          s_a: float = 1.8, cap_a: int = 4096, s_b: float = 2.0, cap_b: int = 2048):
    """A is n_a x m_a with Zipf(s_a) row lengths clipped at cap_a, B is m_a x m_b with Zipf(s_b)
    clipped at cap_b.  B uses seed + 1000003 so the two matrices are independent."""
    A = zipf_rows(n_a, m_a, s_a, cap_a, seed, dtype)
    B = zipf_rows(m_a, m_b, s_b, cap_b, seed + 1000003, dtype)
    return A, B


_STREAM_BLOCKS = 1 << 43


def block_dense_rows(n: int, block: int, blocks_per_row: int, fill: float, dense_frac: float, seed: int,
                     dtype=np.float32) -> CSR:
    """Square matrix of ``n / block`` block rows shaped like the stiffness and power-network matrices whose
    squares are almost all heavy rows (few thousand rows per block structure, rows of a few hundred entries in
    dense blocks, a column space of a few accumulator widths).  A *dense* block row (probability ``dense_frac``)
    couples to itself, its two neighbours and ``blocks_per_row - 3`` uniform-random block columns; inside a coupled
    block every entry is kept with probability ``fill``.  The other block rows keep the diagonal and about two
    more entries of their own diagonal block per row, so their rows stay light.  Duplicate block choices merge."""
    assert n % block == 0 and blocks_per_row >= 3
    nb = n // block
    br = np.arange(nb, dtype=np.int64)
    dense = counter_uniform(seed, _STREAM_BLOCKS, br) < dense_frac
    # chosen block columns, (nb, blocks_per_row): self, neighbours (wrapping), random
    choice = np.empty((nb, blocks_per_row), dtype=np.int64)
    choice[:, 0] = br
    choice[:, 1] = (br + 1) % nb
    choice[:, 2] = (br + nb - 1) % nb
    for j in range(3, blocks_per_row):
        u = counter_uniform(seed, _STREAM_BLOCKS + j, br)
        choice[:, j] = np.minimum((u * nb).astype(np.int64), nb - 1)
    parts = []
    db = br[dense]
    for j in range(blocks_per_row):
        # candidate entries of block (db, choice[db, j]): index = ((block row * blocks_per_row + j) * block + r) * block + c
        r, c = np.meshgrid(np.arange(block, dtype=np.int64), np.arange(block, dtype=np.int64), indexing="ij")
        base = ((db * blocks_per_row + j) * block)[:, None, None]
        idx = (base + r[None]) * block + c[None]
        keep = counter_uniform(seed, _STREAM_COLUMNS, idx.ravel()).reshape(idx.shape) < fill
        rows = (db[:, None, None] * block + r[None])[keep]
        cols = (choice[db, j][:, None, None] * block + c[None])[keep]
        parts.append(rows * n + cols)
    sb = br[~dense]
    if sb.size:
        r, c = np.meshgrid(np.arange(block, dtype=np.int64), np.arange(block, dtype=np.int64), indexing="ij")
        idx = ((sb * blocks_per_row)[:, None, None] * block + r[None]) * block + c[None]
        keep = (counter_uniform(seed, _STREAM_COLUMNS, idx.ravel()).reshape(idx.shape) < 2.0 / block) | (r == c)[None]
        rows = (sb[:, None, None] * block + r[None])[keep]
        cols = (sb[:, None, None] * block + c[None])[keep]
        parts.append(rows * n + cols)
    keys = np.unique(np.concatenate(parts))
    return _csr_from_sorted_keys(keys, n, n, seed, dtype)


CONFIG_NAMES = [
    "er4096_k8_f32",
    "laplacian1024_f64",
    "rmat20_ef16_f32",
    "rmat21_ef8_f64",
    "zipf_rect_f32",
    "block_dense_f32",
]


def config_inputs(index: int, shrink: int = 0):
    """The five benchmark products, and (index 5) a product of the second workload class.  ``shrink`` > 0 scales the problem down by 2**shrink (rows and
    columns; grid side for the Laplacian) with the same recipe, for tests the oracle finishes in
    seconds.  Returns (A, B, description)."""
    if index == 0:
        n = 4096 >> shrink
        A = erdos_renyi_k(n, 8, seed=1, dtype=np.float32)
        return A, A, f"C=A*A, ER {n}x{n}, exactly 8 nnz/row, fp32, seed 1"
    if index == 1:
        N = 1024 >> shrink
        A = laplacian_2d(N, np.float64)
        return A, A, f"C=A*A, 5-point Laplacian on a {N}x{N} grid, fp64"
    if index == 2:
        sc = 20 - shrink
        A = rmat(sc, 16, seed=3, dtype=np.float32)
        return A, A, f"C=A*A, R-MAT scale {sc}, edge factor 16, (0.57,0.19,0.19,0.05), merged, fp32, seed 3"
    if index == 3:
        sc = 21 - shrink
        A = rmat(sc, 8, seed=4, dtype=np.float64)
        return A, A, f"C=A*A, R-MAT scale {sc}, edge factor 8, (0.57,0.19,0.19,0.05), merged, fp64, seed 4"
    if index == 4:
        A, B = zipf_rectangular_pair((1 << 20) >> shrink, (1 << 22) >> shrink, (1 << 24) >> shrink,
                                     seed=5, dtype=np.float32)
        return A, B, (f"C=A*B, A {A.n_rows}x{A.n_cols} Zipf(1.8) rows capped 4096, "
                      f"B {B.n_rows}x{B.n_cols} Zipf(2.0) rows capped 2048, fp32, seed 5")
    if index == 5:
        # second workload class: dense-ish heavy rows, almost every product in a heavy row, a column space of two
        # accumulator widths (one multisplit level, the chunk accumulation dominates)
        n = 65536 >> shrink
        A = block_dense_rows(n, 64, 6, 0.7, 0.7, seed=6, dtype=np.float32)
        return A, A, (f"C=A*A, {n}x{n} in 64x64 blocks, 70% dense block rows coupling to 6 block columns at fill 0.7, "
                      f"fp32, seed 6")
    raise ValueError(f"config index {index} out of range 0..5")
