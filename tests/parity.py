"""Shared parity check: CUDA library (through the C ABI binding) against the CPU oracle."""
import numpy as np
import torch

import oracle
import paper_2607_22866_b200 as gm

TOL = {np.dtype(np.float32): 1e-5, np.dtype(np.float64): 1e-12}  # |c - c_ref| <= tol * sum|a*b|


def make_opts(**kw) -> gm.PlanOpts:
    o = gm.PlanOpts()
    for k, v in kw.items():
        setattr(o, k, v)
    return o


def run_gpu(A, B, smem_bytes=232448, **opts):
    dA = gm.DeviceCSR.from_host(A)
    dB = dA if B is A else gm.DeviceCSR.from_host(B)
    C, info, stats = gm.spgemm(dA, dB, smem_bytes, make_opts(**opts) if opts else None)
    torch.cuda.synchronize()
    return C, info, stats


def compare_rows(C, ref, dtype, r0=0):
    """C: DeviceCSR (whole matrix); ref: oracle rows [r0, r1).  Structure bit-exact, values within
    the tolerance scaled by the sum of absolute products."""
    r1 = ref.r1
    rp = C.row_ptr[r0:r1 + 1].cpu().numpy()
    assert np.array_equal(rp - rp[0], ref.row_ptr), "row_ptr differs from the oracle"
    s, e = int(rp[0]), int(rp[-1])
    col = C.col[s:e].cpu().numpy()
    val = C.val[s:e].cpu().numpy().astype(np.float64)
    assert np.array_equal(col, ref.col), "column indices differ from the oracle"
    tol = TOL[np.dtype(dtype)]
    err = np.abs(val - ref.val)
    bad = err > tol * ref.abs
    assert not bad.any(), f"{bad.sum()} values off; worst ratio {np.max(err / np.maximum(ref.abs, 1e-300)):.3e}"
    zero = ref.abs == 0
    assert np.all(val[zero] == 0)


def check_product(A, B, smem_bytes=232448, **opts):
    # debug mode on unless the test says otherwise: inputs validated on the device, and every product checked to lie in
    # the columns its chunk owns before it is accumulated (a misplaced product would otherwise be folded in silently)
    opts.setdefault("validate_inputs", 1)
    C, info, stats = run_gpu(A, B, smem_bytes, **opts)
    ref = oracle.spgemm(A, B)
    assert C.n_rows == A.n_rows and C.n_cols == B.n_cols
    assert int(C.row_ptr[0]) == 0 and int(C.row_ptr[-1]) == C.nnz == ref.nnz == stats.c_nnz
    compare_rows(C, ref, A.val.dtype)
    ip = oracle.row_products(A, B)
    assert info.products_total == int(ip.sum())
    tau = info.params.tau
    assert info.rows_heavy == int((ip > tau).sum()) and info.products_heavy == int(ip[ip > tau].sum())
    assert stats.staged_products == info.products_heavy
    return C, info, stats
