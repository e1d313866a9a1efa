"""The entry point for callers that cannot allocate device memory (a component with a fixed memory
budget, a latency-critical section, a host whose allocator belongs to another runtime):
gm_row_products_noalloc computes the intermediate products per row with its scratch in a fixed array
of the library image.  Checked here, through the C ABI, against the row analysis of gm_spgemm_plan
(the existing entry point) and against the CPU oracle's count, bit for bit because the result is an
integer count, on two calls in a row that share the scratch array.  This file sorts last so that a stop-at-first-failure run has
already been through every other test."""
import numpy as np
import pytest
import torch

import gen
import oracle

pytestmark = pytest.mark.gpu


def _reference(gm, dA, dB):
    plan = gm.spgemm_plan(dA, dB)
    ip = plan.row_products().clone()
    torch.cuda.synchronize()
    plan.destroy()
    return ip


def test_no_alloc_row_products_matches_plan_twice_in_a_row():
    import paper_2607_22866_b200 as gm

    # second input is larger and rectangular, so stale scratch from the first call would show
    A1 = gen.rmat(12, 16, seed=21, dtype=np.float32)
    A2, B2 = gen.zipf_rectangular_pair(1 << 13, 1 << 15, 1 << 17, seed=22, dtype=np.float32)
    assert A1.nnz <= gm.NOALLOC_MAX_NNZ_A and A2.nnz <= gm.NOALLOC_MAX_NNZ_A
    cases = [(gm.DeviceCSR.from_host(A1),) * 2, (gm.DeviceCSR.from_host(A2), gm.DeviceCSR.from_host(B2))]
    refs = [_reference(gm, dA, dB) for dA, dB in cases]
    # the plan's row analysis itself is pinned to the definition (CPU oracle), so both entry points are
    for ref, (hA, hB) in zip(refs, [(A1, A1), (A2, B2)]):
        assert np.array_equal(ref.cpu().numpy(), oracle.row_products(hA, hB))
    outs = [torch.full((dA.n_rows,), -7, dtype=torch.int64, device="cuda") for dA, _ in cases]
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    for (dA, dB), out in zip(cases, outs):          # back to back on the same stream, no sync in between
        gm.row_products_noalloc(dA, dB, out)
    assert torch.cuda.memory_allocated() == before   # nothing came from torch's allocator (the library's hook)
    torch.cuda.synchronize()
    for out, ref, (hA, hB) in zip(outs, refs, [(A1, A1), (A2, B2)]):
        assert torch.equal(out, ref)
        assert np.array_equal(out.cpu().numpy(), oracle.row_products(hA, hB))
    # and once more in the other order: the scratch is reused, nothing needs clearing
    for (dA, dB), out, ref in reversed(list(zip(cases, outs, refs))):
        out.fill_(-1)
        gm.row_products_noalloc(dA, dB, out)
        torch.cuda.synchronize()
        assert torch.equal(out, ref)


def test_no_alloc_rejects_inputs_beyond_its_fixed_scratch():
    import paper_2607_22866_b200 as gm

    A = gen.erdos_renyi_k(1 << 17, 9, seed=3, dtype=np.float32)   # 1,179,648 stored entries > 1,048,576
    assert A.nnz > gm.NOALLOC_MAX_NNZ_A
    dA = gm.DeviceCSR.from_host(A)
    out = torch.zeros(A.n_rows, dtype=torch.int64, device="cuda")
    with pytest.raises(gm.GmError) as ei:
        gm.row_products_noalloc(dA, dA, out)
    assert ei.value.status == -6 and "at most" in str(ei.value)
    # empty input is fine
    E = gm.DeviceCSR(0, 5, torch.zeros(1, dtype=torch.int64, device="cuda"), torch.zeros(0, dtype=torch.int32, device="cuda"),
                     torch.zeros(0, dtype=torch.float32, device="cuda"), 0)
    B = gm.DeviceCSR.from_host(gen.erdos_renyi_k(5, 2, seed=1, dtype=np.float32))
    gm.row_products_noalloc(E, B, torch.zeros(0, dtype=torch.int64, device="cuda"))
    torch.cuda.synchronize()
