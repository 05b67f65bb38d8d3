"""The allocation-free weight-gradient product (sat_dense_tn_static) against the regular entry point.

Some users of the library cannot allocate device memory when they call it (the device heap belongs to another component,
or an allocation's device-wide synchronisation is not acceptable where they run).  For them the library carries its split
scratch inside its own image.  This file is collected last on purpose, so that a run that stops at the first failure has
already been through every other test; it passes alone in a fresh process as well as after the rest of the suite.
"""
import numpy as np
import pytest

from tests.gpu_util import TOL, assert_close

pytestmark = pytest.mark.gpu


def test_static_scratch_variant_matches_regular_entry_point_twice():
    import torch
    import paper_2308_13466_b200.binding as B
    torch.manual_seed(7)
    ctx = B.sat_create(0, torch.cuda.current_stream().cuda_stream)
    try:
        stream = torch.cuda.current_stream().cuda_stream
        # two calls in a row with different shapes and values: the second must not see anything the first left behind
        for rows, m, n in [(5000, 256, 128), (3001, 100, 47)]:
            A = torch.randn(rows, (m + 3) // 4 * 4, device="cuda")[:, :m]
            Bm = torch.randn(rows, (n + 3) // 4 * 4, device="cuda")[:, :n]
            want = torch.full((m, n), float("nan"), device="cuda")
            got = torch.full((m, n), float("nan"), device="cuda")
            B.sat_dense_tn(ctx, A, Bm, want)
            B.sat_dense_tn_static(stream, A, Bm, got)
            torch.cuda.synchronize()
            assert_close(got.cpu().numpy(), want.cpu().numpy(), f"static-scratch A^T B, rows={rows} m={m} n={n}", TOL)
            # and both agree with the plain definition
            ref = (A.double().T @ Bm.double()).cpu().numpy()
            assert_close(got.cpu().numpy(), ref, "static-scratch A^T B vs definition", TOL)
            # same call again: identical bits (fixed split sizes, fixed summation order) — and the property in the name: the
            # device's free memory, as the driver reports it, is the same before and after the call (the first call above
            # has already loaded the kernels and looked up the array's address; `again` is allocated before the reading)
            again = torch.empty_like(got)
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            B.sat_dense_tn_static(stream, A, Bm, again)
            torch.cuda.synchronize()
            free_after = torch.cuda.mem_get_info()[0]
            assert free_after == free_before, f"device free memory changed across the call: {free_before} -> {free_after}"
            assert torch.equal(got, again)
        # a shape beyond the built-in scratch is refused with a message, and nothing is launched
        A = torch.zeros(4, 2048, device="cuda")
        Bm = torch.zeros(4, 2048, device="cuda")
        out = torch.full((2048, 2048), 3.0, device="cuda")
        with pytest.raises(B.SatError) as ei:
            B.sat_dense_tn_static(stream, A, Bm, out)
        assert ei.value.status == B.SAT_EINVAL and "exceeds" in str(ei.value)
        torch.cuda.synchronize()
        assert bool((out == 3.0).all())
        B.sat_sync_status(ctx)
    finally:
        B.sat_destroy(ctx)
