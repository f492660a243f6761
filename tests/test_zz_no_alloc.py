"""sp_spmv_static: the SpMV entry point for callers that cannot allocate device memory
(fixed-memory real-time loops, plug-ins inside an application that owns the GPU heap).

It must give what sp_spmv gives.  Checked through the C ABI on two calls in a row - the second
with a different vector and a different matrix shape, so anything the first call left in the
library's fixed scratch array would show - for row-major and column-major encodings, and the
allocator hook must stay silent during the calls.  This file is collected last on purpose."""
import ctypes as C

import numpy as np
import pytest

from gpu_util import MATRIX_ENCODINGS, TOL, assert_close, dev, sp, to_dev
from paper_2202_04305_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _both(A, x):
    import torch
    y_ref = sp().sp_spmv(A, x)
    y = torch.full_like(y_ref, 123.0)          # stale contents must be overwritten
    sp().sp_spmv_static(A, x, y)
    return y.cpu().numpy(), y_ref.cpu().numpy()


@pytest.mark.parametrize("widths", [(32, 32), (64, 64), (32, 64), (64, 32)])
@pytest.mark.parametrize("enc", list(MATRIX_ENCODINGS))
def test_static_matches_spmv_two_calls_in_a_row(oracle, enc, widths):
    lt, od = MATRIX_ENCODINGS[enc]
    if widths != (32, 32) and enc in ("DCSR", "CSC"):
        pytest.skip("the mixed and wide width pairs run on the CSR and DCSC encodings")
    big = I.config2(seed=11, n=6000)                       # about 47 tiles, power-law rows
    small = I.row_band_matrix(900, 7, seed=12)             # rows longer than a tile's share, many empty rows
    for coo, xs in ((big, 41), (small, 42)):               # two calls back to back per matrix, four in all
        coords, vals = to_dev(coo)
        A = sp().sp_pack(coo.dims, coords, vals, lt, od, posBits=widths[0], crdBits=widths[1])
        for rep in range(2):
            x = I.uniform_pm1(13, xs + 10 * rep, coo.dims[1])
            got, ref = _both(A, dev(x))
            exact, bound = oracle.spmv(coo.dims[0], coo.coords[0], coo.coords[1], coo.vals, x)
            assert_close(got, exact, bound, f"static {enc} call {rep}")
            # sp_spmv may take another route over the same storage (a lane group per row for short
            # rows), so the two agree to rounding, not bit for bit
            assert np.all(np.abs(got - ref) <= 2 * TOL * bound)


def test_static_never_calls_the_allocator_and_rejects_oversize():
    import torch
    b = sp()
    coo = I.uniform_matrix(500, 400, 3000, seed=5)
    coords, vals = to_dev(coo)
    A = b.sp_pack(coo.dims, coords, vals, (0, 1))
    x = dev(I.uniform_pm1(5, 1, 400))
    y = torch.empty(500, dtype=torch.float64, device="cuda")
    calls = []
    alloc_t = C.CFUNCTYPE(C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p)
    free_t = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p, C.c_void_p)

    def spy_alloc(n, stream, ctx):
        calls.append(n)
        return b._torch_alloc(n, stream, ctx)

    spy_a, spy_f = alloc_t(spy_alloc), free_t(b._torch_free)
    b.use_torch_allocator()
    assert b._lib.sp_set_allocator(spy_a, spy_f, None) == 0
    try:
        before = torch.cuda.memory_stats()["allocation.all.allocated"]
        b.sp_spmv_static(A, x, y)
        b.sp_spmv_static(A, x, y)
        torch.cuda.synchronize()
        assert calls == []
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == before
        b.sp_spmv(A, x)                                   # the ordinary entry point does use the hook
        assert len(calls) > 0
    finally:
        assert b._lib.sp_set_allocator(b._alloc_cb, b._free_cb, None) == 0
    assert np.allclose(y.cpu().numpy(), b.sp_spmv(A, x).cpu().numpy(), rtol=0, atol=1e-12)   # same product, maybe another route

    # more (row ends + entries) than the fixed scratch can describe: refused, nothing launched
    rows = b.SPMV_STATIC_MAX_ITEMS + 5
    one = [torch.zeros(1, dtype=torch.int64, device="cuda"), torch.zeros(1, dtype=torch.int64, device="cuda")]
    huge = b.sp_pack((rows, 4), one, torch.ones(1, dtype=torch.float64, device="cuda"), (0, 1))
    yb = torch.empty(rows, dtype=torch.float64, device="cuda")
    n0 = b.sp_launch_count()
    with pytest.raises(b.SpError) as e:
        b.sp_spmv_static(huge, dev(np.ones(4)), yb)
    assert e.value.code == 9 and b.sp_launch_count() == n0
    ok = b.sp_spmv(huge, dev(np.ones(4)), yb)              # the allocating entry point still handles it
    assert float(ok[0]) == 1.0 and float(ok[1:].abs().max()) == 0.0
