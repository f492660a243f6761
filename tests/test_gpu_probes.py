"""bench.py's own probe library (random row fetches at given row numbers, register-only f64
multiply-adds, the packer with timed phases): argument checking, the work done, and that the
rates are physically plausible.  None of it is part of the product ABI."""
import numpy as np
import pytest
import torch

import bench
from gpu_util import assert_storage_equal, to_dev
from paper_2202_04305_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def probes():
    return bench.Probes()


def _ms(fn):
    fn(); torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(); n = fn(); b.record(); torch.cuda.synchronize()
    return a.elapsed_time(b), n


@pytest.mark.parametrize("row_elems", [1, 16, 32, 64, 128])
def test_gather_probe_moves_the_bytes_it_reports(probes, row_elems):
    rows, blocks = 4096, 16
    table = torch.rand(rows, row_elems, dtype=torch.float64, device="cuda") if row_elems > 1 else \
        torch.rand(rows, dtype=torch.float64, device="cuda")
    ids = torch.randint(0, rows, (blocks * 8 * 256 * 2,), dtype=torch.int32, device="cuda")
    ms, n = _ms(lambda: probes.gather_rows(table, ids, blocks))
    assert n == ids.numel() * row_elems * 8
    gbs = n / (ms * 1e-3) / 1e9
    assert 1.0 < gbs < 100_000.0               # between "stuck" and "faster than any on-chip path"


def test_gather_probe_sums_the_rows_it_was_given(probes):
    # all row numbers equal: every thread's sum is (rows it fetched) x (its share of that row)
    table = torch.arange(8 * 32, dtype=torch.float64, device="cuda").reshape(8, 32)
    blocks = 1
    ids = torch.full((blocks * 8 * 256,), 5, dtype=torch.int32, device="cuda")
    sink = torch.empty(blocks * 256, dtype=torch.float64, device="cuda")
    import ctypes as C
    rc = probes.lib.spb_gather_rows(C.c_void_p(table.data_ptr()), C.c_int64(8), C.c_int64(32), C.c_void_p(ids.data_ptr()),
                                    C.c_int64(ids.numel()), C.c_int64(blocks), C.c_void_p(sink.data_ptr()), None)
    assert rc == 0
    torch.cuda.synchronize()
    assert float(sink.sum()) == ids.numel() * float(table[5].sum())


def test_gather_probe_rejects_bad_arguments(probes):
    b = probes.sp
    ids = torch.zeros(8 * 256 * 4, dtype=torch.int32, device="cuda")
    with pytest.raises(b.SpError) as e:
        probes.gather_rows(torch.rand(64, 24, dtype=torch.float64, device="cuda"), ids, 4)
    assert e.value.code == 2
    with pytest.raises(b.SpError) as e:      # not whole batches per warp
        probes.gather_rows(torch.rand(64, 32, dtype=torch.float64, device="cuda"), ids[:-32], 4)
    assert e.value.code == 1


def test_dfma_probe_counts_and_rate(probes):
    ms, n = _ms(lambda: probes.dfma(296, 4000))
    assert n == 296 * 256 * 8 * 4000
    tflops = 2 * n / (ms * 1e-3) / 1e12
    assert 0.5 < tflops < 200.0


def test_timed_packer_builds_the_same_storage(probes, oracle):
    coo = I.config3(seed=3, n=1 << 12, nnz=30000)
    coords, vals = to_dev(coo)
    h, phases, passes = probes.pack_timed(coo.dims, coords, vals, (1, 1))
    assert_storage_equal(h, oracle.pack(coo.dims, coo.coords, coo.vals, (1, 1)))
    assert passes >= 1 and set(phases) == set(bench.PACK_PHASES) and all(v >= 0 for v in phases.values())
    assert phases["sort_scatter"] > 0
    h.free()
