"""The measurement probes of include/sp.h (random row fetches, register-only f64 multiply-adds):
argument checking, the work they report, and that their rates are physically plausible."""
import pytest
import torch

from gpu_util import sp

pytestmark = pytest.mark.gpu


def _ms(fn):
    fn(); torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(); n = fn(); b.record(); torch.cuda.synchronize()
    return a.elapsed_time(b), n


@pytest.mark.parametrize("row_elems,lanes", [(1, 1), (16, 8), (32, 8), (64, 16), (128, 32)])
def test_gather_probe_counts_rows_and_moves_bytes(row_elems, lanes):
    table = torch.rand(4096, row_elems, dtype=torch.float64, device="cuda")
    blocks, per = 64, 100                      # 100 rounds up to 104 (a multiple of the 8 rows in flight)
    ms, n = _ms(lambda: sp().sp_probe_gather(table, blocks, per))
    assert n == blocks * 256 // lanes * 104
    gbs = n * row_elems * 8 / (ms * 1e-3) / 1e9
    assert 1.0 < gbs < 100_000.0               # between "stuck" and "faster than any on-chip path"


def test_gather_probe_rejects_other_row_lengths():
    b = sp()
    with pytest.raises(b.SpError) as e:
        b.sp_probe_gather(torch.rand(64, 24, dtype=torch.float64, device="cuda"), 4, 8)
    assert e.value.code == 2


def test_dfma_probe_counts_and_rate():
    ms, n = _ms(lambda: sp().sp_probe_dfma(296, 4000))
    assert n == 296 * 256 * 8 * 4000
    tflops = 2 * n / (ms * 1e-3) / 1e12
    assert 0.5 < tflops < 200.0
