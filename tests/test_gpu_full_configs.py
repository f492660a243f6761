"""The five benchmark configurations at full size, through the C ABI, in the encodings and
index widths the benchmark times.  Structure arrays are compared bit for bit with the oracle's
packer and EVERY output value with the oracle's (no sampling: the oracle needs seconds per
configuration), plus properties that hold at any size."""
import numpy as np
import pytest

from gpu_util import assert_close, assert_storage_equal, dev, sp, to_dev
from paper_2202_04305_b200 import inputs as I

pytestmark = pytest.mark.gpu


def test_config1_spmv_csr(oracle):
    coo = I.config1()
    assert coo.dims == (1024, 1024) and coo.nnz == 10486
    coords, vals = to_dev(coo)
    A = sp().sp_pack(coo.dims, coords, vals, (0, 1))
    assert_storage_equal(A, oracle.pack(coo.dims, coo.coords, coo.vals, (0, 1)))
    x = I.uniform_pm1(0, 32, 1024)
    ref, bd = oracle.spmv(1024, coo.coords[0], coo.coords[1], coo.vals, x)
    assert_close(sp().sp_spmv(A, dev(x)).cpu().numpy(), ref, bd, "config 1")


def test_config2_spmm_csr_power_law(oracle):
    coo = I.config2()
    assert coo.dims == (65536, 65536) and abs(coo.nnz / 65536 - 16) < 0.5
    coords, vals = to_dev(coo)
    A = sp().sp_pack(coo.dims, coords, vals, (0, 1))
    assert_storage_equal(A, oracle.pack(coo.dims, coo.coords, coo.vals, (0, 1)))
    B = I.dense_operand(0, 33, 65536, 64)
    ref, bd = oracle.spmm(65536, coo.coords[0], coo.coords[1], coo.vals, B)
    assert_close(sp().sp_spmm(A, dev(B)).cpu().numpy(), ref, bd, "config 2")
    x = I.uniform_pm1(0, 32, 65536)                     # SpMV over the same power-law matrix
    yref, yb = oracle.spmv(65536, coo.coords[0], coo.coords[1], coo.vals, x)
    assert_close(sp().sp_spmv(A, dev(x)).cpu().numpy(), yref, yb, "config 2 spmv")


@pytest.fixture(scope="module")
def c3():
    coo = I.config3()
    assert coo.dims == (1 << 20, 1 << 20) and coo.nnz == 5_000_000
    return coo


@pytest.mark.parametrize("enc", ["CSC", "DCSR"])
def test_config3_pack_and_spmm(oracle, c3, enc):
    import torch
    lt, od = {"CSC": ((0, 1), (1, 0)), "DCSR": ((1, 1), (0, 1))}[enc]
    coords, vals = to_dev(c3)
    A = sp().sp_pack(c3.dims, coords, vals, lt, od)
    assert_storage_equal(A, oracle.pack(c3.dims, c3.coords, c3.vals, lt, od))
    B = I.dense_operand(0, 31, c3.dims[1], 32)
    Cg = sp().sp_spmm(A, dev(B))
    used = np.unique(c3.coords[0])
    assert used.size == c3.meta["rows_used"] == 104858
    rows = used                                        # every row that holds an entry
    ref, bd = oracle.spmm(c3.dims[0], c3.coords[0], c3.coords[1], c3.vals, B, rows)
    assert_close(Cg[dev(rows)].cpu().numpy(), ref, bd, f"config 3 {enc}")
    mask = torch.ones(c3.dims[0], dtype=torch.bool, device="cuda")
    mask[dev(used)] = False
    assert float(Cg[mask].abs().max()) == 0.0          # rows without entries are exactly zero
    x = I.uniform_pm1(0, 32, c3.dims[1])
    yref, yb = oracle.spmv(c3.dims[0], c3.coords[0], c3.coords[1], c3.vals, x, rows)
    yg = sp().sp_spmv(A, dev(x))
    assert_close(yg[dev(rows)].cpu().numpy(), yref, yb, f"config 3 spmv {enc}")
    assert float(yg[mask].abs().max()) == 0.0


def test_config4_sddmm(oracle):
    coo = I.config4()
    assert coo.dims == (131072, 131072) and coo.nnz == 2_000_000
    coords, vals = to_dev(coo)
    S = sp().sp_pack(coo.dims, coords, vals, (0, 1))
    ref = oracle.pack(coo.dims, coo.coords, coo.vals, (0, 1))
    assert_storage_equal(S, ref)
    A = I.dense_operand(0, 35, 131072, 128)
    B = I.dense_operand(0, 36, 128, 131072)
    xg = sp().sp_sddmm(S, dev(A), dev(B)).cpu().numpy()
    xe, be = oracle.sddmm(coo.coords[0], coo.coords[1], coo.vals, A, B)      # all 2,000,000 entries
    assert np.array_equal(np.sort(ref.entry_pos), np.arange(coo.nnz))
    assert_close(xg[ref.entry_pos], xe, be, "config 4")
    # any size: |x_p| <= |s_p| * ||A_i|| * ||B_j||
    An, Bn = np.linalg.norm(A, axis=1), np.linalg.norm(B, axis=0)
    lim = np.empty(coo.nnz); lim[ref.entry_pos] = np.abs(coo.vals) * An[coo.coords[0]] * Bn[coo.coords[1]]
    assert np.all(np.abs(xg) <= lim * (1 + 1e-9))


def test_config5_pack_and_mttkrp(oracle):
    coo = I.config5()
    assert coo.dims == (16384,) * 3 and coo.nnz == 20_000_000
    coords, vals = to_dev(coo)
    T = sp().sp_pack(coo.dims, coords, vals, (1, 1, 1))
    assert_storage_equal(T, oracle.pack(coo.dims, coo.coords, coo.vals, (1, 1, 1)))
    Bf = I.dense_operand(0, 37, 16384, 32)
    Cf = I.dense_operand(0, 38, 16384, 32)
    Mg = sp().sp_mttkrp(T, dev(Bf), dev(Cf)).cpu().numpy()
    ref, bd = oracle.mttkrp(16384, *coo.coords, coo.vals, Bf, Cf)            # all 16,384 x 32 outputs
    assert_close(Mg, ref, bd, "config 5")
    # the dense-first encoding and the interchanged inner order give the same matrix (Section 5.2)
    for lt, od in [((0, 1, 1), (0, 1, 2)), ((0, 1, 1), (0, 2, 1))]:
        T2 = sp().sp_pack(coo.dims, coords, vals, lt, od)
        M2 = sp().sp_mttkrp(T2, dev(Bf), dev(Cf)).cpu().numpy()
        assert_close(M2, ref, bd, f"config 5 {lt} {od}")


def test_row_band_spmv(oracle):
    coo = I.config1b()
    assert coo.nnz == 65_536_000
    coords, vals = to_dev(coo)
    x = I.uniform_pm1(0, 34, 65536)
    ref, bd = oracle.spmv(65536, coo.coords[0], coo.coords[1], coo.vals, x)  # all 65,536 rows
    assert np.all(bd[1000:] == 0) and np.all(bd[:1000] > 0)
    A = sp().sp_pack(coo.dims, coords, vals, (1, 0))          # CDR: the paper's best format for this input
    assert A.nval == 1000 * 65536 and A.positions(0).cpu().numpy().tolist() == [0, 1000]
    y = sp().sp_spmv(A, dev(x)).cpu().numpy()
    assert_close(y, ref, bd, "row band CDR")
    assert np.all(y[1000:] == 0)
    # SpMM over the same handle: the dense contraction (split over the inner dimension, summed with atomics)
    B = I.dense_operand(0, 39, 65536, 32)
    Cg = sp().sp_spmm(A, dev(B)).cpu().numpy()
    cref, cbd = oracle.spmm(65536, coo.coords[0], coo.coords[1], coo.vals, B)   # all 65,536 x 32 outputs
    assert_close(Cg, cref, cbd, "row band CDR SpMM")
    assert np.all(Cg[1000:] == 0)
    for lt in [(0, 1), (1, 1)]:
        A = sp().sp_pack(coo.dims, coords, vals, lt)
        y = sp().sp_spmv(A, dev(x)).cpu().numpy()
        assert_close(y, ref, bd, f"row band {lt}")
        assert np.all(y[1000:] == 0)
        # dense rows: the product is a plain dot with x in column order
        pos = A.positions(1).cpu().numpy().astype(np.int64)
        assert pos[-1] == coo.nnz and np.all(np.diff(pos)[: (1000 if lt == (0, 1) else None)][:1000] == 65536)
