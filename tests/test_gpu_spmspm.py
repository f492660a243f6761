"""sp_spmspm (all-sparse matrix product, Section 4.3 / Table 2) against the oracle:
positions and coordinates bit for bit, values within 1e-12 * sum|a*b|."""
import numpy as np
import pytest

from gpu_util import assert_close, dev, sp, to_dev, unsigned
from paper_2202_04305_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _check(oracle, A, B, pb=32, cb=32, bits=32):
    ac, av = to_dev(A, bits)
    bc, bv = to_dev(B, bits)
    hA = sp().sp_pack(A.dims, ac, av, (0, 1), None, pb, cb)
    hB = sp().sp_pack(B.dims, bc, bv, (0, 1), None, pb, cb)
    hC = sp().sp_spmspm(hA, hB, pb, cb)
    pos, crd, val, bd = oracle.spmspm(A.dims[0], A.dims[1], B.dims[1], A.coords[0], A.coords[1], A.vals,
                                      B.coords[0], B.coords[1], B.vals)
    assert hC.dims == (A.dims[0], B.dims[1]) and hC.lt == (0, 1)
    assert np.array_equal(unsigned(hC.positions(1)), pos)
    assert np.array_equal(unsigned(hC.coordinates(1)), crd)
    assert_close(hC.values().cpu().numpy(), val, bd, "spmspm")
    return hC, (pos, crd, val, bd)


@pytest.mark.parametrize("m,k,n,na,nb", [(9, 7, 8, 20, 25), (30, 30, 30, 90, 90), (5, 6, 4, 0, 10), (12, 3, 40, 36, 100),
                                         (700, 300, 9000, 5000, 20000), (64, 64, 33, 4096, 64 * 33),
                                         # a result row too wide for shared memory: the global workspace path
                                         (300, 200, 60000, 3000, 30000), (40, 50, 28500, 600, 9000)])
def test_small_and_ragged(oracle, m, k, n, na, nb):
    _check(oracle, I.uniform_matrix(m, k, na, seed=m), I.uniform_matrix(k, n, nb, seed=n + 1))


@pytest.mark.parametrize("n", [1024, 2048])
def test_table_2_shapes(oracle, n):
    # uniform random n x n operands of density 0.01 (Section 6.2, Table 2)
    A = I.uniform_matrix(n, n, int(0.01 * n * n), seed=31)
    B = I.uniform_matrix(n, n, int(0.01 * n * n), seed=32)
    hC, (pos, crd, val, bd) = _check(oracle, A, B)
    assert round(crd.size / (n * n), 2) == {1024: 0.10, 2048: 0.19}[n]


def test_wide_indices_power_law_and_reuse_of_the_result(oracle):
    A = I.config2(seed=3, n=1500)
    B = I.config2(seed=4, n=1500)
    hC, (pos, crd, val, bd) = _check(oracle, A, B, 64, 64, 64)
    # the result is an ordinary handle: feed it to SpMV and compare with the oracle on C's entries
    x = I.uniform_pm1(5, 1, 1500)
    rows = np.repeat(np.arange(1500), np.diff(pos))
    yref, yb = oracle.spmv(1500, rows, crd, val, x)
    y = sp().sp_spmv(hC, dev(x)).cpu().numpy()
    assert np.all(np.abs(y - yref) <= 1e-11 * (yb + 1e-300) + 1e-12 * np.abs(bd).sum())


def test_exact_integers_and_errors(oracle):
    A = I.uniform_matrix(200, 150, 3000, seed=7, integer_values=True)
    B = I.uniform_matrix(150, 180, 3000, seed=8, integer_values=True)
    hC, (pos, crd, val, bd) = _check(oracle, A, B)
    assert np.array_equal(hC.values().cpu().numpy(), val)
    b = sp()
    ac, av = to_dev(A)
    csc = b.sp_pack(A.dims, ac, av, (0, 1), (1, 0))
    csr = b.sp_pack(A.dims, ac, av, (0, 1))
    with pytest.raises(b.SpError) as e:
        b.sp_spmspm(csc, csr)
    assert e.value.code == 2
    with pytest.raises(b.SpError) as e:          # inner dimensions differ (200 x 150 times 200 x 150)
        b.sp_spmspm(csr, csr)
    assert e.value.code == 1
