"""The two small kernels of Section 4.3 over storage: in-place scaling and the sparse-sparse
inner product, against the oracle."""
import numpy as np
import pytest

from gpu_util import TOL, sp, to_dev
from paper_2202_04305_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,na,nb,bits", [(50, 10, 12, 32), (100000, 30000, 41000, 32), (20, 0, 5, 64), (4096, 4096, 4096, 64),
                                          (1 << 20, 5, 700000, 32)])
def test_sparse_dot(oracle, n, na, nb, bits):
    a = I.uniform_tensor((n,), na, seed=n % 97)
    b = I.uniform_tensor((n,), nb, seed=n % 89 + 7)
    ha = sp().sp_pack((n,), *to_dev(a, bits), (1,), None, bits, bits)
    hb = sp().sp_pack((n,), *to_dev(b, bits), (1,), None, bits, bits)
    oa, ob = np.argsort(a.coords[0]), np.argsort(b.coords[0])
    x, bd = oracle.vec_dot(a.coords[0][oa], a.vals[oa], b.coords[0][ob], b.vals[ob])
    for u, v in ((ha, hb), (hb, ha)):
        got = float(sp().sp_vec_dot(u, v).cpu()[0])
        assert abs(got - x) <= TOL * bd
        if bd == 0:
            assert got == 0.0


def test_scale_in_place_touches_stored_values_only():
    coo = I.uniform_matrix(40, 30, 300, seed=3)
    coords, vals = to_dev(coo)
    for lt in [(0, 1), (1, 1), (1, 0)]:
        t = sp().sp_pack(coo.dims, coords, vals, lt)
        before = t.values().cpu().numpy().copy()
        pos = [t.positions(l).cpu().numpy().copy() for l in range(2)]
        sp().sp_scale(t, -2.5)
        assert np.array_equal(t.values().cpu().numpy(), before * -2.5)
        for l in range(2):
            assert np.array_equal(t.positions(l).cpu().numpy(), pos[l])


def test_state_space_search_over_encodings():
    # Section 5.2: the result does not depend on the annotation; the search ranks the encodings by time
    import torch
    from paper_2202_04305_b200 import search
    coo = I.row_band_matrix(600, 20, seed=2)
    coords, vals = to_dev(coo)
    x = torch.as_tensor(I.uniform_pm1(2, 3, 600), device="cuda")
    ranked = search.search_matrix_kernel(coo.dims, coords, vals, lambda h: sp().sp_spmv(h, x), widths=[32, 64], reps=2)
    assert len(ranked) == 4 * 2 * 4                     # all level types x orderings x width pairs ran and agreed
    assert all(r["max_dev"] <= 1e-9 for r in ranked)
    # with the narrow widths too: 600 > 2^8 rules 8-bit coordinates out wherever a level is compressed, and
    # 12 000 entries rule 8-bit positions out; (dense, dense) stores no overhead and takes any width
    ranked = search.search_matrix_kernel(coo.dims, coords, vals, lambda h: sp().sp_spmv(h, x), reps=1)
    combos = {(r["levels"], r["posBits"], r["crdBits"]) for r in ranked}
    assert ((0, 0), 8, 8) in combos and ((0, 1), 16, 16) in combos
    assert not any(lt != (0, 0) and cb == 8 for lt, _, cb in combos)
    assert not any(lt[1] == 1 and pb == 8 for lt, pb, _ in combos)
    B = torch.as_tensor(I.dense_operand(2, 4, 600, 8), device="cuda")
    ranked = search.search_matrix_kernel(coo.dims, coords, vals, lambda h: sp().sp_spmm(h, B), widths=[32], reps=2)
    assert len(ranked) == 8
