"""Pins for the oracle's kernels: dense brute force, library routines, closed forms,
exact-integer cases and the error-bound term."""
import numpy as np
import pytest
import scipy.sparse as sp

from paper_2202_04305_b200 import inputs as I


def _dense(coo):
    d = np.zeros(coo.dims)
    d[tuple(coo.coords)] = coo.vals
    return d


def _within(got, ref, bound, tol=1e-12):
    return np.all(np.abs(got - ref) <= tol * bound + 0.0)


@pytest.mark.parametrize("m,n,nnz,N", [(9, 7, 20, 5), (16, 16, 1, 3), (5, 11, 55, 1), (8, 8, 0, 4)])
def test_spmm_dense_brute_force(oracle, m, n, nnz, N):
    coo = I.uniform_matrix(m, n, nnz, seed=m)
    B = I.dense_operand(1, 50, n, N)
    Cm, bd = oracle.spmm(m, coo.coords[0], coo.coords[1], coo.vals, B)
    A = _dense(coo)
    ref = np.zeros((m, N)); refb = np.zeros((m, N))
    for i in range(m):
        for j in range(N):
            for k in range(n):
                ref[i, j] += A[i, k] * B[k, j]
                refb[i, j] += abs(A[i, k] * B[k, j])
    assert _within(Cm, ref, refb)
    assert np.allclose(bd, refb, rtol=1e-14, atol=0)
    assert np.all(Cm[refb == 0] == 0)


def test_spmv_matches_scipy_and_transposed_operand_fails(oracle):
    coo = I.uniform_matrix(40, 31, 300, seed=5)
    x = I.uniform_pm1(5, 60, 31)
    y, bd = oracle.spmv(40, coo.coords[0], coo.coords[1], coo.vals, x)
    A = sp.coo_matrix((coo.vals, (coo.coords[0], coo.coords[1])), shape=coo.dims).tocsr()
    assert _within(y, A @ x, bd, 4e-16 * 31)
    # a transposed operand must not pass (guards the pin itself)
    sq = I.uniform_matrix(31, 31, 200, seed=6)
    y2, b2 = oracle.spmv(31, sq.coords[1], sq.coords[0], sq.vals, x)
    A2 = sp.coo_matrix((sq.vals, (sq.coords[0], sq.coords[1])), shape=sq.dims).tocsr()
    assert not _within(y2, A2 @ x, b2, 1e-9)


def test_spmm_identity_and_ones_closed_forms(oracle):
    n = 12
    eye = np.arange(n)
    B = I.dense_operand(2, 51, n, 6)
    Cm, bd = oracle.spmm(n, eye, eye, np.ones(n), B)
    assert np.array_equal(Cm, B) and np.array_equal(bd, np.abs(B))
    coo = I.uniform_matrix(n, n, 40, seed=9)
    y, _ = oracle.spmv(n, coo.coords[0], coo.coords[1], np.ones(coo.nnz), np.ones(n))
    assert np.array_equal(y, np.bincount(coo.coords[0], minlength=n))


def test_spmm_row_sampling_equals_full(oracle):
    coo = I.uniform_matrix(30, 20, 150, seed=11)
    B = I.dense_operand(3, 52, 20, 4)
    full, fb = oracle.spmm(30, coo.coords[0], coo.coords[1], coo.vals, B)
    rows = np.array([29, 0, 7, 13])
    part, pb = oracle.spmm(30, coo.coords[0], coo.coords[1], coo.vals, B, rows)
    assert np.array_equal(part, full[rows]) and np.array_equal(pb, fb[rows])


@pytest.mark.parametrize("m,n,K,nnz", [(6, 9, 5, 20), (10, 10, 1, 7), (4, 4, 33, 16)])
def test_sddmm_dense_brute_force(oracle, m, n, K, nnz):
    coo = I.uniform_matrix(m, n, nnz, seed=K)
    A = I.dense_operand(4, 53, m, K)
    B = I.dense_operand(4, 54, K, n)
    x, bd = oracle.sddmm(coo.coords[0], coo.coords[1], coo.vals, A, B)
    S = _dense(coo)
    X = S * (A @ B)
    Xb = np.abs(S) * (np.abs(A) @ np.abs(B))
    got = X[coo.coords[0], coo.coords[1]]
    assert _within(x, got, Xb[coo.coords[0], coo.coords[1]], 1e-12)
    assert np.allclose(bd, Xb[coo.coords[0], coo.coords[1]], rtol=1e-13, atol=0)
    # a swapped (i, j) must not pass
    if m == n and nnz > 3:
        x2, b2 = oracle.sddmm(coo.coords[1], coo.coords[0], coo.vals, A, B)
        assert not _within(x2, got, b2, 1e-9)


def test_sddmm_ones_closed_form(oracle):
    coo = I.uniform_matrix(9, 9, 30, seed=2)
    K = 17
    x, bd = oracle.sddmm(coo.coords[0], coo.coords[1], coo.vals, np.ones((9, K)), np.ones((K, 9)))
    assert np.array_equal(x, K * coo.vals) and np.array_equal(bd, K * np.abs(coo.vals))


@pytest.mark.parametrize("dims,nnz,R", [((4, 5, 6), 40, 3), ((3, 3, 3), 27, 8), ((7, 2, 5), 1, 4)])
def test_mttkrp_dense_einsum(oracle, dims, nnz, R):
    coo = I.uniform_tensor(dims, nnz, seed=R)
    B = I.dense_operand(5, 55, dims[1], R)
    Cf = I.dense_operand(5, 56, dims[2], R)
    M, bd = oracle.mttkrp(dims[0], *coo.coords, coo.vals, B, Cf)
    T = _dense(coo)
    ref = np.einsum("ijk,jr,kr->ir", T, B, Cf)
    refb = np.einsum("ijk,jr,kr->ir", np.abs(T), np.abs(B), np.abs(Cf))
    assert _within(M, ref, refb, 1e-12)
    assert np.allclose(bd, refb, rtol=1e-13, atol=0)
    # swapping the two factor matrices must not pass when the modes differ
    if dims[1] == dims[2] and nnz > 3:
        M2, b2 = oracle.mttkrp(dims[0], coo.coords[0], coo.coords[2], coo.coords[1], coo.vals, B, Cf)
        assert not _within(M2, ref, b2, 1e-9)


def test_mttkrp_ones_counts_slice_entries(oracle):
    coo = I.uniform_tensor((6, 5, 4), 50, seed=3)
    M, _ = oracle.mttkrp(6, *coo.coords, np.ones(coo.nnz), np.ones((5, 3)), np.ones((4, 3)))
    assert np.array_equal(M, np.repeat(np.bincount(coo.coords[0], minlength=6)[:, None], 3, 1))


def test_mttkrp_row_sampling_equals_full(oracle):
    t = I.uniform_tensor((9, 7, 6), 120, seed=13)
    R = 5
    Bf = I.dense_operand(3, 53, t.dims[1], R)
    Cf = I.dense_operand(3, 54, t.dims[2], R)
    full, fb = oracle.mttkrp(t.dims[0], *t.coords, t.vals, Bf, Cf)
    rows = np.array([t.dims[0] - 1, 0, 3, 5])
    part, pb = oracle.mttkrp(t.dims[0], *t.coords, t.vals, Bf, Cf, rows)
    assert np.array_equal(part, full[rows]) and np.array_equal(pb, fb[rows])
    # and against the dense definition, so that a slot mapped to the wrong row cannot pass
    T = np.zeros(t.dims)
    T[t.coords[0], t.coords[1], t.coords[2]] = t.vals
    assert np.allclose(part, np.einsum("ijk,jr,kr->ir", T, Bf, Cf)[rows], rtol=0, atol=1e-12)


def test_exact_integer_inputs_are_exact(oracle):
    coo = I.uniform_matrix(20, 20, 120, seed=4, integer_values=True)
    B = I.dense_operand(6, 57, 20, 7, integer_values=True)
    Cm, _ = oracle.spmm(20, coo.coords[0], coo.coords[1], coo.vals, B)
    assert np.array_equal(Cm, _dense(coo) @ B)


def test_extended_precision_accumulation(oracle):
    # 1 + 2^-60 * 4096 terms: a plain f64 running sum would lose every small term.
    n = 4097
    rows = np.zeros(n, np.int64); cols = np.arange(n)
    v = np.full(n, 2.0 ** -60); v[0] = 1.0
    y, bd = oracle.spmv(1, rows, cols, v, np.ones(n))
    assert y[0] == 1.0 + 4096 * 2.0 ** -60 > 1.0
    assert bd[0] == y[0]


@pytest.mark.parametrize("m,k,n,na,nb", [(9, 7, 8, 20, 25), (30, 30, 30, 90, 90), (5, 6, 4, 0, 10), (12, 3, 40, 36, 100)])
def test_spmspm_matches_scipy_and_dense(oracle, m, k, n, na, nb):
    A = I.uniform_matrix(m, k, na, seed=m)
    B = I.uniform_matrix(k, n, nb, seed=n + 1)
    pos, crd, val, bd = oracle.spmspm(m, k, n, A.coords[0], A.coords[1], A.vals, B.coords[0], B.coords[1], B.vals)
    Ad, Bd = _dense(A), _dense(B)
    # pattern: (i, j) is stored iff some k has A[i,k] and B[k,j] both stored
    patt = ((Ad != 0).astype(np.int64) @ (Bd != 0).astype(np.int64)) > 0
    got = np.zeros((m, n), bool)
    rows = np.repeat(np.arange(m), np.diff(pos))
    got[rows, crd] = True
    assert np.array_equal(got, patt)
    for i in range(m):
        seg = crd[pos[i]:pos[i + 1]]
        assert np.all(np.diff(seg) > 0)
    ref = Ad @ Bd
    refb = np.abs(Ad) @ np.abs(Bd)
    assert _within(val, ref[rows, crd], refb[rows, crd])
    assert np.allclose(bd, refb[rows, crd], rtol=1e-13, atol=0)
    S = sp.csr_matrix(Ad) @ sp.csr_matrix(Bd)
    S.sort_indices()
    assert S.nnz <= crd.size           # scipy may drop nothing here, but never has more
    assert np.allclose(S.toarray(), ref)


def test_spmspm_result_density_matches_table_2(oracle):
    # Section 6.2, Table 2: uniform random n x n operands of density 0.01 give rho_C = 0.10 at n = 1,024
    n = 1024
    A = I.uniform_matrix(n, n, int(0.01 * n * n), seed=21)
    B = I.uniform_matrix(n, n, int(0.01 * n * n), seed=22)
    pos, crd, val, bd = oracle.spmspm(n, n, n, A.coords[0], A.coords[1], A.vals, B.coords[0], B.coords[1], B.vals)
    assert round(crd.size / (n * n), 2) == 0.10


@pytest.mark.parametrize("n,na,nb", [(50, 10, 12), (1000, 300, 400), (20, 0, 5), (64, 64, 64)])
def test_sparse_dot_by_co_iteration(oracle, n, na, nb):
    a = I.uniform_tensor((n,), na, seed=n)
    b = I.uniform_tensor((n,), nb, seed=n + 7)
    oa, ob = np.argsort(a.coords[0]), np.argsort(b.coords[0])
    x, bd = oracle.vec_dot(a.coords[0][oa], a.vals[oa], b.coords[0][ob], b.vals[ob])
    da, db = np.zeros(n), np.zeros(n)
    da[a.coords[0]] = a.vals; db[b.coords[0]] = b.vals
    assert abs(x - float(da @ db)) <= 1e-12 * float(np.abs(da) @ np.abs(db)) + 0.0
    assert np.isclose(bd, float(np.abs(da) @ np.abs(db)), rtol=1e-13, atol=0)
    assert oracle.vec_dot(a.coords[0][oa], a.vals[oa], a.coords[0][oa], np.ones(na))[0] == pytest.approx(a.vals.sum(), abs=1e-12)


@pytest.mark.parametrize("lt", [(0, 1), (1, 1)])
def test_storage_loop_nests_match_the_coordinate_loops(oracle, lt):
    """The all-cores baseline loops (over packed storage) against the coordinate-loop definitions."""
    coo = I.confined_rows_matrix(60, 40, 300, row_fraction=0.5, seed=21)
    s = oracle.pack(coo.dims, coo.coords, coo.vals, lt)
    B = I.dense_operand(3, 61, 40, 7)
    ref, bd = oracle.spmm(60, coo.coords[0], coo.coords[1], coo.vals, B)
    got, nt = oracle.par_spmm(s, B)
    assert nt >= 1 and np.all(np.abs(got - ref) <= 1e-15 * bd) and np.all(got[bd == 0] == 0)
    x = I.uniform_pm1(3, 62, 40)
    yref, yb = oracle.spmv(60, coo.coords[0], coo.coords[1], coo.vals, x)
    assert np.all(np.abs(oracle.par_spmv(s, x)[0] - yref) <= 1e-15 * yb)
    A = I.dense_operand(3, 63, 60, 9)
    Bk = I.dense_operand(3, 64, 9, 40)
    xe, xb = oracle.sddmm(coo.coords[0], coo.coords[1], coo.vals, A, Bk)
    xs, _ = oracle.par_sddmm(s, A, Bk)
    assert np.all(np.abs(xs[s.entry_pos] - xe) <= 1e-15 * xb)


@pytest.mark.parametrize("lt", [(0, 1, 1), (1, 1, 1)])
def test_storage_mttkrp_matches_the_coordinate_loop(oracle, lt):
    t = I.zipf_tensor3(12, 400, seed=22)
    s = oracle.pack(t.dims, t.coords, t.vals, lt)
    Bf, Cf = I.dense_operand(3, 65, 12, 6), I.dense_operand(3, 66, 12, 6)
    ref, bd = oracle.mttkrp(12, *t.coords, t.vals, Bf, Cf)
    got, nt = oracle.par_mttkrp(s, Bf, Cf)
    assert nt >= 1 and np.all(np.abs(got - ref) <= 1e-15 * bd) and np.all(got[bd == 0] == 0)
