"""sp_spmv / sp_spmm / sp_sddmm / sp_mttkrp through the C ABI against the oracle.

Tolerance: |gpu - oracle| <= 1e-12 * sum|a*b| for every output entry (entries whose
bound is 0 must be exactly 0); integer-valued inputs must match bit for bit."""
import numpy as np
import pytest

from gpu_util import MATRIX_ENCODINGS, assert_close, dev, sp, to_dev
from paper_2202_04305_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _matrices():
    yield "uniform", I.uniform_matrix(300, 257, 4000, seed=1)
    yield "tiny", I.uniform_matrix(3, 4, 5, seed=2)
    yield "empty", I.uniform_matrix(17, 9, 0, seed=3)
    yield "one_entry", I.uniform_matrix(40, 40, 1, seed=4)
    yield "powerlaw", I.config2(seed=5, n=3000)
    yield "confined", I.config3(seed=6, n=1 << 13, nnz=30000)
    yield "band", I.row_band_matrix(700, 9, seed=7)
    n = 5000   # one row holds everything / one column holds everything
    yield "one_row", I.Coo((64, n), [np.full(n, 37), np.arange(n)], I.uniform_pm1(8, 1, n))
    yield "one_col", I.Coo((n, 64), [np.arange(n), np.full(n, 11)], I.uniform_pm1(9, 1, n))


MATS = list(_matrices())


@pytest.mark.parametrize("enc", list(MATRIX_ENCODINGS))
@pytest.mark.parametrize("name,coo", MATS, ids=[m[0] for m in MATS])
def test_spmv(oracle, enc, name, coo):
    lt, od = MATRIX_ENCODINGS[enc]
    coords, vals = to_dev(coo)
    A = sp().sp_pack(coo.dims, coords, vals, lt, od)
    x = I.uniform_pm1(11, 2, coo.dims[1])
    y = sp().sp_spmv(A, dev(x)).cpu().numpy()
    ref, bd = oracle.spmv(coo.dims[0], coo.coords[0], coo.coords[1], coo.vals, x)
    assert_close(y, ref, bd, f"spmv {enc} {name}")


DENSE_INNER = {"CDR": ((1, 0), (0, 1)), "DD": ((0, 0), (0, 1)), "CDC": ((1, 0), (1, 0)), "DD-col": ((0, 0), (1, 0))}


@pytest.mark.parametrize("enc", list(DENSE_INNER))
@pytest.mark.parametrize("name,coo", MATS, ids=[m[0] for m in MATS])
def test_spmv_dense_inner_level(oracle, enc, name, coo):
    # (compressed, dense) is the paper's CDR (Section 6.2); explicit zeros in the stored slices add nothing
    lt, od = DENSE_INNER[enc]
    outer_dim = coo.dims[od[0]]
    stored = outer_dim if lt[0] == 0 else np.unique(coo.coords[od[0]]).size
    if stored * coo.dims[od[1]] > 1 << 24:
        pytest.skip("dense slices too large to materialise")
    coords, vals = to_dev(coo)
    A = sp().sp_pack(coo.dims, coords, vals, lt, od)
    x = I.uniform_pm1(11, 2, coo.dims[1])
    y = sp().sp_spmv(A, dev(x)).cpu().numpy()
    ref, bd = oracle.spmv(coo.dims[0], coo.coords[0], coo.coords[1], coo.vals, x)
    assert_close(y, ref, bd, f"spmv {enc} {name}")


@pytest.mark.parametrize("enc", list(DENSE_INNER))
@pytest.mark.parametrize("N", [1, 7, 32, 70])
@pytest.mark.parametrize("name,coo", MATS, ids=[m[0] for m in MATS])
def test_spmm_dense_inner_level(oracle, enc, N, name, coo):
    lt, od = DENSE_INNER[enc]
    stored = coo.dims[od[0]] if lt[0] == 0 else np.unique(coo.coords[od[0]]).size
    if stored * coo.dims[od[1]] > 1 << 22 or (N in (7, 70) and name not in ("uniform", "band", "tiny")):
        pytest.skip("dense slices too large, or ragged width covered elsewhere")
    coords, vals = to_dev(coo)
    A = sp().sp_pack(coo.dims, coords, vals, lt, od)
    B = I.dense_operand(12, 3, coo.dims[1], N)
    Cg = sp().sp_spmm(A, dev(B)).cpu().numpy()
    ref, bd = oracle.spmm(coo.dims[0], coo.coords[0], coo.coords[1], coo.vals, B)
    assert_close(Cg, ref, bd, f"spmm {enc} {name} N={N}")


@pytest.mark.parametrize("m,n,nnz,N,ldb,shift,cbits", [
    (700, 518, 60000, 50, 52, 0, 32),      # ragged rows, k and columns; padded B: copy-engine feed
    (700, 518, 60000, 50, 52, 1, 32),      # B starts 8 bytes off a 16-byte boundary: register-staged feed
    (700, 517, 60000, 32, 32, 0, 32),      # odd slice length: register-staged feed
    (300, 20000, 90000, 32, 32, 0, 64),    # few rows, long contraction: split over k, 64-bit coordinates
    (40, 30, 500, 8, 8, 0, 32),            # smaller than one tile in every direction
])
@pytest.mark.parametrize("lt", [(1, 0), (0, 0)])
def test_spmm_dense_inner_both_feeds(oracle, m, n, nnz, N, ldb, shift, cbits, lt):
    """Row-major products over a dense inner level run on the tensor-memory-accelerator feed when
    every row of the stored slices and of B starts on a 16-byte boundary, and on the register-staged
    kernel otherwise; both must agree with the oracle, ignore what lies beyond B's N columns and leave
    the other columns of a strided C alone."""
    import torch
    coo = I.uniform_matrix(m, n, nnz, seed=31)
    B = I.dense_operand(31, 3, n, N)
    ref, bd = oracle.spmm(m, coo.coords[0], coo.coords[1], coo.vals, B)
    coords, vals = to_dev(coo, cbits)
    A = sp().sp_pack(coo.dims, coords, vals, lt, (0, 1), 32, cbits)
    flat = torch.full((n * ldb + 2,), 1e300, dtype=torch.float64, device="cuda")
    Bdev = flat[shift:shift + n * ldb].view(n, ldb)[:, :N]
    Bdev.copy_(dev(B))
    Cbig = torch.full((m, N + 3), 7.0, dtype=torch.float64, device="cuda")
    sp().sp_spmm(A, Bdev, Cbig[:, :N])
    assert_close(Cbig[:, :N].cpu().numpy(), ref, bd, "dense inner")
    assert torch.all(Cbig[:, N:] == 7.0)


@pytest.mark.parametrize("enc", list(MATRIX_ENCODINGS))
@pytest.mark.parametrize("N", [1, 5, 32, 64, 70])
@pytest.mark.parametrize("name,coo", MATS, ids=[m[0] for m in MATS])
def test_spmm(oracle, enc, N, name, coo):
    if N in (5, 70) and name not in ("uniform", "powerlaw", "one_row"):
        pytest.skip("ragged widths are covered on three matrices")
    lt, od = MATRIX_ENCODINGS[enc]
    coords, vals = to_dev(coo)
    A = sp().sp_pack(coo.dims, coords, vals, lt, od)
    B = I.dense_operand(12, 3, coo.dims[1], N)
    Cg = sp().sp_spmm(A, dev(B)).cpu().numpy()
    ref, bd = oracle.spmm(coo.dims[0], coo.coords[0], coo.coords[1], coo.vals, B)
    assert_close(Cg, ref, bd, f"spmm {enc} {name} N={N}")


def test_spmm_strided_operands_and_wide_indices(oracle):
    import torch
    coo = I.config2(seed=3, n=2000)
    B = I.dense_operand(1, 4, 2000, 48)
    ref, bd = oracle.spmm(2000, coo.coords[0], coo.coords[1], coo.vals, B)
    for pb, cb, cbits in [(64, 64, 64), (32, 64, 32), (64, 32, 64)]:
        coords, vals = to_dev(coo, cbits)
        for enc in MATRIX_ENCODINGS.values():
            A = sp().sp_pack(coo.dims, coords, vals, enc[0], enc[1], pb, cb)
            Bbig = torch.zeros((2000, 50), dtype=torch.float64, device="cuda")
            Bbig[:, :48] = dev(B)
            Cbig = torch.full((2000, 51), 7.0, dtype=torch.float64, device="cuda")
            sp().sp_spmm(A, Bbig[:, :48], Cbig[:, :48])
            assert_close(Cbig[:, :48].cpu().numpy(), ref, bd, "strided")
            assert torch.all(Cbig[:, 48:] == 7.0)


@pytest.mark.parametrize("N", [16, 32, 64, 128])
@pytest.mark.parametrize("lt", [(0, 1), (1, 1)])
def test_spmm_lane_group_per_row(oracle, N, lt):
    """Rows of even, moderate length take the lane-group kernel (N = 16, 32, 64, 128): stored rows, rows
    without entries (written as zeros, including those a compressed level 0 elides before the first,
    between, and after the last stored row), a strided C whose other columns must stay untouched, and
    every index width."""
    import torch
    m, n = 900, 700
    rows = np.setdiff1d(np.arange(5, m - 9), np.arange(100, 140))       # rows 0-4, 100-139 and the last 9 hold nothing
    r = np.repeat(rows, 12)
    c = (I.randint(21, 1, r.size, n // 12) + np.tile(np.arange(12) * (n // 12), rows.size)).astype(np.int64)   # distinct per row
    v = I.uniform_pm1(21, 2, r.size)
    perm = I.affine_scramble(r.size, 3)
    coo = I.Coo((m, n), [r[perm], c[perm]], v[perm])
    B = I.dense_operand(21, 3, n, N)
    ref, bd = oracle.spmm(m, coo.coords[0], coo.coords[1], coo.vals, B)
    for pb, cb, cbits in [(32, 32, 32), (64, 64, 64), (32, 64, 32), (64, 32, 64)]:
        coords, vals = to_dev(coo, cbits)
        A = sp().sp_pack(coo.dims, coords, vals, lt, None, pb, cb)
        Bbig = torch.zeros((n, N + 2), dtype=torch.float64, device="cuda")
        Bbig[:, :N] = dev(B)
        Cbig = torch.full((m, N + 4), 7.0, dtype=torch.float64, device="cuda")
        sp().sp_spmm(A, Bbig[:, :N], Cbig[:, :N])
        assert_close(Cbig[:, :N].cpu().numpy(), ref, bd, f"rows {lt} N={N}")
        assert torch.all(Cbig[:, N:] == 7.0)
        x = I.uniform_pm1(21, 4, n)
        yref, yb = oracle.spmv(m, coo.coords[0], coo.coords[1], coo.vals, x)
        y = torch.full((m,), 7.0, dtype=torch.float64, device="cuda")
        assert_close(sp().sp_spmv(A, dev(x), y).cpu().numpy(), yref, yb, f"spmv rows {lt}")


def test_results_do_not_depend_on_encoding(oracle):
    # Section 5.2: the result is independent of the sparsity annotation, up to reassociation.
    coo = I.uniform_matrix(500, 400, 9000, seed=21)
    B = I.dense_operand(2, 5, 400, 16)
    ref, bd = oracle.spmm(500, coo.coords[0], coo.coords[1], coo.vals, B)
    coords, vals = to_dev(coo)
    outs = []
    for lt, od in MATRIX_ENCODINGS.values():
        for pb in (32, 64):
            A = sp().sp_pack(coo.dims, coords, vals, lt, od, pb, pb)
            outs.append(sp().sp_spmm(A, dev(B)).cpu().numpy())
    for o in outs:
        assert_close(o, ref, bd)
        assert np.all(np.abs(o - outs[0]) <= 2e-12 * bd)


def test_exact_for_integer_inputs(oracle):
    coo = I.config2(seed=4, n=1500, integer_values=True)
    B = I.dense_operand(3, 6, 1500, 64, integer_values=True)
    x = I.small_ints(3, 7, 1500)
    ref, _ = oracle.spmm(1500, coo.coords[0], coo.coords[1], coo.vals, B)
    yref, _ = oracle.spmv(1500, coo.coords[0], coo.coords[1], coo.vals, x)
    coords, vals = to_dev(coo)
    for lt, od in MATRIX_ENCODINGS.values():
        A = sp().sp_pack(coo.dims, coords, vals, lt, od)
        assert np.array_equal(sp().sp_spmm(A, dev(B)).cpu().numpy(), ref)
        assert np.array_equal(sp().sp_spmv(A, dev(x)).cpu().numpy(), yref)


def test_unsupported_encodings():
    b = sp()
    coo = I.uniform_matrix(20, 20, 50, seed=1)
    coords, vals = to_dev(coo)
    T = b.sp_pack((20, 20, 1), coords + [coords[0] * 0], vals, (1, 1, 1))
    with pytest.raises(b.SpError) as e:
        b.sp_spmv(T, dev(np.ones(20)))
    assert e.value.code == 2
    with pytest.raises(b.SpError) as e:          # MTTKRP wants a rank-3 tensor
        b.sp_mttkrp(b.sp_pack(coo.dims, coords, vals, (0, 1)), dev(np.ones((20, 4))), dev(np.ones((20, 4))))
    assert e.value.code == 2


# ------------------------------------------------------------------ SDDMM
@pytest.mark.parametrize("lt", [(0, 1), (1, 1)])
@pytest.mark.parametrize("K", [1, 5, 64, 128, 130, 256, 300])
def test_sddmm(oracle, lt, K):
    for name, coo in [("uniform", I.uniform_matrix(300, 257, 4000, seed=1)), ("confined", I.config3(seed=6, n=1 << 12, nnz=9000)),
                      ("one_row", MATS[7][1]), ("empty", I.uniform_matrix(9, 9, 0, seed=1))]:
        coords, vals = to_dev(coo)
        S = sp().sp_pack(coo.dims, coords, vals, lt)
        A = I.dense_operand(13, 8, coo.dims[0], K)
        B = I.dense_operand(13, 9, K, coo.dims[1])
        xg = sp().sp_sddmm(S, dev(A), dev(B)).cpu().numpy()
        xe, be = oracle.sddmm(coo.coords[0], coo.coords[1], coo.vals, A, B)
        ep = oracle.pack(coo.dims, coo.coords, coo.vals, lt).entry_pos
        ref = np.empty_like(xe); bd = np.empty_like(be)
        ref[ep] = xe; bd[ep] = be
        assert_close(xg, ref, bd, f"sddmm {name} K={K}")


def test_sddmm_exact_integers(oracle):
    coo = I.uniform_matrix(200, 200, 3000, seed=2, integer_values=True)
    A = I.dense_operand(1, 8, 200, 128, integer_values=True)
    B = I.dense_operand(1, 9, 128, 200, integer_values=True)
    coords, vals = to_dev(coo)
    S = sp().sp_pack(coo.dims, coords, vals, (0, 1))
    xe, _ = oracle.sddmm(coo.coords[0], coo.coords[1], coo.vals, A, B)
    ref = np.empty_like(xe)
    ref[oracle.pack(coo.dims, coo.coords, coo.vals, (0, 1)).entry_pos] = xe
    assert np.array_equal(sp().sp_sddmm(S, dev(A), dev(B)).cpu().numpy(), ref)


# ----------------------------------------------------------------- MTTKRP
TENSOR_ENCODINGS = {"CSF": ((1, 1, 1), (0, 1, 2)), "DSS": ((0, 1, 1), (0, 1, 2)), "DSS-alt": ((0, 1, 1), (0, 2, 1)),
                    "CSF-alt": ((1, 1, 1), (0, 2, 1))}


def _tensors():
    yield "zipf", I.config5(seed=3, dim=200, nnz=40000)
    yield "zipf_wide", I.config5(seed=11, dim=3000, nnz=120000)     # more leaf coordinates than hot-row slots
    yield "uniform", I.uniform_tensor((50, 40, 30), 3000, seed=4)
    yield "tiny", I.uniform_tensor((3, 3, 4), 5, seed=5)
    yield "empty", I.uniform_tensor((6, 5, 4), 0, seed=6)
    n = 6000
    yield "one_slice", I.Coo((10, 80, 90), [np.full(n, 3), np.arange(n) // 90 % 80, np.arange(n) % 90], I.uniform_pm1(1, 2, n))
    yield "one_fibre", I.Coo((10, 8, n), [np.full(n, 9), np.full(n, 2), np.arange(n)], I.uniform_pm1(1, 3, n))


TENS = list(_tensors())


@pytest.mark.parametrize("enc", list(TENSOR_ENCODINGS))
@pytest.mark.parametrize("R", [1, 5, 32, 40])
@pytest.mark.parametrize("name,coo", TENS, ids=[t[0] for t in TENS])
def test_mttkrp(oracle, enc, R, name, coo):
    lt, od = TENSOR_ENCODINGS[enc]
    coords, vals = to_dev(coo)
    T = sp().sp_pack(coo.dims, coords, vals, lt, od)
    B = I.dense_operand(14, 10, coo.dims[1], R)
    Cf = I.dense_operand(14, 11, coo.dims[2], R)
    M = sp().sp_mttkrp(T, dev(B), dev(Cf)).cpu().numpy()
    ref, bd = oracle.mttkrp(coo.dims[0], *coo.coords, coo.vals, B, Cf)
    assert_close(M, ref, bd, f"mttkrp {enc} {name} R={R}")


def test_mttkrp_exact_integers(oracle):
    coo = I.config5(seed=7, dim=128, nnz=20000, integer_values=True)
    B = I.dense_operand(2, 10, 128, 32, integer_values=True)
    Cf = I.dense_operand(2, 11, 128, 32, integer_values=True)
    ref, _ = oracle.mttkrp(128, *coo.coords, coo.vals, B, Cf)
    coords, vals = to_dev(coo)
    for lt, od in TENSOR_ENCODINGS.values():
        T = sp().sp_pack(coo.dims, coords, vals, lt, od)
        assert np.array_equal(sp().sp_mttkrp(T, dev(B), dev(Cf)).cpu().numpy(), ref)


@pytest.mark.parametrize("pb,cb,cbits", [(64, 64, 64), (32, 64, 32), (64, 32, 64), (0, 0, 32)])
def test_every_kernel_with_wide_positions_and_coordinates(oracle, pb, cb, cbits):
    # Section 4.1: pointer and index bit widths are part of the encoding; 0 means the native 64 bits
    m = I.config2(seed=8, n=1200)
    coords, vals = to_dev(m, cbits)
    x = I.uniform_pm1(1, 2, 1200)
    yref, yb = oracle.spmv(1200, m.coords[0], m.coords[1], m.vals, x)
    for lt, od in list(MATRIX_ENCODINGS.values()) + [((1, 0), (0, 1))]:
        A = sp().sp_pack(m.dims, coords, vals, lt, od, pb, cb)
        assert A.pos_bits == (pb or 64) and A.crd_bits == (cb or 64)
        assert_close(sp().sp_spmv(A, dev(x)).cpu().numpy(), yref, yb, f"spmv widths {pb}/{cb}")
    A4, B4 = I.dense_operand(2, 8, 1200, 64), I.dense_operand(2, 9, 64, 1200)
    xe, be = oracle.sddmm(m.coords[0], m.coords[1], m.vals, A4, B4)
    for lt in [(0, 1), (1, 1)]:
        S = sp().sp_pack(m.dims, coords, vals, lt, None, pb, cb)
        ep = oracle.pack(m.dims, m.coords, m.vals, lt).entry_pos
        ref = np.empty_like(xe); bd = np.empty_like(be)
        ref[ep] = xe; bd[ep] = be
        assert_close(sp().sp_sddmm(S, dev(A4), dev(B4)).cpu().numpy(), ref, bd, f"sddmm widths {pb}/{cb}")
    t = I.config5(seed=9, dim=96, nnz=15000)
    tc, tv = to_dev(t, cbits)
    Bf, Cf = I.dense_operand(3, 10, 96, 32), I.dense_operand(3, 11, 96, 32)
    Mref, Mb = oracle.mttkrp(96, *t.coords, t.vals, Bf, Cf)
    for lt, od in TENSOR_ENCODINGS.values():
        T = sp().sp_pack(t.dims, tc, tv, lt, od, pb, cb)
        assert_close(sp().sp_mttkrp(T, dev(Bf), dev(Cf)).cpu().numpy(), Mref, Mb, f"mttkrp widths {pb}/{cb}")
        for R in (5,):      # the generic (odd R) kernel as well
            B5, C5 = I.dense_operand(3, 12, 96, R), I.dense_operand(3, 13, 96, R)
            r5, b5 = oracle.mttkrp(96, *t.coords, t.vals, B5, C5)
            assert_close(sp().sp_mttkrp(T, dev(B5), dev(C5)).cpu().numpy(), r5, b5, f"mttkrp R=5 widths {pb}/{cb}")


@pytest.mark.parametrize("enc", ["CSC", "DCSC"])
@pytest.mark.parametrize("K", [5, 64, 128, 300])
def test_sddmm_column_major_sample(oracle, enc, K):
    lt, od = MATRIX_ENCODINGS[enc]
    for name, coo in [("uniform", I.uniform_matrix(300, 257, 4000, seed=1)), ("one_col", MATS[8][1]),
                      ("powerlaw", I.config2(seed=2, n=900))]:
        coords, vals = to_dev(coo)
        S = sp().sp_pack(coo.dims, coords, vals, lt, od)
        A = I.dense_operand(13, 8, coo.dims[0], K)
        B = I.dense_operand(13, 9, K, coo.dims[1])
        xg = sp().sp_sddmm(S, dev(A), dev(B)).cpu().numpy()
        xe, be = oracle.sddmm(coo.coords[0], coo.coords[1], coo.vals, A, B)
        ep = oracle.pack(coo.dims, coo.coords, coo.vals, lt, od).entry_pos
        ref = np.empty_like(xe); bd = np.empty_like(be)
        ref[ep] = xe; bd[ep] = be
        assert_close(xg, ref, bd, f"sddmm {enc} {name} K={K}")


@pytest.mark.parametrize("lt", [(1, 0), (0, 0)])
@pytest.mark.parametrize("od", [(0, 1), (1, 0)])
@pytest.mark.parametrize("K", [1, 7, 64, 130])
def test_sddmm_dense_inner_level(oracle, lt, od, K):
    # S with a dense inner level: every cell of a stored row (column) is a stored value, explicit zeros included
    for name, coo in [("uniform", I.uniform_matrix(300, 257, 4000, seed=1)), ("band", I.row_band_matrix(270, 9, seed=4)),
                      ("one_row", MATS[7][1]), ("empty", I.uniform_matrix(9, 9, 0, seed=1))]:
        coords, vals = to_dev(coo)
        S = sp().sp_pack(coo.dims, coords, vals, lt, od)
        A = I.dense_operand(13, 8, coo.dims[0], K)
        B = I.dense_operand(13, 9, K, coo.dims[1])
        xg = sp().sp_sddmm(S, dev(A), dev(B)).cpu().numpy()
        (si, sj), sv = oracle.unpack(oracle.pack(coo.dims, coo.coords, coo.vals, lt, od))   # stored cells, storage order
        assert xg.size == sv.size
        if sv.size:
            ref, bd = oracle.sddmm(si, sj, sv, A, B)
            assert_close(xg, ref, bd, f"sddmm dense inner {lt}{od} {name} K={K}")


@pytest.mark.parametrize("mode", [0, 1, 2])
@pytest.mark.parametrize("R", [5, 32])
def test_mttkrp_any_output_mode(oracle, mode, R):
    t = I.config5(seed=5, dim=150, nnz=30000)
    dims = (150, 150, 150)
    F = [I.dense_operand(6, 20 + d, 150, R) for d in range(3)]
    others = [d for d in range(3) if d != mode]
    # oracle: the mode-0 expression with the coordinates rotated so that `mode` comes first
    ref, bd = oracle.mttkrp(dims[mode], t.coords[mode], t.coords[others[0]], t.coords[others[1]], t.vals,
                            F[others[0]], F[others[1]])
    coords, vals = to_dev(t)
    for lt in [(1, 1, 1), (0, 1, 1)]:
        for od in [(mode, others[0], others[1]), (mode, others[1], others[0])]:
            T = sp().sp_pack(dims, coords, vals, lt, od)
            M = sp().sp_mttkrp_mode(T, mode, [dev(f) for f in F]).cpu().numpy()
            assert_close(M, ref, bd, f"mttkrp mode {mode} {lt} {od}")
    b = sp()
    Tbad = b.sp_pack(dims, coords, vals, (1, 1, 1), ((mode + 1) % 3, mode, 3 - mode - (mode + 1) % 3))
    with pytest.raises(b.SpError) as e:
        b.sp_mttkrp_mode(Tbad, mode, [dev(f) for f in F])
    assert e.value.code == 2


def test_one_handle_on_two_streams(oracle):
    """Calls on different streams share a handle: its cached tables are read-only once built and every
    call's scratch (row carries) is its own.  Two streams run SpMM and SpMV over the same handle, merge
    path and lane-group routes, with different operands, interleaved; both results must be right."""
    import torch
    for coo in (I.config2(seed=31, n=4000), I.config3(seed=32, n=1 << 12, nnz=40000)):
        coords, vals = to_dev(coo)
        A = sp().sp_pack(coo.dims, coords, vals, (0, 1))
        m, n = coo.dims
        Bs = [I.dense_operand(31, 10 + k, n, 32) for k in range(2)]
        xs = [I.uniform_pm1(31, 20 + k, n) for k in range(2)]
        refs = [oracle.spmm(m, coo.coords[0], coo.coords[1], coo.vals, B) for B in Bs]
        yrefs = [oracle.spmv(m, coo.coords[0], coo.coords[1], coo.vals, x) for x in xs]
        streams = [torch.cuda.Stream(), torch.cuda.Stream()]
        dB, dx = [dev(B) for B in Bs], [dev(x) for x in xs]
        outs = [torch.empty(m, 32, dtype=torch.float64, device="cuda") for _ in range(2)]
        ys = [torch.empty(m, dtype=torch.float64, device="cuda") for _ in range(2)]
        torch.cuda.synchronize()
        for rep in range(5):
            for k, st in enumerate(streams):
                with torch.cuda.stream(st):
                    sp().sp_spmm(A, dB[k], outs[k])
                    sp().sp_spmv(A, dx[k], ys[k])
        torch.cuda.synchronize()
        for k in range(2):
            assert_close(outs[k].cpu().numpy(), refs[k][0], refs[k][1], f"stream {k} spmm")
            assert_close(ys[k].cpu().numpy(), yrefs[k][0], yrefs[k][1], f"stream {k} spmv")
