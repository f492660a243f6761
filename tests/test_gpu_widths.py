"""8- and 16-bit position / coordinate widths (Section 4.1: widths of 8, 16, 32 or 64 bits, which must
hold the largest position / coordinate): storage parity, the overflow rule, and every kernel on
narrow handles."""
import numpy as np
import pytest

from paper_2202_04305_b200 import inputs as I
from gpu_util import sp, to_dev, dev, assert_storage_equal, assert_close, all_encodings, unsigned

pytestmark = pytest.mark.gpu
WIDTHS = (8, 16, 32, 64)


def test_pack_at_every_width_or_overflow(oracle):
    # dims straddle 2^8 and nnz straddles 2^8 / 2^16, so every width is both accepted and refused somewhere
    cases = [((200, 256), 255), ((200, 257), 255), ((256, 256), 256), ((300, 70000), 3000), ((300, 300), 66000)]
    b = sp()
    for dims, nnz in cases:
        coo = I.uniform_matrix(dims[0], dims[1], nnz, seed=nnz + dims[1])
        coords, vals = to_dev(coo)
        for lt, od in all_encodings(2):
            ref = oracle.pack(dims, coo.coords, coo.vals, lt, od)
            need_p, need_c = oracle.min_widths(ref)
            for pb in WIDTHS:
                for cb in WIDTHS:
                    if pb >= need_p and cb >= need_c:
                        t = b.sp_pack(dims, coords, vals, lt, od, pb, cb, b.DUP_SUM)
                        assert (t.pos_bits, t.crd_bits) == (pb, cb)
                        for l in range(2):
                            if lt[l] == 1:
                                assert t.positions(l).element_size() * 8 == pb
                                assert t.coordinates(l).element_size() * 8 == cb
                        assert_storage_equal(t, ref)
                    else:
                        with pytest.raises(b.SpError) as e:
                            b.sp_pack(dims, coords, vals, lt, od, pb, cb, b.DUP_SUM)
                        assert e.value.code == 4


def test_rank3_narrow_and_round_trip(oracle):
    b = sp()
    t3 = I.uniform_tensor((40, 250, 30), 3000, seed=4)
    coords, vals = to_dev(t3)
    for lt, od in [((1, 1, 1), (0, 1, 2)), ((0, 1, 1), (0, 2, 1)), ((1, 0, 1), (2, 0, 1)), ((1, 1, 0), (1, 2, 0))]:
        ref = oracle.pack(t3.dims, t3.coords, t3.vals, lt, od)
        t = b.sp_pack(t3.dims, coords, vals, lt, od, 16, 8)
        assert_storage_equal(t, ref)
        oc, ov = oracle.unpack(ref)
        gc, gv = b.sp_unpack(t)
        assert all(np.array_equal(g.cpu().numpy(), o) for g, o in zip(gc, oc))
        assert np.array_equal(gv.cpu().numpy(), ov)
        wide = b.sp_convert(t, lt, od, 64, 32)
        assert_storage_equal(wide, ref)
        # dense levels hand their explicit zeros on as stored entries, so the count may pass 2^16
        want = oracle.pack(t3.dims, oc, ov, (1, 1, 1), (2, 1, 0))
        pb = max(16, oracle.min_widths(want)[0])
        assert_storage_equal(b.sp_convert(wide, (1, 1, 1), (2, 1, 0), pb, 8), want)
        if pb > 16:
            with pytest.raises(b.SpError) as e:
                b.sp_convert(wide, (1, 1, 1), (2, 1, 0), 16, 8)
            assert e.value.code == 4


@pytest.mark.parametrize("pb,cb", [(16, 8), (8, 8), (16, 16), (32, 8), (16, 64)])
def test_matrix_kernels_on_narrow_handles(oracle, pb, cb):
    b = sp()
    m, n, nnz = 180, 250, 240 if pb == 8 else 5000
    coo = I.uniform_matrix(m, n, nnz, seed=pb * 100 + cb)
    coords, vals = to_dev(coo)
    rng = np.random.default_rng(5)
    x = rng.standard_normal(n)
    B = rng.standard_normal((n, 24))
    Ad, Bd = rng.standard_normal((m, 16)), rng.standard_normal((16, n))
    y_ref, y_bound = oracle.spmv(m, coo.coords[0], coo.coords[1], coo.vals, x)
    c_ref, c_bound = oracle.spmm(m, coo.coords[0], coo.coords[1], coo.vals, B)
    for lt, od in all_encodings(2):
        t = b.sp_pack(coo.dims, coords, vals, lt, od, pb, cb)
        assert_close(b.sp_spmv(t, dev(x)).cpu().numpy(), y_ref, y_bound, f"spmv {lt}{od}")
        assert_close(b.sp_spmm(t, dev(B)).cpu().numpy(), c_ref, c_bound, f"spmm {lt}{od}")
        assert_close(b.sp_spmv(t, dev(x)).cpu().numpy(), y_ref, y_bound, "second call (cached shadow)")
        if lt[1] == 1:
            gi, gj = b.sp_unpack(t)[0]
            x_ref, x_bound = oracle.sddmm(gi.cpu().numpy(), gj.cpu().numpy(), t.values().cpu().numpy(), Ad, Bd)
            assert_close(b.sp_sddmm(t, dev(Ad), dev(Bd)).cpu().numpy(), x_ref, x_bound, f"sddmm {lt}{od}")
            with pytest.raises(b.SpError) as e:       # the allocation-free entry point cannot build a shadow
                b.sp_spmv_static(t, dev(x), dev(np.zeros(m)))
            assert e.value.code == 2


def test_mttkrp_spmspm_and_vec_dot_on_narrow_handles(oracle):
    b = sp()
    rng = np.random.default_rng(6)
    t3 = I.uniform_tensor((50, 200, 120), 6000, seed=8)
    coords, vals = to_dev(t3)
    R = 16
    Bf, Cf = rng.standard_normal((200, R)), rng.standard_normal((120, R))
    ref, bound = oracle.mttkrp(50, t3.coords[0], t3.coords[1], t3.coords[2], t3.vals, Bf, Cf)
    for lt in [(1, 1, 1), (0, 1, 1)]:
        t = b.sp_pack(t3.dims, coords, vals, lt, None, 16, 8)
        assert_close(b.sp_mttkrp(t, dev(Bf), dev(Cf)).cpu().numpy(), ref, bound, f"mttkrp {lt}")

    A = I.uniform_matrix(90, 200, 1500, seed=11)
    Bm = I.uniform_matrix(200, 250, 2000, seed=12)
    ta = b.sp_pack(A.dims, *to_dev(A), (0, 1), None, 16, 8)
    tb = b.sp_pack(Bm.dims, *to_dev(Bm), (0, 1), None, 16, 8)
    cpos, ccrd, cval, cbound = oracle.spmspm(90, 200, 250, A.coords[0], A.coords[1], A.vals, Bm.coords[0], Bm.coords[1], Bm.vals)
    tc = b.sp_spmspm(ta, tb, 16, 8)
    assert tc.positions(1).element_size() == 2 and tc.coordinates(1).element_size() == 1
    assert np.array_equal(unsigned(tc.positions(1)), cpos)
    assert np.array_equal(unsigned(tc.coordinates(1)), ccrd)
    assert_close(tc.values().cpu().numpy(), cval, cbound, "spmspm")
    with pytest.raises(b.SpError) as e:               # 6000+ products' pattern does not fit 8-bit positions
        b.sp_spmspm(ta, tb, 8, 8)
    assert e.value.code == 4

    u = I.uniform_tensor((250,), 100, seed=13)
    v = I.uniform_tensor((250,), 140, seed=14)
    tu = b.sp_pack(u.dims, *to_dev(u), (1,), None, 8, 8)
    tv = b.sp_pack(v.dims, *to_dev(v), (1,), None, 8, 8)
    ou, ov = np.argsort(u.coords[0]), np.argsort(v.coords[0])      # the oracle walks stored (sorted) vectors
    d_ref, d_bound = oracle.vec_dot(u.coords[0][ou], u.vals[ou], v.coords[0][ov], v.vals[ov])
    assert abs(float(b.sp_vec_dot(tu, tv).cpu()[0]) - d_ref) <= 1e-12 * d_bound
