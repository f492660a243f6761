"""sp_pack / sp_unpack against the oracle packer: bit-exact positions, coordinates, values."""
import numpy as np
import pytest

from conftest import GOLDEN_FILES, check_invariants, load_golden
from gpu_util import all_encodings, assert_storage_equal, dev, sp, to_dev, unsigned
from paper_2202_04305_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _pack_both(oracle, coo, lt, od, pb=32, cb=32, cbits=32, flags=0):
    coords, vals = to_dev(coo, cbits)
    t = sp().sp_pack(coo.dims, coords, vals, lt, od, pb, cb, flags)
    ref = oracle.pack(coo.dims, coo.coords, coo.vals, lt, od)
    return t, ref


@pytest.mark.parametrize("name", GOLDEN_FILES)
def test_paper_examples(oracle, name):
    g = load_golden(name)
    coo = I.Coo(g["dims"], g["coords"], g["vals"])
    for pb, cb in [(32, 32), (64, 64), (0, 32)]:
        t, _ = _pack_both(oracle, coo, g["lt"], g["ord"], pb, cb)
        for l, tt in enumerate(g["lt"]):
            if tt == 1:
                assert np.array_equal(unsigned(t.positions(l)), g["pos"][l])
                assert np.array_equal(unsigned(t.coordinates(l)), g["crd"][l])
        assert np.array_equal(t.values().cpu().numpy(), g["val"])


@pytest.mark.parametrize("dims,nnz", [((7,), 3), ((1,), 1), ((6, 5), 11), ((5, 8), 0), ((1, 9), 4), ((4, 3, 5), 17),
                                      ((3, 3, 4), 36), ((40, 50, 60), 5000)])
def test_every_encoding_small(oracle, dims, nnz):
    coo = I.uniform_tensor(dims, nnz, seed=len(dims) * 100 + nnz)
    for lt, od in all_encodings(len(dims)):
        for pb, cb, cbits in [(32, 32, 32), (64, 64, 64)]:
            t, ref = _pack_both(oracle, coo, lt, od, pb, cb, cbits)
            assert_storage_equal(t, ref)
            check_invariants(dims, lt, od, [unsigned(t.positions(l)) if lt[l] else None for l in range(len(dims))],
                             [unsigned(t.coordinates(l)) if lt[l] else None for l in range(len(dims))],
                             t.values().cpu().numpy())


@pytest.mark.parametrize("m,n,nnz", [(1000, 900, 4096 * 3 + 17), (70000, 300, 100001), (5, 200000, 4097), (300000, 300000, 250000)])
@pytest.mark.parametrize("enc", [((0, 1), (0, 1)), ((1, 1), (0, 1)), ((0, 1), (1, 0)), ((1, 1), (1, 0)), ((1, 0), (0, 1))])
def test_matrices_spanning_tiles(oracle, m, n, nnz, enc):
    lt, od = enc
    if lt == (1, 0) and m * n > 1 << 26:
        pytest.skip("dense inner level too large to materialise")
    coo = I.uniform_matrix(m, n, nnz, seed=m % 97)
    t, ref = _pack_both(oracle, coo, lt, od)
    assert_storage_equal(t, ref)


def test_widest_keys(oracle):
    # the fused sort key holds at most 63 bits: 3 x 21 bits here (eight radix passes), 2 x 31 for the matrix;
    # one bit more is refused, not truncated
    dims = (1 << 21, 1 << 21, 1 << 21)
    coo = I.uniform_tensor(dims, 9000, seed=12)
    for od in [(0, 1, 2), (2, 0, 1)]:
        t, ref = _pack_both(oracle, coo, (1, 1, 1), od, 32, 32, 32)
        assert_storage_equal(t, ref)
    mat = I.uniform_matrix(1 << 31, 1 << 31, 7000, seed=13)
    for lt, od in [((1, 1), (0, 1)), ((1, 1), (1, 0))]:
        t, ref = _pack_both(oracle, mat, lt, od, 64, 64, 64)
        assert_storage_equal(t, ref)
    b = sp()
    big = I.Coo((1 << 22, 1 << 21, 1 << 21), [np.arange(10) * 7, np.arange(10) * 5, np.arange(10) * 3], np.ones(10))
    coords, vals = to_dev(big, 32)
    with pytest.raises(b.SpError) as e:
        b.sp_pack(big.dims, coords, vals, (1, 1, 1))
    assert e.value.code == 2


def test_confined_rows_and_power_law(oracle):
    for coo in (I.config3(seed=1, n=1 << 14, nnz=60000), I.config2(seed=1, n=4096)):
        for lt, od in [((0, 1), (0, 1)), ((1, 1), (0, 1)), ((0, 1), (1, 0))]:
            t, ref = _pack_both(oracle, coo, lt, od)
            assert_storage_equal(t, ref)


@pytest.mark.parametrize("enc", [((1, 1, 1), (0, 1, 2)), ((0, 1, 1), (0, 1, 2)), ((0, 1, 1), (0, 2, 1)), ((1, 1, 1), (2, 0, 1)),
                                 ((0, 0, 1), (1, 2, 0)), ((1, 0, 1), (0, 1, 2))])
def test_zipf_tensor(oracle, enc):
    coo = I.config5(seed=2, dim=256, nnz=70001)
    t, ref = _pack_both(oracle, coo, *enc)
    assert_storage_equal(t, ref)


def test_duplicates_zeros_and_flags(oracle):
    coo = I.uniform_matrix(50, 60, 500, seed=8)
    coords = [np.concatenate([c, c[:100], c[50:80]]) for c in coo.coords]
    vals = np.concatenate([coo.vals, I.uniform_pm1(8, 70, 130)])
    vals[::7] = 0.0
    dup = I.Coo(coo.dims, coords, vals)
    for lt, od in [((0, 1), (0, 1)), ((1, 1), (1, 0)), ((1, 0), (0, 1))]:
        t, ref = _pack_both(oracle, dup, lt, od)
        assert_storage_equal(t, ref)          # same summation order => same bits
    # the same with keys too wide to carry the entry index inside them (the value travels beside the key then)
    wide = I.uniform_tensor((1 << 20, 1 << 20, 1 << 20), 3000, seed=9)
    wc = [np.concatenate([c, c[:400], c[100:300]]) for c in wide.coords]
    wv = np.concatenate([wide.vals, I.uniform_pm1(8, 71, 600)])
    t, ref = _pack_both(oracle, I.Coo(wide.dims, wc, wv), (1, 1, 1), (1, 2, 0))
    assert_storage_equal(t, ref)
    b = sp()
    c, v = to_dev(dup)
    with pytest.raises(b.SpError) as e:
        b.sp_pack(dup.dims, c, v, (0, 1), None, 32, 32, b.DUP_ERROR)
    assert e.value.code == 5
    c, v = to_dev(coo)
    b.sp_pack(coo.dims, c, v, (0, 1), None, 32, 32, b.DUP_ERROR)   # duplicate-free input passes


@pytest.mark.parametrize("wide", [False, True])
def test_duplicate_runs_across_warp_and_tile_boundaries(oracle, wide):
    """Runs of equal coordinates longer than a warp's round (32), a warp's share (256) and a tile (2048),
    placed so that they straddle those boundaries in sorted order; summed in input order, so the bits
    must match the oracle's.  wide: keys that cannot hold the entry index (values travel with the keys)."""
    dims = (1 << 20, 1 << 20, 1 << 20) if wide else (64, 64, 64)
    base = I.uniform_tensor(dims, 3000, seed=41)
    reps = {5: 40, 700: 300, 701: 31, 1500: 2500, 2999: 270}      # entry of the base list -> copies of it
    cols = [[c] for c in base.coords]
    for e, r in reps.items():
        for d in range(3):
            cols[d].append(np.full(r, base.coords[d][e]))
    coords = [np.concatenate(c) for c in cols]
    n = coords[0].size
    vals = I.uniform_pm1(41, 5, n)
    perm = np.argsort(I.uniform_pm1(41, 6, n), kind="stable")       # a seeded shuffle of the input order
    coo = I.Coo(dims, [c[perm] for c in coords], vals[perm])
    for lt, od in [((1, 1, 1), (0, 1, 2)), ((0, 1, 1), (2, 0, 1))] if not wide else [((1, 1, 1), (0, 1, 2)), ((1, 1, 1), (2, 1, 0))]:
        t, ref = _pack_both(oracle, coo, lt, od)
        assert_storage_equal(t, ref)
        assert t.nval == 3000 if lt == (1, 1, 1) else True


def test_error_codes():
    b = sp()
    coo = I.uniform_matrix(10, 10, 20, seed=1)
    c, v = to_dev(coo)
    bad = [c[0].clone(), c[1].clone()]
    bad[1][3] = 10
    with pytest.raises(b.SpError) as e:
        b.sp_pack(coo.dims, bad, v, (0, 1))
    assert e.value.code == 3
    bad[1][3] = -1
    with pytest.raises(b.SpError) as e:
        b.sp_pack(coo.dims, bad, v, (0, 1))
    assert e.value.code == 3
    with pytest.raises(b.SpError) as e:
        b.sp_pack(coo.dims, c, v, (0, 1), (0, 0))
    assert e.value.code == 1
    with pytest.raises(b.SpError) as e:
        b.sp_pack(coo.dims, c, v, (0, 1), None, 12, 32)
    assert e.value.code == 1
    with pytest.raises(b.SpError) as e:           # 2^33 columns do not fit 32-bit coordinates
        b.sp_pack((4, 1 << 33), c, v, (0, 1), None, 32, 32)
    assert e.value.code == 4
    t = b.sp_pack((4, 1 << 33), [c[0] % 4, c[1]], v, (0, 1), None, 32, 64)
    assert t.coordinates(1).dtype.itemsize == 8


def test_unpack_round_trip(oracle):
    for dims, nnz in [((30, 40), 333), ((9, 8, 7), 200)]:
        coo = I.uniform_tensor(dims, nnz, seed=5)
        for lt, od in all_encodings(len(dims)):
            coords, vals = to_dev(coo)
            t = sp().sp_pack(dims, coords, vals, lt, od)
            oc, ov = sp().sp_unpack(t)
            rc, rv = oracle.unpack(oracle.pack(dims, coo.coords, coo.vals, lt, od))
            for d in range(len(dims)):
                assert np.array_equal(oc[d].cpu().numpy(), rc[d])
            assert np.array_equal(ov.cpu().numpy(), rv)


def test_pack_is_repeatable():
    coo = I.uniform_matrix(5000, 5000, 200000, seed=3)
    coords, vals = to_dev(coo)
    a = sp().sp_pack(coo.dims, coords, vals, (1, 1))
    b = sp().sp_pack(coo.dims, coords, vals, (1, 1))
    for l in range(2):
        assert np.array_equal(a.positions(l).cpu().numpy(), b.positions(l).cpu().numpy())
        assert np.array_equal(a.coordinates(l).cpu().numpy(), b.coordinates(l).cpu().numpy())
    assert np.array_equal(a.values().cpu().numpy(), b.values().cpu().numpy())


def test_rank_four_every_encoding(oracle):
    dims = (5, 3, 6, 4)
    coo = I.uniform_tensor(dims, 97, seed=44)
    coords, vals = to_dev(coo)
    n = 0
    for lt, od in all_encodings(4):
        t = sp().sp_pack(dims, coords, vals, lt, od)
        assert_storage_equal(t, oracle.pack(dims, coo.coords, coo.vals, lt, od))
        n += 1
    assert n == 2 ** 4 * 24


def test_rank_five_sampled_encodings_and_round_trip(oracle):
    dims = (4, 3, 2, 5, 3)
    coo = I.uniform_tensor(dims, 150, seed=45)
    coords, vals = to_dev(coo, 64)
    for n, (lt, od) in enumerate(all_encodings(5)):
        if n % 53:
            continue
        t = sp().sp_pack(dims, coords, vals, lt, od, 64, 32)
        ref = oracle.pack(dims, coo.coords, coo.vals, lt, od)
        assert_storage_equal(t, ref)
        oc, ov = sp().sp_unpack(t)
        rc, rv = oracle.unpack(ref)
        for d in range(5):
            assert np.array_equal(oc[d].cpu().numpy(), rc[d])
        assert np.array_equal(ov.cpu().numpy(), rv)


@pytest.mark.parametrize("dims,nnz", [((183, 24, 1140, 1717), 300_000), ((165427, 11374, 2, 100, 89), 400_000)])
def test_all_compressed_four_and_five_dimensional_shapes(oracle, dims, nnz):
    # the shapes (not the contents) of the 4-d and 5-d tensors whose packing Table 1 times; uniform entries stand in
    coo = I.uniform_tensor(dims, nnz, seed=len(dims))
    coords, vals = to_dev(coo)
    lt = (1,) * len(dims)
    t = sp().sp_pack(dims, coords, vals, lt)
    assert_storage_equal(t, oracle.pack(dims, coo.coords, coo.vals, lt))
    od = tuple(reversed(range(len(dims))))
    t = sp().sp_pack(dims, coords, vals, lt, od)
    assert_storage_equal(t, oracle.pack(dims, coo.coords, coo.vals, lt, od))


def test_convert_between_encodings(oracle):
    # Section 4.2's example converts CSR to CSC; every pair of all-compressed / CSR-like encodings here
    coo = I.uniform_matrix(60, 45, 700, seed=9)
    coords, vals = to_dev(coo)
    encs = [((0, 1), (0, 1)), ((0, 1), (1, 0)), ((1, 1), (0, 1)), ((1, 1), (1, 0))]
    for lt_a, od_a in encs:
        src = sp().sp_pack(coo.dims, coords, vals, lt_a, od_a)
        for lt_b, od_b in encs:
            dst = sp().sp_convert(src, lt_b, od_b, 64, 32)
            assert_storage_equal(dst, oracle.pack(coo.dims, coo.coords, coo.vals, lt_b, od_b))
    t3 = I.uniform_tensor((9, 8, 7), 200, seed=10)
    c3, v3 = to_dev(t3)
    src = sp().sp_pack(t3.dims, c3, v3, (1, 1, 1))
    dst = sp().sp_convert(src, (0, 1, 1), (0, 2, 1))
    assert_storage_equal(dst, oracle.pack(t3.dims, t3.coords, t3.vals, (0, 1, 1), (0, 2, 1)))
    # from a dense-inner encoding the explicit zeros travel along as stored entries
    cdr = sp().sp_pack(coo.dims, coords, vals, (1, 0))
    back = sp().sp_convert(cdr, (0, 1))
    oc, ov = oracle.unpack(oracle.pack(coo.dims, coo.coords, coo.vals, (1, 0)))
    assert_storage_equal(back, oracle.pack(coo.dims, oc, ov, (0, 1)))
