"""Pins for the oracle packer: the paper's worked examples, invariants, library and
textbook reductions, round trip and dense brute force over every encoding (d <= 3)."""
import itertools

import numpy as np
import pytest
import scipy.sparse as sp

from conftest import GOLDEN_FILES, check_invariants, load_golden
from paper_2202_04305_b200 import inputs as I


@pytest.mark.parametrize("name", GOLDEN_FILES)
def test_paper_examples(oracle, name):
    g = load_golden(name)
    s = oracle.pack(g["dims"], g["coords"], g["vals"], g["lt"], g["ord"])
    for l, t in enumerate(g["lt"]):
        if t == 1:
            assert np.array_equal(s.pos[l], g["pos"][l]), (name, l)
            assert np.array_equal(s.crd[l], g["crd"][l]), (name, l)
        else:
            assert s.pos[l] is None and l not in g["pos"]
    assert np.array_equal(s.val, g["val"])
    check_invariants(g["dims"], g["lt"], g["ord"], s.pos, s.crd, s.val)


@pytest.mark.parametrize("name", GOLDEN_FILES)
def test_paper_examples_any_input_order(oracle, name):
    g = load_golden(name)
    n = g["vals"].size
    for perm in itertools.islice(itertools.permutations(range(n)), 0, 120, 7):
        perm = list(perm)
        s = oracle.pack(g["dims"], [c[perm] for c in g["coords"]], g["vals"][perm], g["lt"], g["ord"])
        assert np.array_equal(s.val, g["val"])
        for l in g["pos"]:
            assert np.array_equal(s.pos[l], g["pos"][l]) and np.array_equal(s.crd[l], g["crd"][l])


def test_storage_saving_sparse_vector(oracle):
    # Section 4.1: the compressed vector stores 4 doubles and 6 integers instead of 16 doubles.
    g = load_golden("sparse_vector_16.txt")
    s = oracle.pack(g["dims"], g["coords"], g["vals"], g["lt"], g["ord"])
    assert s.val.size == 4 and s.pos[0].size + s.crd[0].size == 6


def _all_encodings(rank):
    for lt in itertools.product((0, 1), repeat=rank):
        for ord in itertools.permutations(range(rank)):
            yield lt, ord


def _dense_of(dims, coords, vals):
    d = np.zeros(dims)
    np.add.at(d, tuple(coords), vals)
    return d


@pytest.mark.parametrize("dims,nnz", [((7,), 3), ((6, 5), 11), ((5, 8), 0), ((4, 3, 5), 17), ((3, 3, 4), 36),
                                      ((3, 2, 4, 3), 19)])
def test_round_trip_dense_brute_force_all_encodings(oracle, dims, nnz):
    rank = len(dims)
    coo = I.uniform_tensor(dims, nnz, seed=rank + nnz)
    ref = _dense_of(dims, coo.coords, coo.vals)
    key_in = sorted(zip(*[c.tolist() for c in coo.coords], coo.vals.tolist()))
    count = 0
    for lt, ord in _all_encodings(rank):
        s = oracle.pack(dims, coo.coords, coo.vals, lt, ord)
        check_invariants(dims, lt, ord, s.pos, s.crd, s.val)
        cs, vs = oracle.unpack(s)
        # densify what unpack lists: must be the dense tensor exactly
        assert np.array_equal(_dense_of(dims, cs, vs), ref), (lt, ord)
        # storage order is lexicographic in level coordinates
        lv = np.stack([cs[ord[l]] for l in range(rank)], axis=1)
        assert lv.tolist() == sorted(lv.tolist())
        # every input entry is where entry_pos says
        assert np.array_equal(s.val[s.entry_pos], coo.vals)
        for d in range(rank):
            assert np.array_equal(cs[d][s.entry_pos], coo.coords[d])
        if all(t == 1 for t in lt):
            assert sorted(zip(*[c.tolist() for c in cs], vs.tolist())) == key_in
        count += 1
    assert count == 2 ** rank * len(list(itertools.permutations(range(rank))))  # 2^d * d! (Section 4.1)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_csr_csc_match_scipy(oracle, seed):
    coo = I.uniform_matrix(37, 53, 211, seed)
    m = sp.coo_matrix((coo.vals, (coo.coords[0], coo.coords[1])), shape=coo.dims)
    csr = m.tocsr(); csr.sort_indices()
    s = oracle.pack(coo.dims, coo.coords, coo.vals, (0, 1))
    assert np.array_equal(s.pos[1], csr.indptr) and np.array_equal(s.crd[1], csr.indices)
    assert np.array_equal(s.val, csr.data)
    csc = m.tocsc(); csc.sort_indices()
    s = oracle.pack(coo.dims, coo.coords, coo.vals, (0, 1), (1, 0))
    assert np.array_equal(s.pos[1], csc.indptr) and np.array_equal(s.crd[1], csc.indices)
    assert np.array_equal(s.val, csc.data)


def test_csr_is_prefix_sum_of_row_histogram_and_dcsr_drops_empty_rows(oracle):
    coo = I.confined_rows_matrix(200, 64, 300, 0.1, seed=3)
    s = oracle.pack(coo.dims, coo.coords, coo.vals, (0, 1))
    hist = np.bincount(coo.coords[0], minlength=200)
    assert np.array_equal(s.pos[1], np.concatenate([[0], np.cumsum(hist)]))
    d = oracle.pack(coo.dims, coo.coords, coo.vals, (1, 1))
    rows = np.flatnonzero(hist)
    assert np.array_equal(d.crd[0], rows) and np.array_equal(d.pos[0], [0, rows.size])
    assert np.array_equal(d.pos[1], np.concatenate([[0], np.cumsum(hist[rows])]))
    assert np.array_equal(d.crd[1], s.crd[1]) and np.array_equal(d.val, s.val)


def test_three_cycle_ordering_reading(oracle):
    # Reading used here: ord[l] names the logical dimension stored at level l.
    # With ord = (2, 0, 1) level 0 must hold the coordinates of logical dim 2.
    dims = (2, 3, 5)
    coords = [np.array([1, 0]), np.array([2, 1]), np.array([4, 0])]
    s = oracle.pack(dims, coords, [10.0, 20.0], (1, 1, 1), (2, 0, 1))
    assert s.crd[0].tolist() == [0, 4] and s.crd[1].tolist() == [0, 1] and s.crd[2].tolist() == [1, 2]
    assert s.val.tolist() == [20.0, 10.0]


def test_duplicates_sum_in_input_order_and_zeros_kept(oracle):
    coords = [np.array([1, 0, 1, 1]), np.array([2, 0, 2, 2])]
    vals = np.array([1e16, 0.0, 1.0, -1e16])
    s = oracle.pack((2, 3), coords, vals, (0, 1))
    assert s.crd[1].tolist() == [0, 2] and s.pos[1].tolist() == [0, 1, 2]
    assert s.val.tolist() == [0.0, (1e16 + 1.0) - 1e16]     # explicit zero kept; (a+b)+c order
    assert s.entry_pos.tolist() == [1, 0, 1, 1]


def test_bad_arguments(oracle):
    with pytest.raises(ValueError):
        oracle.pack((2, 2), [[0], [2]], [1.0], (0, 1))
    with pytest.raises(ValueError):
        oracle.pack((2, 2), [[0], [1]], [1.0], (0, 1), (0, 0))


def test_empty(oracle):
    s = oracle.pack((4, 5), [[], []], [], (0, 1))
    assert s.pos[1].tolist() == [0] * 5 and s.crd[1].size == 0 and s.val.size == 0
    s = oracle.pack((4, 5), [[], []], [], (1, 1))
    assert s.pos[0].tolist() == [0, 0] and s.pos[1].tolist() == [0]


def test_min_widths_follow_the_largest_position_and_level_size(oracle):
    # Section 4.1: a width must hold the largest position / coordinate.  Hand-computed cases:
    # 255 entries in a 256-long vector fit 8 bits; 256 entries need 16-bit positions; a level of
    # size 257 needs 16-bit coordinates even if only coordinate 0 is stored.
    v = oracle.pack((256,), [np.arange(255)], np.ones(255), (1,))
    assert oracle.min_widths(v) == (8, 8)
    v = oracle.pack((256,), [np.arange(256)], np.ones(256), (1,))
    assert oracle.min_widths(v) == (16, 8)
    v = oracle.pack((257,), [np.zeros(1, np.int64)], np.ones(1), (1,))
    assert oracle.min_widths(v) == (8, 16)
    m = oracle.pack((3, 1 << 33), [np.array([0, 2]), np.array([5, 1 << 32])], np.ones(2), (0, 1))
    assert oracle.min_widths(m) == (8, 64)
    d = oracle.pack((300, 300), [np.array([0]), np.array([0])], np.ones(1), (0, 0))
    assert oracle.min_widths(d) == (8, 8)          # dense levels store no overhead at all
