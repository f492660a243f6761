"""CPU oracle: test infrastructure only.

numpy-facing wrappers around ``oracle.c`` (see its header for what each
function follows in the paper).  Nothing here imports or calls the CUDA
library, and no product code may import this package: only tests, the smoke
check and the benchmark's CPU-baseline leg do.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass

import numpy as np

from .build import build as _build

DENSE, COMPRESSED = 0, 1
_MAXR = 8
_P64 = C.POINTER(C.c_int64)
_PD = C.POINTER(C.c_double)


class _Storage(C.Structure):
    _fields_ = [("rank", C.c_int), ("npos", C.c_int64 * _MAXR), ("ncrd", C.c_int64 * _MAXR),
                ("pos", _P64 * _MAXR), ("crd", _P64 * _MAXR), ("nval", C.c_int64), ("val", _PD),
                ("entry_pos", _P64)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build())
        _lib.orc_unpack.restype = C.c_int64
    return _lib


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _ptr(a, t=_P64):
    return a.ctypes.data_as(t)


@dataclass
class Storage:
    """pos[l] / crd[l] are int64 arrays (None at dense levels); val is f64."""
    dims: tuple
    lt: tuple
    ord: tuple
    pos: list
    crd: list
    val: np.ndarray
    entry_pos: np.ndarray


def pack(dims, coords, vals, lt, ord=None) -> Storage:
    """Section 4.1 storage from a coordinate list (coords[d] per logical dim)."""
    rank = len(dims)
    ord = tuple(range(rank)) if ord is None else tuple(int(o) for o in ord)
    cs = [_i64(c) for c in coords]
    v = _f64(vals)
    nnz = v.size
    carr = (_P64 * rank)(*[_ptr(c) for c in cs])
    st = _Storage()
    rc = lib().orc_pack(C.c_int(rank), _ptr(_i64(dims)), C.c_int64(nnz), carr, _ptr(v, _PD),
                        (C.c_int * rank)(*[int(t) for t in lt]), (C.c_int * rank)(*ord), C.byref(st))
    if rc != 0:
        lib().orc_free_storage(C.byref(st))
        raise ValueError({-1: "invalid argument", -2: "coordinate out of range", -3: "out of memory"}.get(rc, rc))
    pos, crd = [], []
    for l in range(rank):
        if lt[l] == COMPRESSED:
            pos.append(np.ctypeslib.as_array(st.pos[l], (st.npos[l],)).copy())
            crd.append(np.ctypeslib.as_array(st.crd[l], (st.ncrd[l],)).copy() if st.ncrd[l] else np.empty(0, np.int64))
        else:
            pos.append(None)
            crd.append(None)
    val = np.ctypeslib.as_array(st.val, (st.nval,)).copy() if st.nval else np.empty(0, np.float64)
    ep = np.ctypeslib.as_array(st.entry_pos, (nnz,)).copy() if nnz else np.empty(0, np.int64)
    lib().orc_free_storage(C.byref(st))
    return Storage(tuple(int(d) for d in dims), tuple(int(t) for t in lt), ord, pos, crd, val, ep)


def min_widths(s: Storage):
    """Section 4.1's rule on pointerBitWidth / indexBitWidth: a width is usable when the largest stored
    position (resp. coordinate) fits it.  Returns the smallest admissible (position, coordinate) widths
    among 8, 16, 32, 64; the coordinate bound is the level size, not the largest coordinate present."""
    pmax = max([int(p.max()) for p in s.pos if p is not None and p.size] + [0])
    cmax = max([int(s.dims[s.ord[l]]) - 1 for l in range(len(s.dims)) if s.lt[l] == COMPRESSED] + [0])
    fit = lambda v: next(w for w in (8, 16, 32, 64) if v < (1 << w))
    return fit(pmax), fit(cmax)


def unpack(s: Storage):
    """Stored entries in storage order as (logical coords per dim, values)."""
    rank = len(s.dims)
    st = _Storage()
    st.rank = rank
    keep = []
    for l in range(rank):
        if s.lt[l] == COMPRESSED:
            p, c = _i64(s.pos[l]), _i64(s.crd[l])
            keep += [p, c]
            st.pos[l], st.crd[l] = _ptr(p), _ptr(c)
            st.npos[l], st.ncrd[l] = p.size, c.size
    v = _f64(s.val)
    st.val, st.nval = _ptr(v, _PD), v.size
    outs = [np.empty(v.size, np.int64) for _ in range(rank)]
    vo = np.empty(v.size, np.float64)
    n = lib().orc_unpack(C.byref(st), _ptr(_i64(s.dims)), (C.c_int * rank)(*s.lt), (C.c_int * rank)(*s.ord),
                         (_P64 * rank)(*[_ptr(o) for o in outs]), _ptr(vo, _PD))
    assert n == v.size
    return outs, vo


def _slots(rows, m):
    if rows is None:
        return None, m
    rows = _i64(rows)
    slot = np.full(m, -1, np.int64)
    slot[rows] = np.arange(rows.size)
    return slot, rows.size


def spmm(m, ai, ak, av, B, rows=None):
    """C = A * B over the coordinate list; returns (C, bound) for all rows or the listed ones."""
    B = _f64(B)
    N = B.shape[1]
    slot, ns = _slots(rows, m)
    Cm = np.empty((ns, N)); bd = np.empty((ns, N))
    ai, ak, av = _i64(ai), _i64(ak), _f64(av)
    rc = lib().orc_spmm(C.c_int64(av.size), _ptr(ai), _ptr(ak), _ptr(av, _PD), _ptr(B, _PD), C.c_int64(N),
                        C.c_int64(N), _ptr(slot) if slot is not None else None, C.c_int64(ns),
                        _ptr(Cm, _PD), _ptr(bd, _PD))
    assert rc == 0
    return Cm, bd


def spmv(m, ai, ak, av, x, rows=None):
    y, b = spmm(m, ai, ak, av, _f64(x).reshape(-1, 1), rows)
    return y[:, 0], b[:, 0]


def sddmm(si, sj, sv, A, B):
    """x_e = S_e * sum_k A[i_e,k] B[k,j_e], one value per listed entry (input order)."""
    A, B = _f64(A), _f64(B)
    si, sj, sv = _i64(si), _i64(sj), _f64(sv)
    x = np.empty(sv.size); bd = np.empty(sv.size)
    rc = lib().orc_sddmm(C.c_int64(sv.size), _ptr(si), _ptr(sj), _ptr(sv, _PD), _ptr(A, _PD), C.c_int64(A.shape[1]),
                         _ptr(B, _PD), C.c_int64(B.shape[1]), C.c_int64(A.shape[1]), _ptr(x, _PD), _ptr(bd, _PD))
    assert rc == 0
    return x, bd


def mttkrp(I, ti, tj, tk, tv, B, Cf, rows=None):
    """M[i,r] = sum T[i,j,k] B[j,r] C[k,r]; returns (M, bound)."""
    B, Cf = _f64(B), _f64(Cf)
    R = B.shape[1]
    slot, ns = _slots(rows, I)
    M = np.empty((ns, R)); bd = np.empty((ns, R))
    ti, tj, tk, tv = _i64(ti), _i64(tj), _i64(tk), _f64(tv)
    rc = lib().orc_mttkrp(C.c_int64(tv.size), _ptr(ti), _ptr(tj), _ptr(tk), _ptr(tv, _PD), _ptr(B, _PD),
                          _ptr(Cf, _PD), C.c_int64(R), _ptr(slot) if slot is not None else None, C.c_int64(ns),
                          _ptr(M, _PD), _ptr(bd, _PD))
    assert rc == 0
    return M, bd


def spmspm(m, kdim, n, ai, ak, av, bk, bj, bv):
    """C = A * B, all sparse: returns CSR (pos, crd, val) of C and the per-entry bound sum|a*b|."""
    ai, ak, av = _i64(ai), _i64(ak), _f64(av)
    bk, bj, bv = _i64(bk), _i64(bj), _f64(bv)
    f = lib().orc_spmspm
    f.restype = C.c_int64
    pos = np.zeros(m + 1, np.int64)
    args = [C.c_int64(m), C.c_int64(kdim), C.c_int64(n), C.c_int64(av.size), _ptr(ai), _ptr(ak), _ptr(av, _PD),
            C.c_int64(bv.size), _ptr(bk), _ptr(bj), _ptr(bv, _PD), _ptr(pos)]
    total = f(*args, None, None, None)
    assert total >= 0
    crd = np.empty(total, np.int64); val = np.empty(total); bd = np.empty(total)
    total2 = f(*args, _ptr(crd), _ptr(val, _PD), _ptr(bd, _PD))
    assert total2 == total
    return pos, crd, val, bd


def vec_dot(ai, av, bi, bv):
    """Inner product of two sparse vectors given as sorted (coordinates, values); returns (x, bound)."""
    ai, av, bi, bv = _i64(ai), _f64(av), _i64(bi), _f64(bv)
    f = lib().orc_vec_dot
    f.restype = C.c_double
    bd = C.c_double()
    x = f(C.c_int64(av.size), _ptr(ai), _ptr(av, _PD), C.c_int64(bv.size), _ptr(bi), _ptr(bv, _PD), C.byref(bd))
    return float(x), float(bd.value)


# ---------------------------------------------------------------------------
# The same products as loop nests over packed storage, outer loop on all host cores
# (the "N cores" leg of the CPU baseline).  s: a Storage from pack().  Each returns
# (result, threads used).
# ---------------------------------------------------------------------------
def _rowmajor_matrix(s: Storage):
    if len(s.dims) != 2 or s.ord != (0, 1) or s.lt[1] != COMPRESSED:
        raise ValueError("row-major (dense|compressed, compressed) storage expected")
    rowid = _i64(s.crd[0]) if s.lt[0] == COMPRESSED else None
    pos1, crd1 = _i64(s.pos[1]), _i64(s.crd[1])
    return rowid, pos1, crd1, pos1.size - 1


def par_spmm(s: Storage, B):
    B = _f64(B)
    N = B.shape[1]
    rowid, pos1, crd1, nstored = _rowmajor_matrix(s)
    Cm = np.zeros((s.dims[0], N))
    v = _f64(s.val)
    nt = lib().orc_par_spmm(C.c_int64(nstored), _ptr(rowid) if rowid is not None else None, _ptr(pos1), _ptr(crd1),
                            _ptr(v, _PD), _ptr(B, _PD), C.c_int64(N), C.c_int64(N), _ptr(Cm, _PD), C.c_int64(N))
    return Cm, nt


def par_spmv(s: Storage, x):
    y, nt = par_spmm(s, _f64(x).reshape(-1, 1))
    return y[:, 0], nt


def par_sddmm(s: Storage, A, B):
    A, B = _f64(A), _f64(B)
    rowid, pos1, crd1, nstored = _rowmajor_matrix(s)
    v = _f64(s.val)
    x = np.zeros(v.size)
    nt = lib().orc_par_sddmm(C.c_int64(nstored), _ptr(rowid) if rowid is not None else None, _ptr(pos1), _ptr(crd1),
                             _ptr(v, _PD), _ptr(A, _PD), C.c_int64(A.shape[1]), _ptr(B, _PD), C.c_int64(B.shape[1]),
                             C.c_int64(A.shape[1]), _ptr(x, _PD))
    return x, nt


def par_mttkrp(s: Storage, B, Cf):
    if len(s.dims) != 3 or s.ord != (0, 1, 2) or s.lt[1] != COMPRESSED or s.lt[2] != COMPRESSED:
        raise ValueError("(dense|compressed, compressed, compressed) storage in identity order expected")
    B, Cf = _f64(B), _f64(Cf)
    R = B.shape[1]
    crd0 = _i64(s.crd[0]) if s.lt[0] == COMPRESSED else None
    pos1, crd1, pos2, crd2, v = _i64(s.pos[1]), _i64(s.crd[1]), _i64(s.pos[2]), _i64(s.crd[2]), _f64(s.val)
    M = np.zeros((s.dims[0], R))
    nt = lib().orc_par_mttkrp(C.c_int64(pos1.size - 1), _ptr(crd0) if crd0 is not None else None, _ptr(pos1), _ptr(crd1),
                              _ptr(pos2), _ptr(crd2), _ptr(v, _PD), _ptr(B, _PD), _ptr(Cf, _PD), C.c_int64(R), _ptr(M, _PD))
    return M, nt
